// hs_entropy_quantify: one launch.
//
// Stage 1 (every CTA): a CTA owns one chunk of one logits row (up to 32 KiB), brings it on chip in
// one piece and reduces max / sum e^x / sum x e^x with warp shuffles.  Staged variant (the default):
// one bulk copy into shared memory, issued by one thread before the dependency wait; the passes read
// shared memory, so a thread needs few registers and four CTAs share an SM (at one tree every CTA of
// the launch is resident at once: no row waits for a second wave).  Register variant (the
// allocation-free entry point, and rows a caller of the launcher hands over unaligned: the C entry
// point rejects those): 16-byte coalesced loads that are all issued before the first use, two CTAs per SM.  The Top-K of the chunk is found without sorting: the K-th largest of 32 group maxima
// is a lower bound of the chunk's K-th largest logit, only threads whose own maximum reaches it
// re-scan their registers, and the few candidates are ranked by counting.
// Stage 2 (last CTA of a row to arrive): merges the row's chunk partials into max, log-sum-exp,
// Shannon entropy, Top-K and the two Top-K entropies (Eq. 1 inner sum).
// Stage 3 (last row of a tree to arrive): path confidence ln V_i (Sec. 2.2), cumulative
// meta-path Top-K entropy Phi (Eq. 1) and the operational path P* (Sec. 4.1) of that tree.
#include <math_constants.h>

#include <mutex>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

#define CAND_CAP 512
#define LOG2E 1.4426950408889634f

struct QuantParams {
    const void* logits;
    int64_t row_stride;
    int vocab;
    int nvec;        // 16-byte vectors per row, the last one may be partial
    int chunks;      // CTAs per row
    int chunk_vecs;  // vectors per chunk
    int rows;
    int batch;
    const int* node_off;
    const int* parent;
    const int* token;
    hs_quant_out out;
    float4* part_stats;             // [rows*chunks] {max, sum e, sum e*x, -}
    unsigned long long* part_keys;  // [rows*chunks*HS_MAX_TOPK]
    int* row_cnt;
    int* tree_cnt;
    int K, d_base, phi_mode, pstar_mode, entropy_mode, is_bf16;
    int* err;        // sticky device error word (a bounded wait that expired)
};

template <bool BF16>
__device__ __forceinline__ void unpack(const uint4& v, float* x) {
    if (BF16) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    } else {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
}

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Rank candidates s_cand[0..n) by key (all distinct, 0 = empty) and write the K best to s_top.
__device__ __forceinline__ void rank_select(const unsigned long long* s_cand, int n, int K,
                                            unsigned long long* s_top) {
    for (int t = threadIdx.x; t < n; t += blockDim.x) {
        unsigned long long k = s_cand[t];
        if (k == 0ull) continue;
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (s_cand[j] > k);
        if (rank < K) s_top[rank] = k;
    }
}

// Cold path of the chunk Top-K: K block-wide arg-max rounds over the chunk, each restricted to keys
// below the previous winner.  Exact for any number of ties.
template <bool BF16>
__device__ __noinline__ void topk_by_rounds(const char* rowp, int v0, int v1, int vocab, int K,
                                            unsigned long long* s_top, unsigned long long* s_red) {
    constexpr int VE = BF16 ? 8 : 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long last = ~0ull;
    for (int r = 0; r < K; ++r) {
        unsigned long long best = 0ull;
        for (int v = v0 + tid; v < v1; v += HS_ROW_THREADS) {
            uint4 dv = __ldg((const uint4*)(rowp) + v);
            float x[8];
            unpack<BF16>(dv, x);
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                if (v * VE + e < vocab) {
                    unsigned long long k = make_key(x[e], v * VE + e);
                    if (k < last && k > best) best = k;
                }
            }
        }
        best = warp_max_u64(best);
        if (lane == 0) s_red[warp] = best;
        __syncthreads();
        best = s_red[0];
        for (int w = 1; w < 8; ++w) best = s_red[w] > best ? s_red[w] : best;
        if (tid == 0) s_top[r] = best;
        last = best;
        __syncthreads();
        if (best == 0ull) break;
    }
}

__device__ void tree_scores(const QuantParams& p, int b, float* s_f, int* s_i);

// MODE 0: register variant; 1: staged, loops over the vectors unrolled; 2: staged, loops rolled
template <bool BF16, int MODE>
__global__ void __launch_bounds__(HS_ROW_THREADS, MODE ? 4 : 2) quantify_kernel(const QuantParams p) {
    constexpr bool STAGED = MODE != 0;
    constexpr int VE = BF16 ? 8 : 4;
    constexpr int VPT = HS_ROW_VPT;
    extern __shared__ __align__(16) unsigned char s_stage[];   // STAGED: the chunk, HS_ROW_THREADS * VPT vectors
    __shared__ unsigned long long s_bar;
    __shared__ unsigned long long s_cand[CAND_CAP];
    __shared__ unsigned long long s_top[HS_MAX_TOPK];
    __shared__ unsigned long long s_red[8];
    __shared__ float s_gm[32];
    __shared__ float s_w[8][3];
    __shared__ int s_cnt;
    __shared__ int s_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x, row = blockIdx.y;
    const int K = p.K;
    const char* rowp = (const char*)p.logits + (size_t)row * p.row_stride * (BF16 ? 2 : 4);
    const int v0 = chunk * p.chunk_vecs;
    const int v1 = min(v0 + p.chunk_vecs, p.nvec);

    if (tid < HS_MAX_TOPK) s_top[tid] = 0ull;
    if (tid == 0) s_cnt = 0;

    // ---- the chunk comes on chip: one bulk copy (STAGED) or all loads first ---------------------------
    const unsigned int ninf = BF16 ? 0xff80ff80u : 0xff800000u;
    uint4 d[STAGED ? 1 : VPT];
    const uint4* sv = reinterpret_cast<const uint4*>(s_stage);
    if (STAGED) {
        const unsigned int bar = smem_u32(&s_bar);
        if (tid == 0) {
            mbar_init(bar, 1);
            mbar_init_fence();
            const unsigned int bytes = (unsigned int)max(v1 - v0, 0) * 16u;
            mbar_expect_tx(bar, bytes);
            if (bytes) bulk_load(smem_u32(s_stage), (const uint4*)(rowp) + v0, bytes, bar);
        }
        pdl_launch_dependents();
        pdl_wait();        // the copy above is in flight; partials and outputs may still be in use upstream
        __syncthreads();   // the barrier is initialised
        mbar_wait(bar, 0u, p.err);
    } else {
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            int v = v0 + tid + j * HS_ROW_THREADS;
            d[STAGED ? 0 : j] = (v < v1) ? __ldcs((const uint4*)(rowp) + v) : make_uint4(ninf, ninf, ninf, ninf);
        }
        pdl_launch_dependents();
        pdl_wait();        // the loads above are in flight; partials and outputs may still be in use upstream
    }
    // vector j of this thread: from shared memory or from its registers
    auto vec = [&](int j) -> uint4 {
        if (STAGED) {
            const int v = tid + j * HS_ROW_THREADS;
            return (v0 + v < v1) ? sv[v] : make_uint4(ninf, ninf, ninf, ninf);
        }
        return d[STAGED ? 0 : j];
    };
    // ---- maxima ---------------------------------------------------------------------------
    // Rolled loops over the vectors need 40 registers instead of 64, so six CTAs share an SM: measured 20 % faster
    // on launches of many waves, 3 us slower on a launch that is resident at once (the launcher chooses).  The
    // candidate scan is rolled in both staged variants: few threads run it, mostly from a cold instruction cache.
    constexpr int UJ = MODE == 2 ? 2 : VPT, UC = MODE != 0 ? 1 : VPT;
    float vmax[STAGED ? 1 : VPT];
    float tmax = -CUDART_INF_F;
#pragma unroll UJ
    for (int j = 0; j < VPT; ++j) {
        float x[8];
        unpack<BF16>(vec(j), x);
        int v = v0 + tid + j * HS_ROW_THREADS;
        if (v == p.nvec - 1) {                       // the row's last vector may run past vocab
#pragma unroll
            for (int e = 0; e < VE; ++e)
                if (v * VE + e >= p.vocab) x[e] = -CUDART_INF_F;
        }
        float m = x[0];
#pragma unroll
        for (int e = 1; e < VE; ++e) m = fmaxf(m, x[e]);
        if (!STAGED) vmax[STAGED ? 0 : j] = m;
        tmax = fmaxf(tmax, m);
    }
    // ---- sums relative to the thread's own maximum ------------------------------------------
    const float nml = (tmax == -CUDART_INF_F) ? 0.f : -tmax * LOG2E;
    float s = 0.f, u = 0.f;
#pragma unroll UJ
    for (int j = 0; j < VPT; ++j) {
        float x[8];
        unpack<BF16>(vec(j), x);
        int v = v0 + tid + j * HS_ROW_THREADS;
        if (v == p.nvec - 1) {
#pragma unroll
            for (int e = 0; e < VE; ++e)
                if (v * VE + e >= p.vocab) x[e] = -CUDART_INF_F;
        }
#pragma unroll
        for (int e = 0; e < VE; ++e) {
            float xc = fmaxf(x[e], -1e30f);
            float ev = ex2f(fmaf(xc, LOG2E, nml));
            s += ev;
            u = fmaf(ev, xc, u);
        }
    }
    // ---- warp / block reduction of (max, s, u) ------------------------------------------------
    {
        float wm = warp_max(tmax);
        float f = (tmax == -CUDART_INF_F) ? 0.f : ex2f((tmax - wm) * LOG2E);
        float ws = warp_sum(s * f), wu = warp_sum(u * f);
        if (lane == 0) { s_w[warp][0] = wm; s_w[warp][1] = ws; s_w[warp][2] = wu; }
        float g = tmax;
        g = fmaxf(g, __shfl_xor_sync(HS_FULL_MASK, g, 1));
        g = fmaxf(g, __shfl_xor_sync(HS_FULL_MASK, g, 2));
        g = fmaxf(g, __shfl_xor_sync(HS_FULL_MASK, g, 4));
        if ((lane & 7) == 0) s_gm[warp * 4 + (lane >> 3)] = g;
    }
    __syncthreads();
    if (warp == 0) {       // the eight warps' (max, s, u): lanes 0..7 of warp 0, shuffle reductions
        const float wm = lane < 8 ? s_w[lane & 7][0] : -CUDART_INF_F;
        float M = wm;
        M = fmaxf(M, __shfl_xor_sync(HS_FULL_MASK, M, 1));
        M = fmaxf(M, __shfl_xor_sync(HS_FULL_MASK, M, 2));
        M = fmaxf(M, __shfl_xor_sync(HS_FULL_MASK, M, 4));
        const float f = (lane >= 8 || wm == -CUDART_INF_F) ? 0.f : ex2f((wm - M) * LOG2E);
        float S = s_w[lane & 7][1] * f, U = s_w[lane & 7][2] * f;
        // the serial order w = 0..7 of the sum is kept (the result does not depend on the launch shape)
        float St = 0.f, Ut = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            St += __shfl_sync(HS_FULL_MASK, S, w);
            Ut += __shfl_sync(HS_FULL_MASK, U, w);
        }
        if (lane == 0) p.part_stats[(size_t)row * p.chunks + chunk] = make_float4(M, St, Ut, 0.f);
    }
    // ---- Top-K of the chunk -------------------------------------------------------------------
    float tau;
    {
        float v = s_gm[lane];
        int ge = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) ge += (__shfl_sync(HS_FULL_MASK, v, j) >= v);
        tau = warp_max(ge >= K ? v : -CUDART_INF_F);   // K-th largest group maximum
    }
    if (tmax >= tau && tmax > -CUDART_INF_F) {
#pragma unroll UC
        for (int j = 0; j < VPT; ++j) {
            if (STAGED || vmax[STAGED ? 0 : j] >= tau) {
                float x[8];
                unpack<BF16>(vec(j), x);
                int base = (v0 + tid + j * HS_ROW_THREADS) * VE;
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    if (x[e] >= tau && base + e < p.vocab) {
                        int slot = atomicAdd(&s_cnt, 1);
                        if (slot < CAND_CAP) s_cand[slot] = make_key(x[e], base + e);
                    }
                }
            }
        }
    }
    __syncthreads();
    const int ncand = s_cnt;
    if (ncand <= CAND_CAP) {
        rank_select(s_cand, ncand, K, s_top);
    } else {
        // Heavy ties (e.g. a constant row): K rounds of "largest key below the previous one",
        // re-reading the chunk from global memory (cold path).
        topk_by_rounds<BF16>(rowp, v0, v1, p.vocab, K, s_top, s_red);
    }
    __syncthreads();
    if (tid < HS_MAX_TOPK)
        p.part_keys[((size_t)row * p.chunks + chunk) * HS_MAX_TOPK + tid] = (tid < K) ? s_top[tid] : 0ull;

    // ---- stage 2: the last chunk of this row merges -----------------------------------------------
    // (the CTA's stores are ordered before thread 0's fence by the barrier, the fence before its arrival)
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_flag = (atomicAdd(&p.row_cnt[row], 1) == p.chunks - 1);
        __threadfence();
    }
    __syncthreads();
    if (!s_flag) return;
    const int nk = p.chunks * HS_MAX_TOPK;     // <= CAND_CAP, checked by the launcher
    for (int t = tid; t < nk; t += HS_ROW_THREADS)
        s_cand[t] = __ldcg(&p.part_keys[(size_t)row * p.chunks * HS_MAX_TOPK + t]);
    if (tid < HS_MAX_TOPK) s_top[tid] = 0ull;
    __syncthreads();
    rank_select(s_cand, nk, K, s_top);
    __syncthreads();
    if (warp == 0) {
        float m = -CUDART_INF_F, cs = 0.f, cu = 0.f;
        if (lane < p.chunks) {
            float4 st = __ldcg(&p.part_stats[(size_t)row * p.chunks + lane]);
            m = st.x; cs = st.y; cu = st.z;
        }
        float M = warp_max(m);
        float f = (m == -CUDART_INF_F) ? 0.f : ex2f((m - M) * LOG2E);
        float S = warp_sum(cs * f), U = warp_sum(cu * f);
        float lse = M + logf(S);
        float H = lse - U / S;
        // Top-K entropies: lanes 0..K-1 hold one entry each
        unsigned long long key = (lane < K) ? s_top[lane] : 0ull;
        bool valid = key != 0ull;
        float tv = valid ? key_value(key) : 0.f;
        float t0 = __shfl_sync(HS_FULL_MASK, tv, 0);
        float pv = valid ? expf(tv - lse) : 0.f;
        float itr = warp_sum(valid ? -pv * (tv - lse) : 0.f);
        float z = valid ? expf(tv - t0) : 0.f;
        float Z = warp_sum(z);
        float itk = logf(Z) - warp_sum(valid ? z * (tv - t0) : 0.f) / Z;
        if (lane < K) {
            p.out.topk_val[(size_t)row * K + lane] = valid ? tv : -CUDART_INF_F;
            p.out.topk_idx[(size_t)row * K + lane] = valid ? key_index(key) : -1;
        }
        if (lane == 0) {
            p.out.row_max[row] = M;
            p.out.row_lse[row] = lse;
            p.out.h_full[row] = fmaxf(H, 0.f);
            p.out.i_topk[row] = fmaxf(itk, 0.f);
            p.out.i_trunc[row] = itr;
            p.row_cnt[row] = 0;                 // ready for the next launch
        }
    }
    // sequences without any node never reach stage 3: flag them here (first CTA only)
    if (row == 0) {
        for (int b = tid; b < p.batch; b += HS_ROW_THREADS)
            if (p.node_off[b + 1] <= p.node_off[b]) {
                p.out.status[b] = HS_ERR_BAD_TREE; p.out.pstar_node[b] = 0; p.out.phi_star[b] = 0.f;
            }
    }
    // ---- stage 3: the last row of this tree scores the tree -----------------------------------------
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        int lo = 0, hi = p.batch;               // largest b with node_off[b] <= row
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (p.node_off[mid] <= row) lo = mid; else hi = mid;
        }
        int n = p.node_off[lo + 1] - p.node_off[lo];
        int last = (atomicAdd(&p.tree_cnt[lo], 1) == n - 1);
        if (last) p.tree_cnt[lo] = 0;
        s_flag = last ? lo : -1;
        __threadfence();
    }
    __syncthreads();
    const int b = s_flag;
    if (b < 0) return;
    tree_scores(p, b, (float*)s_cand, (int*)(s_cand + 256));
}

// One CTA, n <= HS_MAX_NODES nodes.  s_f: 3*128 floats, s_i: 2*128 ints of shared memory.
__device__ void tree_scores(const QuantParams& p, int b, float* s_f, int* s_i) {
    __shared__ unsigned long long s_best[8];
    __shared__ int s_maxd[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int base = p.node_off[b];
    const int n = p.node_off[b + 1] - base;
    float* s_logc = s_f;
    float* s_I = s_f + HS_MAX_NODES;
    float* s_phi = s_f + 2 * HS_MAX_NODES;
    int* s_par = s_i;
    // validation
    int bad = (n > HS_MAX_NODES);
    int par = -1, tok = 0;
    if (!bad && tid < n) {
        par = p.parent[base + tid];
        tok = p.token[base + tid];
        if (tid == 0) bad = (par != -1);
        else bad = (par < 0 || par >= tid || tok < 0 || tok >= p.vocab);
    }
    bad = __syncthreads_or(bad);
    if (bad) {
        for (int i = tid; i < n; i += blockDim.x) {
            p.out.logc[base + i] = 0.f; p.out.score[base + i] = 0.f; p.out.phi[base + i] = 0.f;
            p.out.depth[base + i] = 0;
        }
        if (tid == 0) { p.out.status[b] = HS_ERR_BAD_TREE; p.out.pstar_node[b] = 0; p.out.phi_star[b] = 0.f; }
        return;
    }
    if (tid < n) {
        float lc = 0.f;
        if (tid > 0) {
            size_t off = (size_t)(base + par) * p.row_stride + tok;
            float lv = p.is_bf16 ? __bfloat162float(((const __nv_bfloat16*)p.logits)[off])
                                 : ((const float*)p.logits)[off];
            lc = lv - __ldcg(&p.out.row_lse[base + par]);
        }
        s_logc[tid] = lc;
        s_I[tid] = __ldcg(p.entropy_mode == 0 ? &p.out.i_topk[base + tid] : &p.out.i_trunc[base + tid]);
        s_par[tid] = par;
    }
    __syncthreads();
    float S = 0.f, Phi = 0.f;
    int dep = 0;
    if (tid < n) {
        int a = tid;
        while (a > 0) {
            int pa = s_par[a];
            S += s_logc[a];
            Phi += s_I[pa];
            a = pa;
            ++dep;
        }
        if (p.phi_mode == 1) Phi += s_I[tid];
        s_phi[tid] = Phi;
        p.out.logc[base + tid] = s_logc[tid];
        p.out.score[base + tid] = S;
        p.out.phi[base + tid] = Phi;
        p.out.depth[base + tid] = dep;
    }
    // deepest level, then P* among the nodes of depth min(d_base, deepest)
    int md = dep;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) md = max(md, __shfl_xor_sync(HS_FULL_MASK, md, o));
    if (lane == 0) s_maxd[warp] = md;
    __syncthreads();
    md = s_maxd[0];
    for (int w = 1; w < 8; ++w) md = max(md, s_maxd[w]);
    const int t_eval = min(p.d_base, md);
    unsigned long long key = 0ull;
    if (tid < n && dep == t_eval) key = make_key(p.pstar_mode == 0 ? s_logc[tid] : S, tid);
    key = warp_max_u64(key);
    if (lane == 0) s_best[warp] = key;
    __syncthreads();
    if (tid == 0) {
        unsigned long long best = s_best[0];
        for (int w = 1; w < 8; ++w) best = s_best[w] > best ? s_best[w] : best;
        int node = key_index(best);
        p.out.pstar_node[b] = node;
        p.out.phi_star[b] = s_phi[node];
        p.out.status[b] = HS_OK;
    }
}

hs_status hs_launch_quantify(hs_ctx* ctx, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                             int64_t row_stride, int32_t vocab, const hs_policy* policy,
                             const hs_quant_out* out, cudaStream_t stream) {
    QuantParams p;
    const int ve = hs_vec_elems(dtype);
    p.logits = logits;
    p.row_stride = row_stride;
    p.vocab = vocab;
    p.nvec = (vocab + ve - 1) / ve;
    p.chunks = hs_row_chunks(vocab, dtype);
    if (p.chunks * HS_MAX_TOPK > CAND_CAP || p.chunks > 32) return HS_ERR_SHAPE;
    p.chunk_vecs = (p.nvec + p.chunks - 1) / p.chunks;
    p.rows = tree->n_nodes_total;
    p.batch = tree->batch;
    p.node_off = tree->node_off;
    p.parent = tree->parent;
    p.token = tree->token;
    p.out = *out;
    size_t stats_bytes = hs_align_up((size_t)p.rows * p.chunks * sizeof(float4), 256);
    size_t keys_bytes = (size_t)p.rows * p.chunks * HS_MAX_TOPK * sizeof(unsigned long long);
    if (stats_bytes + keys_bytes > ctx->scratch_bytes) return HS_ERR_WORKSPACE;
    p.part_stats = (float4*)ctx->scratch;
    p.part_keys = (unsigned long long*)(ctx->scratch + stats_bytes);
    p.row_cnt = ctx->counters + HS_CNT_QUANT_ROW;
    p.tree_cnt = ctx->counters + HS_CNT_QUANT_TREE;
    p.K = policy->top_k;
    p.d_base = policy->d_base;
    p.phi_mode = policy->phi_mode;
    p.pstar_mode = policy->pstar_mode;
    p.entropy_mode = policy->entropy_mode;
    p.is_bf16 = dtype == HS_BF16;
    p.err = ctx->counters + HS_CNT_ERROR;
    dim3 grid(p.chunks, p.rows);
    // the bulk copy wants 16-byte aligned rows
    const size_t esz = dtype == HS_BF16 ? 2 : 4;
    const bool staged = ((uintptr_t)logits % 16 == 0) && ((size_t)row_stride * esz % 16 == 0);
    const size_t stage_bytes = (size_t)HS_ROW_THREADS * HS_ROW_VPT * 16;
    const bool many_waves = (long long)p.chunks * p.rows > 4ll * ctx->sm_count;
    cudaError_t e;
    if (staged && many_waves)
        e = dtype == HS_BF16
            ? hs_launch(quantify_kernel<true, 2>, grid, dim3(HS_ROW_THREADS), stage_bytes, stream, ctx->pdl, dim3(1, 1, 1), p)
            : hs_launch(quantify_kernel<false, 2>, grid, dim3(HS_ROW_THREADS), stage_bytes, stream, ctx->pdl, dim3(1, 1, 1), p);
    else if (staged)
        e = dtype == HS_BF16
            ? hs_launch(quantify_kernel<true, 1>, grid, dim3(HS_ROW_THREADS), stage_bytes, stream, ctx->pdl, dim3(1, 1, 1), p)
            : hs_launch(quantify_kernel<false, 1>, grid, dim3(HS_ROW_THREADS), stage_bytes, stream, ctx->pdl, dim3(1, 1, 1), p);
    else
        e = dtype == HS_BF16
            ? hs_launch(quantify_kernel<true, 0>, grid, dim3(HS_ROW_THREADS), 0, stream, ctx->pdl, dim3(1, 1, 1), p)
            : hs_launch(quantify_kernel<false, 0>, grid, dim3(HS_ROW_THREADS), 0, stream, ctx->pdl, dim3(1, 1, 1), p);
    return e == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

// ---- hs_entropy_quantify_static: the same pass without any allocated workspace -------------------------------
//
// Some hosts of this library may not allocate device memory at all: a serving process that hands
// its whole memory budget to one arena at start-up, or code running under a capture / real-time
// rule that forbids cudaMalloc.  For them the chunk partials and arrival counters of the pass live
// in one fixed array that is part of the library image, so every GPU that loads the library carries
// HS_STATIC_SCRATCH_BYTES of it until the process exits.
#define HS_STATIC_MAX_CHUNKS 16
#define HS_STATIC_COUNTER_BYTES 2048    // (HS_STATIC_MAX_ROWS + HS_STATIC_MAX_BATCH) ints, rounded up
#define HS_STATIC_STATS_BYTES (HS_STATIC_MAX_ROWS * HS_STATIC_MAX_CHUNKS * 16)
#define HS_STATIC_KEYS_BYTES (HS_STATIC_MAX_ROWS * HS_STATIC_MAX_CHUNKS * HS_MAX_TOPK * 8)
#define HS_STATIC_SCRATCH_BYTES (HS_STATIC_COUNTER_BYTES + HS_STATIC_STATS_BYTES + HS_STATIC_KEYS_BYTES)
#define HS_STATIC_MAX_DEVICES 64

static __device__ __align__(256) unsigned char g_static_scratch[HS_STATIC_SCRATCH_BYTES];
// Device address of g_static_scratch on each device.  In host code the symbol itself is only a
// handle, never an address a kernel may use: the address is asked for once per device.
static unsigned char* g_static_addr[HS_STATIC_MAX_DEVICES];
static std::mutex g_static_mutex;

extern "C" hs_status hs_entropy_quantify_static(const hs_tree_batch* tree, const void* draft_logits, hs_dtype dtype,
                                                int64_t row_stride, int32_t vocab, const hs_policy* policy,
                                                const hs_quant_out* out, hs_stream stream_) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!tree || !policy || !out || !draft_logits || ((uintptr_t)draft_logits & 15)) return HS_ERR_INVALID_ARG;
    if (dtype != HS_F32 && dtype != HS_BF16) return HS_ERR_INVALID_ARG;
    if (tree->batch < 1 || tree->n_nodes_total < tree->batch || !tree->node_off || !tree->parent || !tree->token)
        return HS_ERR_INVALID_ARG;
    const int ve = hs_vec_elems(dtype);
    if (vocab < 1 || row_stride < vocab || row_stride % ve != 0) return HS_ERR_INVALID_ARG;
    if (policy->top_k < 1 || policy->top_k > HS_MAX_TOPK || policy->d_base < 0 || policy->phi_mode < 0 ||
        policy->phi_mode > 1 || policy->pstar_mode < 0 || policy->pstar_mode > 1 || policy->entropy_mode < 0 ||
        policy->entropy_mode > 1)
        return HS_ERR_INVALID_ARG;
    if (!out->row_max || !out->row_lse || !out->h_full || !out->i_topk || !out->i_trunc || !out->topk_val ||
        !out->topk_idx || !out->logc || !out->score || !out->phi || !out->depth || !out->pstar_node ||
        !out->phi_star || !out->status)
        return HS_ERR_INVALID_ARG;
    const int chunks = hs_row_chunks(vocab, dtype);
    if (tree->n_nodes_total > HS_STATIC_MAX_ROWS || tree->batch > HS_STATIC_MAX_BATCH || chunks > HS_STATIC_MAX_CHUNKS)
        return HS_ERR_STATIC_LIMIT;

    int dev = -1;
    HS_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= HS_STATIC_MAX_DEVICES) return HS_ERR_UNSUPPORTED;
    unsigned char* base;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_addr[dev]) {              // first call on this device (it is the current one)
            void* sym = nullptr;
            if (cudaGetSymbolAddress(&sym, g_static_scratch) != cudaSuccess || !sym) return HS_ERR_CUDA;
            g_static_addr[dev] = (unsigned char*)sym;
        }
        base = g_static_addr[dev];
    }

    QuantParams p;
    p.logits = draft_logits;
    p.row_stride = row_stride;
    p.vocab = vocab;
    p.nvec = (vocab + ve - 1) / ve;
    p.chunks = chunks;
    p.chunk_vecs = (p.nvec + p.chunks - 1) / p.chunks;
    p.rows = tree->n_nodes_total;
    p.batch = tree->batch;
    p.node_off = tree->node_off;
    p.parent = tree->parent;
    p.token = tree->token;
    p.out = *out;
    p.row_cnt = (int*)base;
    p.tree_cnt = (int*)base + HS_STATIC_MAX_ROWS;
    p.part_stats = (float4*)(base + HS_STATIC_COUNTER_BYTES);
    p.part_keys = (unsigned long long*)(base + HS_STATIC_COUNTER_BYTES + HS_STATIC_STATS_BYTES);
    p.K = policy->top_k;
    p.d_base = policy->d_base;
    p.phi_mode = policy->phi_mode;
    p.pstar_mode = policy->pstar_mode;
    p.entropy_mode = policy->entropy_mode;
    p.is_bf16 = dtype == HS_BF16;
    // The array keeps whatever the previous call left: the arrival counters must start at zero.
    HS_CUDA_OK(cudaMemsetAsync(base, 0, HS_STATIC_COUNTER_BYTES, stream));
    dim3 grid(p.chunks, p.rows);
    p.err = nullptr;       // (the register variant has no bounded wait)
    if (dtype == HS_BF16) quantify_kernel<true, 0><<<grid, HS_ROW_THREADS, 0, stream>>>(p);
    else quantify_kernel<false, 0><<<grid, HS_ROW_THREADS, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
