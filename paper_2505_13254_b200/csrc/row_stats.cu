// hs_entropy_quantify: two launches.
//
// quantify_stream_kernel   The logits matrix is one long stream of 16-byte vectors (row after row) that is cut
//     into equal contiguous shares, one per CTA, one CTA per SM.  A producer warp brings the share on chip in
//     items of up to 32 KiB (bulk copies into a ring of shared-memory slots, completion on mbarriers); sixteen
//     consumer warps reduce each item in ONE pass: running maximum per thread (packed bf16 maxima), then
//     sum e^(x-m) and sum x e^(x-m) with the exponent's multiply-add and the two sums as packed fp32 pairs.
//     Top-K without sorting: after the first items of a row share a warp takes a lower bound of the K-th
//     largest logit of the row share from maxima of disjoint element sets (the 32 half-warp maxima of the
//     CTA, or its own 32 lane maxima on a short share), and only lanes whose window maximum reaches the bound
//     re-scan their vectors in shared memory and push candidates; the few candidates are ranked by counting.
//     A share that ends inside a row leaves a partial {max, sum, sum x e, K keys}; the last CTA of a row to
//     arrive merges the partials into max, log-sum-exp, Shannon entropy, Top-K and the two Top-K entropies
//     (Eq. 1 inner sum).  Rows that lie inside one share need no partial and no atomic.  With few rows every row
//     is cut into the same number of shares, which form a thread-block cluster: the partials then go into the
//     shared memory of the cluster's first CTA instead of through global memory.
// tree_scores_kernel       One CTA per sequence: path confidence ln V_i (Sec. 2.2), cumulative meta-path
//     Top-K entropy Phi (Eq. 1) and the operational path P* (Sec. 4.1).  (The fused call launches the kernel
//     of stratify_prune.cu that runs the same tree stage and then prunes, in its place.)
//
// quantify_chunk_kernel (a CTA owns one chunk of one row, registers only) serves the allocation-free entry.
#include <math_constants.h>

#include <mutex>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"
#include "tree_stage.cuh"

#define CAND_CAP 512
#define LOG2E 1.4426950408889634f

#define QS_CONSUMERS 512                      // sixteen consumer warps
#define QS_THREADS (QS_CONSUMERS + 32)        // + the producer warp
#define QS_ITEM_VECS 2048                     // vectors per item: 32 KiB, four per consumer thread
#define QS_VPT (QS_ITEM_VECS / QS_CONSUMERS)
#define QS_SLOTS 6                            // ring of item slots
#define QS_WINDOW 4                           // items a consumer holds before it hands their slots back
#define QS_MAX_SEGS 32                        // shares a row may be split over
#define QS_SMEM_BYTES (QS_SLOTS * QS_ITEM_VECS * 16 + 128)

struct QuantParams {
    const void* logits;
    int64_t row_stride;
    int vocab;
    int nvec;        // 16-byte vectors per row, the last one may be partial
    int chunks;      // chunk kernel: CTAs per row
    int chunk_vecs;  // chunk kernel: vectors per chunk
    int per;         // stream kernel: vectors per share
    int split;       // stream kernel: shares per row (row-split geometry), 0 = byte-balanced stream
    int extra;       // stream kernel, row split: the first `extra` rows have one share more
    int nslots;      // stream kernel: item slots in shared memory
    int clustered;   // stream kernel, row split: the shares of a row are one thread-block cluster and merge in shared memory
    int rows;
    int batch;
    const int* node_off;
    const int* parent;
    const int* token;
    hs_quant_out out;
    float4* part_stats;             // {max, sum e, sum e*x, -} per partial
    unsigned long long* part_keys;  // HS_MAX_TOPK keys per partial
    int* row_cnt;
    int K, d_base, phi_mode, pstar_mode, entropy_mode, is_bf16;
    int prefetch;    // the rows may be fetched before the dependency wait (the caller vouches that they are complete)
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

// Rank candidates s_cand[0..n) by key (all distinct, 0 = empty) and write the K best to s_top (zeroed before).
__device__ __forceinline__ void rank_select(const unsigned long long* s_cand, int n, int K,
                                            unsigned long long* s_top, int tid, int nthr) {
    for (int t = tid; t < n; t += nthr) {
        unsigned long long k = s_cand[t];
        if (k == 0ull) continue;
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (s_cand[j] > k);
        if (rank < K) s_top[rank] = k;
    }
}

// The same by whole warps: warp w takes candidates w, w + nwarp, ...; the 32 lanes compare 32 others at a time.
__device__ __forceinline__ void rank_select_warps(const unsigned long long* s_cand, int n, int K,
                                                  unsigned long long* s_top, int warp, int lane, int nwarp) {
    for (int c = warp; c < n; c += nwarp) {
        const unsigned long long k = s_cand[c];
        if (k == 0ull) continue;
        int rank = 0;
        for (int j0 = 0; j0 < n && rank < K; j0 += 32) {
            const int j = j0 + lane;
            rank += __popc(__ballot_sync(HS_FULL_MASK, j < n && s_cand[j] > k));
        }
        if (rank < K && lane == 0) s_top[rank] = k;
    }
}

// barrier over the first `nthr` threads of the CTA (a multiple of 32); id 0 is __syncthreads' own
__device__ __forceinline__ void bar_sync(int id, int nthr) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthr) : "memory");
}

// Cold path of the Top-K: K rounds of "largest key below the previous winner" over vectors [v0, v1) of a row,
// read from global memory by `nthr` threads (barrier `bar`).  Exact for any number of ties; -inf logits are no
// candidates.  s_red: one slot per warp.
template <bool BF16>
__device__ __noinline__ void topk_by_rounds(const char* rowp, int v0, int v1, int vocab, int K,
                                            unsigned long long* s_top, unsigned long long* s_red,
                                            int tid, int nthr, int bar) {
    constexpr int VE = BF16 ? 8 : 4;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    unsigned long long last = ~0ull;
    for (int r = 0; r < K; ++r) {
        unsigned long long best = 0ull;
        for (int v = v0 + tid; v < v1; v += nthr) {
            uint4 dv = __ldg((const uint4*)(rowp) + v);
            float x[8];
            unpack<BF16>(dv, x);
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                if (v * VE + e < vocab && x[e] > -CUDART_INF_F) {
                    unsigned long long k = make_key(x[e], v * VE + e);
                    if (k < last && k > best) best = k;
                }
            }
        }
        best = warp_max_u64(best);
        if (lane == 0) s_red[warp] = best;
        bar_sync(bar, nthr);
        best = s_red[0];
        for (int w = 1; w < nwarp; ++w) best = s_red[w] > best ? s_red[w] : best;
        if (tid == 0) s_top[r] = best;
        last = best;
        bar_sync(bar, nthr);
        if (best == 0ull) break;
    }
}

// One warp: the statistics of a whole row from its {max, sum e^(x-max), sum x e^(x-max)} and its K best keys
// (s_top, 0 = none): log-sum-exp, Shannon entropy, Top-K values and token ids, the entropy of the renormalised
// Top-K probabilities (Eq. 1 inner sum) and the truncated variant.
__device__ __forceinline__ void finalize_row(const QuantParams& p, int row, float M, float S, float U,
                                             const unsigned long long* s_top, int lane) {
    const int K = p.K;
    const float lse = M + logf(S);
    const float H = lse - U / S;
    const unsigned long long key = (lane < K) ? s_top[lane] : 0ull;
    const bool valid = key != 0ull;
    const float tv = valid ? key_value(key) : 0.f;
    const float t0 = __shfl_sync(HS_FULL_MASK, tv, 0);
    const float pv = valid ? expf(tv - lse) : 0.f;
    const float itr = warp_sum(valid ? -pv * (tv - lse) : 0.f);
    const float z = valid ? expf(tv - t0) : 0.f;
    const float Z = warp_sum(z);
    const float itk = logf(Z) - warp_sum(valid ? z * (tv - t0) : 0.f) / Z;
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
    }
}

// K-th largest of the warp's 32 values (one per lane), -inf if fewer than K are above -inf.  K rounds of a
// warp-wide maximum that retires one holder of the maximum per round (ties count one by one).
__device__ __forceinline__ float warp_kth_largest(float v, int K, int lane) {
    unsigned int ob = (v > -CUDART_INF_F) ? float_order_bits(v) : 0u;
    unsigned int mx = 0u;
    for (int i = 0; i < K; ++i) {
        mx = __reduce_max_sync(HS_FULL_MASK, ob);
        const unsigned int holders = __ballot_sync(HS_FULL_MASK, ob == mx);
        if (lane == __ffs(holders) - 1) ob = 0u;
    }
    return mx ? order_bits_float(mx) : -CUDART_INF_F;
}

// ================================================================================================================
// The streaming kernel
// ================================================================================================================
// Geometry of the shares.  split == 0 ("stream"): the rows form one stream of rows * nvec vectors, share c is
// [c * per, (c + 1) * per), a share may hold several rows and a row may lie in several shares.  split == S > 0 ("row
// split", for launches with at most one row per SM): the first `extra` rows are cut into S + 1 equal parts, the
// others into S, one share per part, so that every share is a single row segment.  split < 0 ("whole rows", for
// launches with many rows per SM): share c of `extra` shares holds the rows [c * rows / extra, (c + 1) * rows / extra).
struct Share {
    long long g0, g1;
};
__device__ __forceinline__ void shares_of_row(const QuantParams& p, int row, int& c_first, int& nseg) {
    if (p.split < 0) {
        c_first = 0; nseg = 1;
    } else if (p.split) {
        if (row < p.extra) { c_first = row * (p.split + 1); nseg = p.split + 1; }
        else { c_first = p.extra * (p.split + 1) + (row - p.extra) * p.split; nseg = p.split; }
    } else {
        const long long r0 = (long long)row * p.nvec;
        c_first = (int)(r0 / p.per);
        nseg = (int)((r0 + p.nvec - 1) / p.per) - c_first + 1;
    }
}
__device__ __forceinline__ Share share_of(const QuantParams& p, int c) {
    Share sh;
    if (p.split < 0) {
        sh.g0 = ((long long)c * p.rows / p.extra) * p.nvec;
        sh.g1 = ((long long)(c + 1) * p.rows / p.extra) * p.nvec;
    } else if (p.split) {
        const int wide = p.extra * (p.split + 1);           // shares of the rows with S + 1 parts
        const int parts = c < wide ? p.split + 1 : p.split;
        const int row = c < wide ? c / parts : p.extra + (c - wide) / parts;
        const int part = c < wide ? c - row * parts : (c - wide) - (row - p.extra) * parts;
        const int pv = (p.nvec + parts - 1) / parts;
        sh.g0 = (long long)row * p.nvec + min(part * pv, p.nvec);
        sh.g1 = (long long)row * p.nvec + min((part + 1) * pv, p.nvec);
    } else {
        sh.g0 = (long long)c * p.per;
        sh.g1 = min(sh.g0 + (long long)p.per, (long long)p.rows * p.nvec);
    }
    return sh;
}
// partial slot of share c for `row`: stream mode has two per share (the leading one for a row that began in an
// earlier share), row-split mode one
__device__ __forceinline__ int partial_slot(const QuantParams& p, int row, int c) {
    if (p.split) return c;
    return 2 * c + ((long long)row * p.nvec < (long long)c * p.per ? 0 : 1);
}

// 72 registers per thread (no spills): the 17 warps then leave room in the register file for a CTA of the kernel
// ahead that is still at work on the same SM (in a decode loop: the CTA that walks the accepted path of the step
// before), so this kernel's CTA is resident, and its share on chip, before that kernel has ended.
template <bool BF16>
__global__ void __maxnreg__(72) quantify_stream_kernel(const QuantParams p) {
    constexpr int VE = BF16 ? 8 : 4;
    constexpr int NW = QS_CONSUMERS / 32;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ unsigned long long s_full[QS_SLOTS], s_empty[QS_SLOTS];
    __shared__ unsigned long long s_list[CAND_CAP];
    __shared__ unsigned long long s_top[2][HS_MAX_TOPK];   // (two copies: a finished row is written out by warp 0
    __shared__ unsigned long long s_red[NW];               //  while the other warps read the next one)
    __shared__ __align__(16) float s_gm[32];
    __shared__ __align__(16) float s_lm[NW][32];
    __shared__ float s_wstat[2][NW][3];
    __shared__ int s_cnt;
    __shared__ int s_flag;
    __shared__ unsigned long long s_ck[8][HS_MAX_TOPK];   // clustered launch, first CTA of a row: the shares' Top-K keys
    __shared__ __align__(16) float4 s_cs[8];               //   and their {max, sum e, sum x e}

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned int slots0 = (smem_u32(s_dyn) + 127u) & ~127u;
    const unsigned char* slots_gen = s_dyn + (slots0 - smem_u32(s_dyn));
    const Share sh = share_of(p, blockIdx.x);
    const long long g0 = sh.g0, g1 = sh.g1;
    const size_t esz = BF16 ? 2 : 4;
    const int nslots = p.nslots;

    if (tid == 0) {
        for (int s = 0; s < nslots; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), NW);
        }
        mbar_init_fence();
        s_cnt = 0;
    }
    __syncthreads();
    pdl_launch_dependents();
    // Clustered launch: first half of a cluster barrier - when it completes every CTA of the row's cluster runs and
    // its shared memory may be written from outside.  Every thread of the CTA, the producer warp included, takes part
    // in the two barrier phases of the launch.
    if (p.clustered) cluster_arrive();

    if (warp == NW) {
        // ---- producer: one lane walks the share item by item ----------------------------------------------------
        if (lane == 0) {
            long long g = g0;
            int it = 0, slot = 0;
            unsigned int epar = 1u;          // parity of the slot's `empty` barrier before its first completion
            bool waited = false;
            if (!p.prefetch) { pdl_wait(); waited = true; }
            while (g < g1) {
                const int row = (int)(g / p.nvec);
                const int v = (int)(g - (long long)row * p.nvec);
                const int len = (int)min((long long)min(QS_ITEM_VECS, p.nvec - v), g1 - g);
                if (it >= nslots) {
                    if (!waited) { pdl_wait(); waited = true; }     // (nothing of this kernel is written by the producer)
                    mbar_wait(smem_u32(&s_empty[slot]), epar, p.err);
                }
                const unsigned int bar = smem_u32(&s_full[slot]);
                mbar_expect_tx(bar, (unsigned int)len * 16u);
                bulk_load(slots0 + (unsigned int)slot * (QS_ITEM_VECS * 16),
                          (const char*)p.logits + (size_t)row * p.row_stride * esz + (size_t)v * 16, (unsigned int)len * 16u, bar);
                g += len;
                ++it;
                if (++slot == nslots) { slot = 0; epar ^= 1u; }
            }
        }
        if (p.clustered) {
            __syncwarp();
            cluster_wait();
            cluster_arrive();
            cluster_wait();
        }
        return;
    }

    // ---- consumers -------------------------------------------------------------------------------------------------
    // Partials, counters and outputs may still be in use by the kernel ahead: nothing is written before the wait.
    // Reading the logits and reducing them in registers and shared memory needs no wait if the caller vouches that
    // they were complete before the call (prefetch): then the wait comes at the end of the first segment.
    bool waited = false;
    if (!p.prefetch) { pdl_wait(); waited = true; }
    const int K = p.K;
    const unsigned int ninf = BF16 ? 0xff80ff80u : 0xff800000u;
    int cslot = 0;                 // slot of the next item and the parity of its `full` barrier (the producer fills
    unsigned int cpar = 0u;        // the slots round-robin in the same order)
    int seg = 0;                   // segments of this share finished so far (parity selects the s_top / s_wstat copy)
    long long g = g0;

    // One item: waits for its slot, keeps the maxima of the thread's QS_VPT vectors in vm[], folds the item into the
    // thread's running (max, sum e^(x-max), sum x e^(x-max)).
    auto consume_item = [&](int slot, int v_item, int len, float* vm, float& m_t, float2& s2, float2& u2) {
        mbar_wait(smem_u32(&s_full[slot]), cpar, p.err);
        if (++cslot == nslots) { cslot = 0; cpar ^= 1u; }
        const uint4* st = reinterpret_cast<const uint4*>(slots_gen + (size_t)slot * (QS_ITEM_VECS * 16));
        uint4 d[QS_VPT];
        float imax = -CUDART_INF_F;
        if (len == QS_ITEM_VECS) {                                           // (the usual case: no lane is idle)
#pragma unroll
            for (int j = 0; j < QS_VPT; ++j) d[j] = st[tid + j * QS_CONSUMERS];
        } else {
#pragma unroll
            for (int j = 0; j < QS_VPT; ++j) {
                const int vl = tid + j * QS_CONSUMERS;
                d[j] = (vl < len) ? st[vl] : make_uint4(ninf, ninf, ninf, ninf);
            }
        }
        if (v_item + len == p.nvec && p.nvec * VE != p.vocab) {               // the row's last vector runs past vocab
#pragma unroll
            for (int j = 0; j < QS_VPT; ++j) {
                if (v_item + tid + j * QS_CONSUMERS == p.nvec - 1) {
                    unsigned int* wd = reinterpret_cast<unsigned int*>(&d[j]);
#pragma unroll
                    for (int e = 0; e < VE; ++e)
                        if ((p.nvec - 1) * VE + e >= p.vocab) {
                            if (BF16) wd[e >> 1] = (e & 1) ? ((wd[e >> 1] & 0x0000ffffu) | 0xff800000u)
                                                           : ((wd[e >> 1] & 0xffff0000u) | 0x0000ff80u);
                            else wd[e] = 0xff800000u;
                        }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < QS_VPT; ++j) {
            if (BF16) {
                const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&d[j].x),
                                                *reinterpret_cast<const __nv_bfloat162*>(&d[j].y));
                const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&d[j].z),
                                                *reinterpret_cast<const __nv_bfloat162*>(&d[j].w));
                const __nv_bfloat162 c = __hmax2(a, b);
                const unsigned int cw = *reinterpret_cast<const unsigned int*>(&c);
                vm[j] = fmaxf(bf16_lo(cw), bf16_hi(cw));
            } else {
                vm[j] = fmaxf(fmaxf(__uint_as_float(d[j].x), __uint_as_float(d[j].y)),
                              fmaxf(__uint_as_float(d[j].z), __uint_as_float(d[j].w)));
            }
            imax = fmaxf(imax, vm[j]);
        }
        if (imax > m_t) {                         // the thread's maximum grows: rescale its sums
            const float f = (m_t == -CUDART_INF_F) ? 0.f : ex2f((m_t - imax) * LOG2E);
            s2.x *= f; s2.y *= f; u2.x *= f; u2.y *= f;
            m_t = imax;
        }
        const float nml = (m_t == -CUDART_INF_F) ? 0.f : -m_t * LOG2E;
        const float2 l2 = make_float2(LOG2E, LOG2E), n2 = make_float2(nml, nml);
        const unsigned int floor2 = 0xf149f149u;  // bf16 pair of -1e30: keeps 0 * x finite for x = -inf
#pragma unroll
        for (int j = 0; j < QS_VPT; ++j) {
            const unsigned int* wd = reinterpret_cast<const unsigned int*>(&d[j]);
            if (BF16) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const __nv_bfloat162 cl = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&wd[q]),
                                                     *reinterpret_cast<const __nv_bfloat162*>(&floor2));
                    const unsigned int cw = *reinterpret_cast<const unsigned int*>(&cl);
                    const float2 x = make_float2(bf16_lo(cw), bf16_hi(cw));
                    const float2 t = fma2_ftz(x, l2, n2);
                    const float2 e = make_float2(ex2f(t.x), ex2f(t.y));
                    s2 = add2_ftz(s2, e);
                    u2 = fma2_ftz(e, x, u2);
                }
            } else {
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const float2 x = make_float2(fmaxf(__uint_as_float(wd[2 * q]), -1e30f),
                                                 fmaxf(__uint_as_float(wd[2 * q + 1]), -1e30f));
                    const float2 t = fma2_ftz(x, l2, n2);
                    const float2 e = make_float2(ex2f(t.x), ex2f(t.y));
                    s2 = add2_ftz(s2, e);
                    u2 = fma2_ftz(e, x, u2);
                }
            }
        }
    };
    // A lower bound of the segment's K-th largest logit.  Maxima of disjoint element sets are distinct elements, so
    // the K-th largest of any such family is a bound.  With at least one full item behind the segment: the CTA's 32
    // half-warp maxima (published in shared memory; an entry another warp has not refreshed yet is an older maximum
    // of the same segment, still an element of it).  Shorter: this warp's own 32 lane maxima.
    auto kth_bound = [&](float m_t, bool full_item, bool barrier) -> float {
        const float4* fam;                                   // the family of 32 maxima, read back as eight float4
        if (full_item) {
            float hm = m_t;
            hm = fmaxf(hm, __shfl_xor_sync(HS_FULL_MASK, hm, 1));
            hm = fmaxf(hm, __shfl_xor_sync(HS_FULL_MASK, hm, 2));
            hm = fmaxf(hm, __shfl_xor_sync(HS_FULL_MASK, hm, 4));
            hm = fmaxf(hm, __shfl_xor_sync(HS_FULL_MASK, hm, 8));
            if ((lane & 15) == 0) s_gm[warp * 2 + (lane >> 4)] = hm;
            if (barrier) bar_sync(1, QS_CONSUMERS);          // every warp has published maxima of this segment
            else __syncwarp();
            fam = reinterpret_cast<const float4*>(s_gm);
        } else {
            s_lm[warp][lane] = m_t;
            if (barrier) bar_sync(1, QS_CONSUMERS);          // (the same barrier count for every warp)
            else __syncwarp();
            fam = reinterpret_cast<const float4*>(s_lm[warp]);
        }
        const float w = reinterpret_cast<const float*>(fam)[lane];
        int ge = 0;                                          // members >= this lane's
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float4 f4 = fam[j];
            ge += (f4.x >= w) + (f4.y >= w) + (f4.z >= w) + (f4.w >= w);
        }
        return warp_max(ge >= K ? w : -CUDART_INF_F);
    };
    // Candidates of one item: the warp works through the vectors whose maximum reaches the bound, four at a time
    // (eight lanes per vector, one element each, read back from the item's slot in shared memory).
    auto scan_item = [&](int slot, int v_item, const float* vm, float tau) {
        unsigned int hits = 0u;
#pragma unroll
        for (int j = 0; j < QS_VPT; ++j) hits |= (vm[j] >= tau && vm[j] > -CUDART_INF_F) ? (1u << j) : 0u;
        unsigned int any = __ballot_sync(HS_FULL_MASK, hits != 0u);
        while (any) {
            const int src = __ffs(any) - 1;
            unsigned int m = __shfl_sync(HS_FULL_MASK, hits, src);
            any &= any - 1;                                   // (a lane has at most QS_VPT = 4 hit vectors: one round)
            for (int q = (lane >> 3); q > 0; --q) m &= m - 1; // lanes 8q .. 8q+7 take the q-th hit vector
            const int e = lane & 7;
            if (m && e < VE) {
                const int j = __ffs(m) - 1;
                const int vl = (warp * 32 + src) + j * QS_CONSUMERS;
                const unsigned char* vp = slots_gen + (size_t)slot * (QS_ITEM_VECS * 16) + (size_t)vl * 16;
                const float x = BF16 ? __uint_as_float((unsigned int)reinterpret_cast<const unsigned short*>(vp)[e] << 16)
                                     : reinterpret_cast<const float*>(vp)[e];
                const int idx = (v_item + vl) * VE + e;
                if (x >= tau && x > -CUDART_INF_F && idx < p.vocab) {
                    const int sl = atomicAdd(&s_cnt, 1);
                    if (sl < CAND_CAP) s_list[sl] = make_key(x, idx);
                }
            }
        }
    };

    while (g < g1) {
        // ---- one segment: the part [g, seg_end) of this share inside row `row` ------------------------------------
        const int row = (int)(g / p.nvec);
        const long long row_g0 = (long long)row * p.nvec;
        const int sv0 = (int)(g - row_g0);
        const int sv1 = (int)(min(g1, row_g0 + p.nvec) - row_g0);
        const char* rowp = (const char*)p.logits + (size_t)row * p.row_stride * esz;
        unsigned long long* top = s_top[seg & 1];
        float m_t = -CUDART_INF_F;                // running maximum of this thread's logits of the segment
        float2 s2 = make_float2(0.f, 0.f), u2 = make_float2(0.f, 0.f);
        float tau;                                // lower bound of the K-th largest logit of the segment
        int v = sv0;
        int items_done = 0;
        {
            // ---- first window: up to QS_WINDOW items are held, the bound is taken from all of them -----------------
            float vmx[QS_WINDOW][QS_VPT];
            int w_slot[QS_WINDOW], w_v0[QS_WINDOW];
#pragma unroll
            for (int wi = 0; wi < QS_WINDOW; ++wi) {
                w_slot[wi] = -1; w_v0[wi] = 0;
                if (v < sv1) {
                    const int len = min(QS_ITEM_VECS, sv1 - v);
                    w_slot[wi] = cslot; w_v0[wi] = v;
                    consume_item(w_slot[wi], v, len, vmx[wi], m_t, s2, u2);
                    v += len; ++items_done;
                }
            }
            tau = kth_bound(m_t, v - sv0 >= QS_ITEM_VECS, true);
#pragma unroll
            for (int wi = 0; wi < QS_WINDOW; ++wi)
                if (w_slot[wi] >= 0) scan_item(w_slot[wi], w_v0[wi], vmx[wi], tau);
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int wi = 0; wi < QS_WINDOW; ++wi)
                    if (w_slot[wi] >= 0) mbar_arrive(smem_u32(&s_empty[w_slot[wi]]));
            }
        }
        // ---- the rest of the segment item by item: scanned against the bound and handed back at once; the bound is
        // refreshed whenever the number of items read reaches a power of two -----------------------------------------
        while (v < sv1) {
            float vm[QS_VPT];
            const int len = min(QS_ITEM_VECS, sv1 - v);
            const int slot = cslot;
            consume_item(slot, v, len, vm, m_t, s2, u2);
            ++items_done;
            if ((items_done & (items_done - 1)) == 0) tau = fmaxf(tau, kth_bound(m_t, true, false));
            scan_item(slot, v, vm, tau);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
            v += len;
        }
        // ---- end of the segment: warp, then CTA reduction of (max, s, u); Top-K of the candidates ------------------
        {
            const float wm = warp_max(m_t);
            const float f = (m_t == -CUDART_INF_F) ? 0.f : ex2f((m_t - wm) * LOG2E);
            const float ws = warp_sum((s2.x + s2.y) * f), wu = warp_sum((u2.x + u2.y) * f);
            if (lane == 0) { s_wstat[seg & 1][warp][0] = wm; s_wstat[seg & 1][warp][1] = ws; s_wstat[seg & 1][warp][2] = wu; }
        }
        if (tid < HS_MAX_TOPK) top[tid] = 0ull;       // (this copy was last read two segments ago)
        bar_sync(1, QS_CONSUMERS);                    // all candidates are pushed, all warp sums written
        const int ncand = s_cnt;
        if (ncand <= CAND_CAP) rank_select_warps(s_list, ncand, K, top, warp, lane, NW);
        else topk_by_rounds<BF16>(rowp, sv0, sv1, p.vocab, K, top, s_red, tid, QS_CONSUMERS, 1);   // heavy ties
        bar_sync(1, QS_CONSUMERS);                    // the Top-K is complete; s_list and s_cnt are free again
        if (!waited) { pdl_wait(); waited = true; }   // from here on the segment's results go to global memory
        if (p.clustered) cluster_wait();              // (the arrival at the start: every CTA of the cluster runs)
        int c_first, nseg;
        shares_of_row(p, row, c_first, nseg);
        if (warp == 0) {
            if (lane == 0) s_cnt = 0;                 // (the next push comes after the next segment's first barrier)
            // the consumer warps' (max, s, u) in a fixed order
            const float wm = lane < NW ? s_wstat[seg & 1][lane][0] : -CUDART_INF_F;
            const float M = warp_max(wm);
            const float f = (lane >= NW || wm == -CUDART_INF_F) ? 0.f : ex2f((wm - M) * LOG2E);
            const float S = lane < NW ? s_wstat[seg & 1][lane][1] * f : 0.f, U = lane < NW ? s_wstat[seg & 1][lane][2] * f : 0.f;
            float St = 0.f, Ut = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                St += __shfl_sync(HS_FULL_MASK, S, w);
                Ut += __shfl_sync(HS_FULL_MASK, U, w);
            }
            if (nseg == 1) {
                // the whole row lay in this share: the other warps are already on their way to the next segment
                finalize_row(p, row, M, St, Ut, top, lane);
            } else if (p.clustered) {
                // this share's partial goes into slot `part` of the first CTA of the row's cluster (posted stores
                // through distributed shared memory; the cluster barrier below makes them visible there)
                const int part = blockIdx.x - c_first;
                if (lane < HS_MAX_TOPK) {
                    const unsigned int dst = cluster_map_addr(smem_u32(&s_ck[part][lane]), 0);
                    asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(dst), "l"((lane < K) ? top[lane] : 0ull) : "memory");
                }
                if (lane == 0) {
                    const unsigned int dst = cluster_map_addr(smem_u32(&s_cs[part]), 0);
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(__float_as_uint(M)),
                                 "r"(__float_as_uint(St)), "r"(__float_as_uint(Ut)), "r"(0u) : "memory");
                    s_flag = (part == 0);
                }
            } else {
                const int ps = partial_slot(p, row, blockIdx.x);
                if (lane == 0) p.part_stats[ps] = make_float4(M, St, Ut, 0.f);
                if (lane < HS_MAX_TOPK) p.part_keys[(size_t)ps * HS_MAX_TOPK + lane] = (lane < K) ? top[lane] : 0ull;
                __syncwarp();
                if (lane == 0) {
                    // one release-acquire arrival at device scope: the partial written by this warp (ordered before the
                    // arrival by the warp barrier above) is visible to whoever arrives last, and the last one sees all
                    int old;
                    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(&p.row_cnt[row]) : "memory");
                    const int last = old == nseg - 1;
                    if (last) p.row_cnt[row] = 0;              // ready for the next launch
                    s_flag = last;
                }
            }
        }
        if (nseg > 1) {
            if (p.clustered) {
                cluster_arrive();                     // (second phase: the stores above are released, and acquired below)
                cluster_wait();
            } else {
                bar_sync(1, QS_CONSUMERS);            // s_flag
            }
            if (s_flag) {
                // ---- the last share of a split row (clustered: the first CTA of its cluster) merges the partials ----
                if (tid < HS_MAX_TOPK) top[tid] = 0ull;
                float4 stv = make_float4(-CUDART_INF_F, 0.f, 0.f, 0.f);       // (warp 0: requested with the keys)
                if (warp == 0 && lane < nseg)
                    stv = p.clustered ? s_cs[lane] : __ldcg(&p.part_stats[partial_slot(p, row, c_first + lane)]);
                for (int t = tid; t < nseg * HS_MAX_TOPK; t += QS_CONSUMERS) {
                    if (p.clustered) {
                        s_list[t] = s_ck[t / HS_MAX_TOPK][t % HS_MAX_TOPK];
                        continue;
                    }
                    const int ps = partial_slot(p, row, c_first + t / HS_MAX_TOPK);
                    s_list[t] = __ldcg(&p.part_keys[(size_t)ps * HS_MAX_TOPK + (t % HS_MAX_TOPK)]);
                }
                bar_sync(1, QS_CONSUMERS);
                rank_select_warps(s_list, nseg * HS_MAX_TOPK, K, top, warp, lane, NW);
                bar_sync(1, QS_CONSUMERS);
                if (warp == 0) {
                    const float m = stv.x, cs = stv.y, cu = stv.z;
                    const float M = warp_max(m);
                    const float f = (m == -CUDART_INF_F) ? 0.f : ex2f((m - M) * LOG2E);
                    const float S = warp_sum(cs * f), U = warp_sum(cu * f);
                    finalize_row(p, row, M, S, U, top, lane);
                }
            }
        }
        ++seg;
        g = row_g0 + sv1;
    }
    if (p.clustered && seg == 0) {                    // (a CTA without a segment still owes the cluster its two phases)
        cluster_wait();
        cluster_arrive();
        cluster_wait();
    }
}

// ================================================================================================================
// Tree stage: one CTA of 128 threads per sequence, one thread per node
// ================================================================================================================
__global__ void __launch_bounds__(HS_MAX_NODES) tree_scores_kernel(const QuantParams p) {
    __shared__ TreeStageSmem sm;
    pdl_launch_dependents();
    tree_stage_cta(p, blockIdx.x, sm);
}

static void fill_common(QuantParams& p, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                        int64_t row_stride, int32_t vocab, const hs_policy* policy, const hs_quant_out* out) {
    const int ve = hs_vec_elems(dtype);
    p.logits = logits;
    p.row_stride = row_stride;
    p.vocab = vocab;
    p.nvec = (vocab + ve - 1) / ve;
    p.chunks = 0;
    p.chunk_vecs = 0;
    p.per = 0;
    p.split = 0;
    p.extra = 0;
    p.nslots = QS_SLOTS;
    p.clustered = 0;
    p.rows = tree->n_nodes_total;
    p.batch = tree->batch;
    p.node_off = tree->node_off;
    p.parent = tree->parent;
    p.token = tree->token;
    p.out = *out;
    p.K = policy->top_k;
    p.d_base = policy->d_base;
    p.phi_mode = policy->phi_mode;
    p.pstar_mode = policy->pstar_mode;
    p.entropy_mode = policy->entropy_mode;
    p.is_bf16 = dtype == HS_BF16;
    p.prefetch = 0;
    p.err = nullptr;
}

// Geometry of a launch, one CTA per SM.  With at most one row per SM and rows short enough for the item slots,
// every SM gets one part of one row (the first rows are cut into one part more than the others so that every SM
// has work): a CTA then has a single row segment.  With two or more rows per SM every CTA takes whole rows (no row
// needs a merge).  In between every CTA takes an equal share of the stream, at least one item long and so large
// that no row is split over more than QS_MAX_SEGS shares.
static void quantify_geometry(int rows, int nvec, int sm_count, QuantParams& p, int& nctas, size_t& smem) {
    int S = rows <= sm_count ? sm_count / rows : 0;
    while (S > 1 && (S + 1 > QS_MAX_SEGS || nvec / (S + 1) < 256)) --S;      // parts of at least 4 KiB
    const int extra = (S >= 1 && S + 1 <= QS_MAX_SEGS && nvec / (S + 1) >= 256) ? min(rows, sm_count - rows * S) : 0;
    const int pv_max = S >= 1 ? (nvec + S - 1) / S : 0;
    // With at most half as many rows as SMs every row is cut into the same number of parts (at most eight, the portable
    // cluster size): the CTAs of a row are one thread-block cluster and merge the row in the shared memory of its first
    // CTA.  (The critical path is the same as with one part more for some rows - the rows with fewer parts - but the
    // merge costs a cluster barrier instead of partials, an atomic and their read-back through global memory.)
    int Sc = rows <= sm_count / 2 ? (sm_count / rows < 8 ? sm_count / rows : 8) : 0;
    while (Sc > 1 && nvec / Sc < 256) --Sc;
    const int pv_c = Sc >= 2 ? (nvec + Sc - 1) / Sc : 0;
    p.clustered = 0;
    if (rows >= 2 * sm_count) {
        p.split = -1;
        p.extra = sm_count;
        p.per = 0;
        p.nslots = QS_SLOTS;
        nctas = sm_count;
    } else if (Sc >= 2 && pv_c <= QS_SLOTS * QS_ITEM_VECS) {
        p.split = Sc;
        p.extra = 0;
        p.per = pv_c;
        p.nslots = (pv_c + QS_ITEM_VECS - 1) / QS_ITEM_VECS;
        p.clustered = 1;
        nctas = rows * Sc;
    } else if (S >= 1 && pv_max <= QS_SLOTS * QS_ITEM_VECS) {
        p.split = S;
        p.extra = extra;
        p.per = pv_max;
        p.nslots = (pv_max + QS_ITEM_VECS - 1) / QS_ITEM_VECS;
        nctas = rows * S + extra;
    } else {
        const long long total = (long long)rows * nvec;
        long long per = (total + sm_count - 1) / sm_count;
        const long long floor_row = (nvec + (QS_MAX_SEGS - 2) - 1) / (QS_MAX_SEGS - 2);
        if (per < floor_row) per = floor_row;
        if (per < QS_ITEM_VECS) per = QS_ITEM_VECS;
        p.split = 0;
        p.extra = 0;
        p.per = (int)per;
        p.nslots = QS_SLOTS;
        nctas = (int)((total + per - 1) / per);
    }
    smem = (size_t)p.nslots * QS_ITEM_VECS * 16 + 128;
}

hs_status hs_launch_quantify(hs_ctx* ctx, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                             int64_t row_stride, int32_t vocab, const hs_policy* policy,
                             const hs_quant_out* out, cudaStream_t stream, bool with_tree_stage) {
    QuantParams p;
    fill_common(p, tree, logits, dtype, row_stride, vocab, policy, out);
    if (p.nvec > QS_ITEM_VECS * 64) return HS_ERR_SHAPE;            // vocabulary beyond 2^20 bf16 / 2^19 fp32 logits
    int nctas = 0;
    size_t smem = 0;
    quantify_geometry(p.rows, p.nvec, ctx->sm_count, p, nctas, smem);
    const int nparts = p.split ? nctas : 2 * nctas;      // (whole rows: none is used)
    const size_t stats_bytes = hs_align_up((size_t)nparts * sizeof(float4), 256);
    const size_t keys_bytes = (size_t)nparts * HS_MAX_TOPK * sizeof(unsigned long long);
    if (stats_bytes + keys_bytes > ctx->scratch_bytes) return HS_ERR_WORKSPACE;
    p.part_stats = (float4*)ctx->scratch;
    p.part_keys = (unsigned long long*)(ctx->scratch + stats_bytes);
    p.row_cnt = ctx->counters + HS_CNT_QUANT_ROW;
    p.err = ctx->counters + HS_CNT_ERROR;
    p.prefetch = (ctx->prefetch & HS_PREFETCH_LOGITS) != 0;
    if (!ctx->quant_ready) {
        if (cudaFuncSetAttribute(quantify_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, QS_SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(quantify_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, QS_SMEM_BYTES) != cudaSuccess)
            return HS_ERR_CUDA;
        ctx->quant_ready = true;
    }
    cudaError_t e = dtype == HS_BF16
        ? hs_launch(quantify_stream_kernel<true>, dim3(nctas), dim3(QS_THREADS), smem, stream, ctx->pdl,
                    dim3(p.clustered ? p.split : 1, 1, 1), p)
        : hs_launch(quantify_stream_kernel<false>, dim3(nctas), dim3(QS_THREADS), smem, stream, ctx->pdl,
                    dim3(p.clustered ? p.split : 1, 1, 1), p);
    if (e != cudaSuccess) return HS_ERR_CUDA;
    if (!with_tree_stage) return HS_OK;              // (the caller launches the kernel that also prunes)
    e = hs_launch(tree_scores_kernel, dim3(p.batch), dim3(HS_MAX_NODES), 0, stream, ctx->pdl, dim3(1, 1, 1), p);
    return e == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

// ================================================================================================================
// The chunk kernel: a CTA owns one chunk of one row (at most 256 * 8 vectors), everything in registers: 16-byte
// coalesced loads that are all issued before the first use, max / sum e^x / sum x e^x by warp shuffles, the chunk's
// Top-K from the K-th largest of 32 group maxima as the bound; the last chunk of a row to arrive merges the row.
// ================================================================================================================
template <bool BF16>
__global__ void __launch_bounds__(HS_ROW_THREADS, 2) quantify_chunk_kernel(const QuantParams p) {
    constexpr int VE = BF16 ? 8 : 4;
    constexpr int VPT = HS_ROW_VPT;
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

    const unsigned int ninf = BF16 ? 0xff80ff80u : 0xff800000u;
    uint4 d[VPT];
    pdl_launch_dependents();
    pdl_wait();
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        int v = v0 + tid + j * HS_ROW_THREADS;
        d[j] = (v < v1) ? __ldcs((const uint4*)(rowp) + v) : make_uint4(ninf, ninf, ninf, ninf);
    }
    // ---- maxima ---------------------------------------------------------------------------
    float vmax[VPT];
    float tmax = -CUDART_INF_F;
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        float x[8];
        unpack<BF16>(d[j], x);
        int v = v0 + tid + j * HS_ROW_THREADS;
        if (v == p.nvec - 1) {                       // the row's last vector may run past vocab
#pragma unroll
            for (int e = 0; e < VE; ++e)
                if (v * VE + e >= p.vocab) x[e] = -CUDART_INF_F;
        }
        float m = x[0];
#pragma unroll
        for (int e = 1; e < VE; ++e) m = fmaxf(m, x[e]);
        vmax[j] = m;
        tmax = fmaxf(tmax, m);
    }
    // ---- sums relative to the thread's own maximum ------------------------------------------
    const float nml = (tmax == -CUDART_INF_F) ? 0.f : -tmax * LOG2E;
    float s = 0.f, u = 0.f;
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        float x[8];
        unpack<BF16>(d[j], x);
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
    const float tau = warp_kth_largest(s_gm[lane], K, lane);   // K-th largest group maximum
    if (tmax >= tau && tmax > -CUDART_INF_F) {
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            if (vmax[j] >= tau) {
                float x[8];
                unpack<BF16>(d[j], x);
                int base = (v0 + tid + j * HS_ROW_THREADS) * VE;
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    if (x[e] >= tau && x[e] > -CUDART_INF_F && base + e < p.vocab) {
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
        rank_select(s_cand, ncand, K, s_top, tid, HS_ROW_THREADS);
    } else {
        // Heavy ties (e.g. a constant row): K rounds of "largest key below the previous one",
        // re-reading the chunk from global memory (cold path).
        topk_by_rounds<BF16>(rowp, v0, v1, p.vocab, K, s_top, s_red, tid, HS_ROW_THREADS, 0);
    }
    __syncthreads();
    if (tid < HS_MAX_TOPK)
        p.part_keys[((size_t)row * p.chunks + chunk) * HS_MAX_TOPK + tid] = (tid < K) ? s_top[tid] : 0ull;

    // ---- the last chunk of this row merges -----------------------------------------------
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
    rank_select(s_cand, nk, K, s_top, tid, HS_ROW_THREADS);
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
        finalize_row(p, row, M, S, U, s_top, lane);
        if (lane == 0) p.row_cnt[row] = 0;                 // ready for the next launch
    }
}

// ---- hs_entropy_quantify_static: the same pass without any allocated workspace -------------------------------
//
// Some hosts of this library may not allocate device memory at all: a serving process that hands
// its whole memory budget to one arena at start-up, or code running under a capture / real-time
// rule that forbids cudaMalloc.  For them the chunk partials and arrival counters of the pass live
// in one fixed array that is part of the library image, so every GPU that loads the library carries
// HS_STATIC_SCRATCH_BYTES of it until the process exits.
#define HS_STATIC_MAX_CHUNKS 16
#define HS_STATIC_COUNTER_BYTES 2048    // HS_STATIC_MAX_ROWS ints (one arrival counter per row), rounded up
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
    fill_common(p, tree, draft_logits, dtype, row_stride, vocab, policy, out);
    p.chunks = chunks;
    p.chunk_vecs = (p.nvec + p.chunks - 1) / p.chunks;
    p.row_cnt = (int*)base;
    p.part_stats = (float4*)(base + HS_STATIC_COUNTER_BYTES);
    p.part_keys = (unsigned long long*)(base + HS_STATIC_COUNTER_BYTES + HS_STATIC_STATS_BYTES);
    // The array keeps whatever the previous call left: the arrival counters must start at zero.
    HS_CUDA_OK(cudaMemsetAsync(base, 0, HS_STATIC_COUNTER_BYTES, stream));
    dim3 grid(p.chunks, p.rows);
    if (dtype == HS_BF16) quantify_chunk_kernel<true><<<grid, HS_ROW_THREADS, 0, stream>>>(p);
    else quantify_chunk_kernel<false><<<grid, HS_ROW_THREADS, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return HS_ERR_CUDA;
    tree_scores_kernel<<<p.batch, HS_MAX_NODES, 0, stream>>>(p);      // (needs no scratch)
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
