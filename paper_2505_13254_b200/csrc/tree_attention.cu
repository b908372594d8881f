// hs_tree_verify_attention (Sec. 2.2, tree-mask attention): one launch.
//
// CTA = (block of 128 query rows, KV split, sequence x kv-head).  The GQA group times the kept tree
// nodes forms the dense M dimension: query row r = node * G + g.  The KV prefix is cut into tiles of
// 64 keys that are shared out evenly over the splits; a CTA requests its first tiles by TMA
// (cp.async.bulk.tensor into 128-byte-swizzled shared memory, four stages, K and V on mbarriers of
// their own) before it waits for the kernel ahead of it in the stream, because the cache does not
// depend on the pruned tree.  The <= 128 tree keys are gathered with plain loads (their rows may be
// indirect) and belong to the last split.  S = Q K^T and O += P V run on the 5th-generation tensor
// cores (tcgen05.mma, accumulators in tensor memory) with fp32 accumulation; the softmax is the
// online (running max / running sum) form in base 2.  Prefix columns are fully visible, tree column j
// is visible to row r iff bit j of the ancestor mask of r's node is set.  The splits of one (query
// block, head) form a thread-block cluster: every CTA stages its partial (max, sum, O) in its own
// shared memory and pushes each owner's rows there by bulk copies through distributed shared memory;
// an owner merges its rows once all pieces have landed.  No partial ever goes to global memory and
// there is no second launch.
#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

#define ATT_BM 128
#define ATT_BN 64
#define ATT_MAX_SPLIT 8
#define ATT_TILE_BYTES (ATT_BN * HS_HEAD_DIM * 2)   // 16 KiB: one K or V tile
#define ATT_STAGE_BYTES (2 * ATT_TILE_BYTES)
#define ATT_Q_BYTES (ATT_BM * HS_HEAD_DIM * 2)      // 32 KiB
#define ATT_PB_STRIDE (HS_HEAD_DIM * 2 + 16)        // bytes per row of a pushed partial: 128 bf16 of O / l, {max, sum}, padding
#define LOG2E 1.4426950408889634f
#define LN2 0.6931471805599453f

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_tree;
    const __nv_bfloat16* v_tree;
    __nv_bfloat16* out;
    float* lse_out;
    const int* n_keep;
    const int* keep_off;
    const int* keep_idx;
    const unsigned long long* anc_mask;
    const int* status;
    const int* node_off;
    const int* kv_off;
    int batch, hq, hkv, G, layout, nsplit, head_first, prefetch;
    float scale_log2;
    int* err;
};

__device__ __forceinline__ unsigned int pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned int*>(&v);
}
// byte offset of (key row, 16-byte chunk 0..15 of the 128 d's) inside a swizzled 64x128 bf16 tile:
// two halves of 64 d's, rows of 128 bytes, chunk index XOR-ed with the row (the TMA 128-byte swizzle)
__device__ __forceinline__ unsigned int tile_off(int key, int chunk) {
    return (unsigned int)((chunk >> 3) * (ATT_TILE_BYTES / 2) + key * 128 + (((chunk & 7) ^ (key & 7)) << 4));
}
// same layout for the 128-row query tile
__device__ __forceinline__ unsigned int q_off(int row, int chunk) {
    return (unsigned int)((chunk >> 3) * (ATT_Q_BYTES / 2) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// prefix tiles of split `split`: the ceil(L / 64) tiles are shared out evenly, independent of the tree
__device__ __forceinline__ void prefix_range(int L, int nsplit, int split, int& t_prefix, int& t0, int& t1) {
    t_prefix = (L + ATT_BN - 1) / ATT_BN;
    const int per = (t_prefix + nsplit - 1) / nsplit;
    t0 = min(split * per, t_prefix);
    t1 = min(t0 + per, t_prefix);
}

// =====================================================================================================
// The kernel: S = Q K^T and O += P V by the 5th-generation tensor cores, accumulators in tensor
// memory.  Two softmax warpgroups run two independent online-softmax streams over the block's 128 query
// rows: warpgroup g takes the KV tiles i = g, g + 2, ... and keeps its own S buffer, P buffer, running
// (max, sum) and O accumulator; thread t of a warpgroup owns query row t (= tensor-memory lane t), so the
// softmax needs no shuffles and the two streams never wait for one another: while one exponentiates (the
// special-function unit), the other loads, masks and stores.  Three more warps give one elected thread each: the S issuer
// (S = Q K^T of tile i + 2 as soon as S of tile i is in registers; 8 instructions of K = 16, operands
// straight from the swizzled TMA tiles: Q and K are K-major), the P V issuer (O_g += P V as soon as a P
// is written; V is the MN-major operand, the same swizzled tile as it arrived by TMA) and the TMA
// producer (a stage's K is refilled as soon as the S that read it is complete, its V once its P V is).
// A stream rescales its O in tensor memory only when a row's running maximum grows.  After the last
// tile the two streams are combined like two splits, in registers.
// =====================================================================================================
#define UM_THREADS 352                               // two softmax warpgroups + P V issuer, TMA producer, S issuer warps
#define UM_ROWS_THREADS 128
#define UM_SM_THREADS 256                            // softmax threads: row = tid & 127, stream = tid >> 7
#define UM_MAP_BYTES 1024                            // output-row map of the rows a CTA merges (<= 65 rows x 8 bytes)
#define UM_TMEM_COLS 512                             // S of stream g: columns 64 g ..; O: 128 + 128 g ..; P (bf16 pairs): 384 + 32 g ..
#define UM_STAGES 4
#define UM_RECV_BYTES (40 * 1024)                    // after the tile loop: partials pushed by the splits of the cluster
#define UM_SMEM_BYTES (UM_STAGES * ATT_STAGE_BYTES + ATT_Q_BYTES + UM_MAP_BYTES + 4096 + 1024)

__global__ void __launch_bounds__(UM_THREADS, 1)
tree_attn_umma_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ unsigned char smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5;
    // Sequences are taken longest prefix first (a ragged batch then ends on its short sequences, not on a long one
    // that started late): grid slot z / hkv holds the sequence of that rank by (length descending, index ascending).
    // kv_off is an input of the call, so the ranking runs ahead of the dependency wait.
    __shared__ int s_seq;
    int b = blockIdx.z / p.hkv;
    const int h = blockIdx.z % p.hkv;
    if (p.batch > 1 && p.batch <= UM_THREADS) {
        if (tid < p.batch) {
            const int len = p.kv_off[tid + 1] - p.kv_off[tid];
            int rank = 0;
            for (int j = 0; j < p.batch; ++j) {
                const int lj = p.kv_off[j + 1] - p.kv_off[j];
                rank += (lj > len || (lj == len && j < tid));
            }
            if (rank == b) s_seq = tid;
        }
        __syncthreads();
        b = s_seq;
    }
    const int split = blockIdx.y;
    const int m0 = blockIdx.x * ATT_BM;

    const unsigned int smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const unsigned int sQ = smem_base + UM_STAGES * ATT_STAGE_BYTES;
    const unsigned int sM = sQ + ATT_Q_BYTES;                // row map, then barriers and exchange arrays
    // barriers: K-full[UM_STAGES], V-full[UM_STAGES], K-free[UM_STAGES], V-free[UM_STAGES], S-ready[2],
    // partials-received, all-MMAs-done, P-written[2], S-read[2]; then the tensor-memory base.  A parity wait can only tell the
    // current phase from the one before, so every barrier is laid out such that its next completion depends on the
    // thread that waits: a stage's barriers complete once per UM_STAGES tiles, S-ready and P-written alternate with
    // the tile's parity.
    const unsigned int bar0 = sM + UM_MAP_BYTES, bar_v = bar0 + UM_STAGES * 8, bar_ek = bar_v + UM_STAGES * 8,
                       bar_ev = bar_ek + UM_STAGES * 8;
    const unsigned int bar_s = bar_ev + UM_STAGES * 8, bar_r = bar_s + 16, bar_done = bar_r + 8,
                       bar_p = bar_done + 8, bar_sr = bar_p + 16, tslot = bar_sr + 16;
    unsigned char* gQ = smem_gen + UM_STAGES * ATT_STAGE_BYTES;
    unsigned char* gM = gQ + ATT_Q_BYTES;
    volatile unsigned int* tslot_gen = reinterpret_cast<volatile unsigned int*>(gM + UM_MAP_BYTES + (4 * UM_STAGES + 8) * 8);
    float* s_mx = reinterpret_cast<float*>(gM + UM_MAP_BYTES + 1024);      // [2][128]: the streams' row maxima at the end
    float* s_lx = s_mx + 2 * ATT_BM;                                     // [2][128]: the streams' row sums

    // ---- before the dependency wait: barriers, tensor memory, the first KV prefix tiles -----------------
    const int kv0 = p.kv_off[b];
    const int L = p.kv_off[b + 1] - kv0;
    int t_prefix, t0, t1;
    prefix_range(L, p.nsplit, split, t_prefix, t0, t1);
    const int np = t1 - t0;
    // one thread: K (V) of prefix tile i of this CTA into stage i % UM_STAGES; K and V complete on barriers of their own,
    // because a stage's K is free again (after S = Q K^T) two tiles before its V is (after O += P V)
    auto issue_kv = [&](int i, bool is_v) {
        const int stage = i % UM_STAGES;
        const unsigned int dst = smem_base + stage * ATT_STAGE_BYTES + (is_v ? ATT_TILE_BYTES : 0);
        const unsigned int bar = (is_v ? bar_v : bar0) + stage * 8;
        const CUtensorMap* tm = is_v ? &tmV : &tmK;
        const int tok = kv0 + (t0 + i) * ATT_BN;
        mbar_expect_tx(bar, ATT_TILE_BYTES);
        if (p.head_first) {
            tma_load_3d(dst, tm, 0, tok, h, bar);
            tma_load_3d(dst + ATT_TILE_BYTES / 2, tm, 64, tok, h, bar);
        } else {
            tma_load_3d(dst, tm, 0, h, tok, bar);
            tma_load_3d(dst + ATT_TILE_BYTES / 2, tm, 64, h, tok, bar);
        }
    };
    const int pre = min(np, UM_STAGES);
    if (tid == 0) {
        for (int i = 0; i < 4 * UM_STAGES + 4; ++i) mbar_init(bar0 + i * 8, 1);
        mbar_init(bar_p, UM_ROWS_THREADS);               // P of a tile is written: one arrival per thread of the stream
        mbar_init(bar_p + 8, UM_ROWS_THREADS);
        mbar_init(bar_sr, UM_ROWS_THREADS);              // S of a tile is in registers: its buffer may take the next S
        mbar_init(bar_sr + 8, UM_ROWS_THREADS);
        mbar_init_fence();
        if (p.prefetch)                                  // the caller vouches for the cache: tiles requested ahead of the wait
            for (int i = 0; i < pre; ++i) { issue_kv(i, false); issue_kv(i, true); }
    }
    if (warp == 0) {
        tmem_alloc(tslot, UM_TMEM_COLS);
        tmem_relinquish();
    }
    pdl_launch_dependents();
    pdl_wait();                                      // the pruned tree, q, k_tree, v_tree come from upstream
    if (tid == 0 && !p.prefetch)
        for (int i = 0; i < pre; ++i) { issue_kv(i, false); issue_kv(i, true); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const unsigned int tmem_base = *tslot_gen;
    const unsigned int lane_off = (unsigned int)((warp & 3) * 32) << 16;   // a warp reaches lanes 32 * (warp % 4) ...
    const int row = tid & (ATT_BM - 1), half = (tid >> 7) & 1;               // the thread's query row and stream
    const unsigned int tS = tmem_base, tO = tmem_base + 128, tP = tmem_base + 384;   // (+ 64 / + 128 / + 32 columns for stream 1)

    const int nk = (p.status[b] == 0) ? p.n_keep[b] : 0;
    const int M = nk * p.G;
    if (m0 >= M) {                                   // nothing to do (the same for every CTA of the cluster)
        if (tid == 0)
            for (int i = 0; i < pre; ++i) {              // no copy may outlive the CTA
                mbar_wait(bar0 + i * 8, 0u, p.err);
                mbar_wait(bar_v + i * 8, 0u, p.err);
            }
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem_base, UM_TMEM_COLS);
        return;
    }
    const int koff = p.keep_off[b];
    const int nt_tree = (split == p.nsplit - 1) ? (nk + ATT_BN - 1) / ATT_BN : 0;
    const int ntiles = np + nt_tree;

    // tree keys and/or values of tile i: gathered rows, 16-byte loads (four of a thread's loads per matrix in flight
    // together), swizzled stores; 1024 chunks per matrix by nthr threads (thread t of them), chunks t + (it0 .. it0 + 3) * nthr
    auto gather_tree = [&](int i, int t, int nthr, int it0, bool do_k, bool do_v) {
        unsigned char* gK = smem_gen + (i % UM_STAGES) * ATT_STAGE_BYTES;
        unsigned char* gV = gK + ATT_TILE_BYTES;
        const int j0 = (i - np) * ATT_BN;
        uint4 kvv[4], vvv[4];
        int trow[4];
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int j = j0 + ((t + (it0 + it) * nthr) >> 4);
            trow[it] = -1;
            if (j < nk) trow[it] = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + j] : koff + j;
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            kvv[it] = make_uint4(0, 0, 0, 0);
            vvv[it] = make_uint4(0, 0, 0, 0);
            if (trow[it] >= 0) {
                const size_t off = ((size_t)trow[it] * p.hkv + h) * HS_HEAD_DIM + (t & 15) * 8;
                if (do_k) kvv[it] = __ldg(reinterpret_cast<const uint4*>(p.k_tree + off));
                if (do_v) vvv[it] = __ldg(reinterpret_cast<const uint4*>(p.v_tree + off));
            }
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int c = t + (it0 + it) * nthr;
            if (do_k) *reinterpret_cast<uint4*>(gK + tile_off(c >> 4, c & 15)) = kvv[it];
            if (do_v) *reinterpret_cast<uint4*>(gV + tile_off(c >> 4, c & 15)) = vvv[it];
        }
    };

    // ---- this thread's query row -> shared memory, its ancestor mask and output row ---------------------------
    const int r = m0 + row;
    long long orow = -1;
    unsigned long long mk0 = 0ull, mk1 = 0ull;
    {
        uint4 qv[8];                                     // this thread's half of the row
#pragma unroll
        for (int c = 0; c < 8; ++c) qv[c] = make_uint4(0, 0, 0, 0);
        if (r < M && warp < 8) {
            const int node = r / p.G, g = r - node * p.G;
            const int trow = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + node] : koff + node;
            orow = (long long)trow * p.hq + h * p.G + g;
            mk0 = p.anc_mask[2 * (size_t)(koff + node)];
            mk1 = p.anc_mask[2 * (size_t)(koff + node) + 1];
            const uint4* src = reinterpret_cast<const uint4*>(p.q + (size_t)orow * HS_HEAD_DIM) + half * 8;
#pragma unroll
            for (int c = 0; c < 8; ++c) qv[c] = __ldg(src + c);
        }
        if (warp < 8) {
#pragma unroll
            for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(gQ + q_off(row, half * 8 + c)) = qv[c];
        }
    }
    if (warp < 8)
        for (int i = np; i < min(ntiles, UM_STAGES); ++i) gather_tree(i, tid, UM_SM_THREADS, 0, true, true);  // tree tiles that open the pipeline
    fence_proxy_async_smem();                        // generic stores -> visible to the tensor cores
    __syncthreads();

    const unsigned int idesc_qk = umma_idesc_bf16(ATT_BM, ATT_BN, false);
    const unsigned int idesc_pv = umma_idesc_bf16(ATT_BM, HS_HEAD_DIM, true);
    // Operand descriptors: the start-address field (16-byte units, low 14 bits) is the only part that varies, and no
    // shared-memory address reaches 2^18, so an offset is added to a descriptor built once.
    const unsigned long long dq0 = umma_desc_sw128(sQ, 16, 1024), dk0 = umma_desc_sw128(smem_base, 16, 1024);
    const unsigned long long dv0 = umma_desc_sw128(smem_base + ATT_TILE_BYTES, ATT_TILE_BYTES / 2, 1024);
    // the issuing thread: S = Q K^T of tile i into S buffer i & 1 (waits for K if it comes by TMA), then commit
    auto issue_qk = [&](int i) {
        const int stage = i % UM_STAGES;
        if (i < np) mbar_wait(bar0 + stage * 8, (unsigned int)(i / UM_STAGES) & 1u, p.err);
        tc_fence_after_sync();
        const unsigned long long dk = dk0 + (unsigned long long)(stage * (ATT_STAGE_BYTES >> 4));
        const unsigned int ts = tS + (i & 1) * ATT_BN;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const unsigned int koffb = (ks >> 2) * (ATT_TILE_BYTES / 2) + (ks & 3) * 32;
            const unsigned int qoffb = (ks >> 2) * (ATT_Q_BYTES / 2) + (ks & 3) * 32;
            umma_ss_bf16(ts, dq0 + (qoffb >> 4), dk + (koffb >> 4), idesc_qk, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_s + (i & 1) * 8);
        if (i + UM_STAGES < np) umma_commit(bar_ek + stage * 8);     // (the producer waits for it only then)
    };
    // O of stream i & 1 += P V of tile i (waits for V if it comes by TMA), then commit
    auto issue_pv = [&](int i) {
        const int stage = i % UM_STAGES;
        if (i < np) mbar_wait(bar_v + stage * 8, (unsigned int)(i / UM_STAGES) & 1u, p.err);
        tc_fence_after_sync();
        const unsigned long long dv = dv0 + (unsigned long long)(stage * (ATT_STAGE_BYTES >> 4));
        const unsigned int tp = tP + (i & 1) * (ATT_BN / 2);
        const unsigned int to = tO + (i & 1) * HS_HEAD_DIM;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)                       // 16 keys per instruction: two 8-key groups of V
            umma_ts_bf16(to, tp + kk * 8, dv + (kk * 2048 >> 4), idesc_pv, (i > 1 || kk > 0) ? 1u : 0u);
        umma_commit(bar_ev + stage * 8);
    };
    float mrun = -CUDART_INF_F, lrun = 0.f;

    // ---- KV tiles ------------------------------------------------------------------------------------------
    // Both single-thread roles sit behind a branch on a warp-uniform value with the thread chosen by elect.sync in
    // every round (all lanes run the loop): the compiler then keeps loop counters, addresses and descriptors uniform.
    const int warp_u = __shfl_sync(HS_FULL_MASK, warp, 0);
    if (warp_u == 8) {
        // The P V issuer: O += P V of tile i as soon as its P is written.  It is short work on the streams' critical
        // path (a stream may not write P of tile i + 2 before it is complete), so it has a thread of its own that is
        // never held up behind the issue of an S.
#pragma unroll 1
        for (int i = 0; i < ntiles; ++i) {
            if (elect_one()) {
                mbar_wait(bar_p + (i & 1) * 8, (unsigned int)(i >> 1) & 1u, p.err);   // P of tile i is written
                issue_pv(i);
                // every S was read before the last P was written: all tensor-core work of this CTA is complete
                if (i == ntiles - 1) umma_commit(bar_done);
            }
            __syncwarp();
        }
    } else if (warp_u == 10) {
        // The S issuer: S of tile i + 2 as soon as the stream has S of tile i in registers, so a stream never waits
        // for its next S.
        if (elect_one()) {
            if (ntiles > 0) issue_qk(0);
            if (ntiles > 1) issue_qk(1);
        }
        __syncwarp();
#pragma unroll 1
        for (int i = 0; i + 2 < ntiles; ++i) {
            if (elect_one()) {
                mbar_wait(bar_sr + (i & 1) * 8, (unsigned int)(i >> 1) & 1u, p.err);      // S of tile i is read
                issue_qk(i + 2);
            }
            __syncwarp();
        }
    } else if (warp_u == 9) {
        // The TMA producer, in the order in which the tensor pipe frees the stage halves: S runs four tiles ahead
        // of O += P V, so after the first K refills it is V of tile i + 4 (after P V of tile i), then K of tile i + 8
        // (after S of tile i + 4).
#pragma unroll 1
        for (int t = UM_STAGES; t < min(np, 2 * UM_STAGES); ++t) {
            if (elect_one()) {
                mbar_wait(bar_ek + (t % UM_STAGES) * 8, 0u, p.err);
                issue_kv(t, false);
            }
            __syncwarp();
        }
#pragma unroll 1
        for (int i = 0; i + UM_STAGES < np; ++i) {
            if (elect_one()) {
                mbar_wait(bar_ev + (i % UM_STAGES) * 8, (unsigned int)(i / UM_STAGES) & 1u, p.err);
                issue_kv(i + UM_STAGES, true);
                if (i + 2 * UM_STAGES < np) {
                    mbar_wait(bar_ek + (i % UM_STAGES) * 8, (unsigned int)(i / UM_STAGES + 1) & 1u, p.err);
                    issue_kv(i + 2 * UM_STAGES, false);
                }
            }
            __syncwarp();
        }
    }
    // Stream `half`: tiles half, half + 2, ...  As soon as S of tile i is in registers its buffer is handed back.  The
    // stream's P buffer and O were last used by O += P V of tile i - 2, which is waited for before they are touched
    // (its barrier's next completion is tile i + 2's, which needs this stream's P of tile i + 2).
#pragma unroll 1
    for (int i = half; i < ntiles && warp < 8; i += 2) {
        mbar_wait(bar_s + half * 8, (unsigned int)(i >> 1) & 1u, p.err);         // S of tile i is complete
        tc_fence_after_sync();
        unsigned int sr[64];                                 // the row's 64 scores
        tmem_ld32(tS + half * ATT_BN + lane_off, sr);
        tmem_ld32(tS + half * ATT_BN + 32 + lane_off, sr + 32);
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive(bar_sr + half * 8);

        const bool is_tree = i >= np;
        const int col0 = is_tree ? (i - np) * ATT_BN : (t0 + i) * ATT_BN;
        const int nvis = (is_tree ? nk : L) - col0;          // columns of this tile inside the sequence / tree
        // The scores stay unscaled in registers (the scale is positive: it commutes with the maximum and folds into
        // the exponent's multiply-add). A prefix tile inside the sequence needs no mask at all.
        float mxa = -CUDART_INF_F, mxb = -CUDART_INF_F;
        if (is_tree || nvis < ATT_BN) {
            // a tree tile of 64 keys lies inside one 64-bit word of the ancestor mask
            unsigned long long vis64 = nvis >= 64 ? ~0ull : ((1ull << max(nvis, 0)) - 1ull);
            if (is_tree) vis64 &= (col0 == 0 ? mk0 : mk1);
            const unsigned int vlo = (unsigned int)vis64, vhi = (unsigned int)(vis64 >> 32);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                if (!((vlo >> c) & 1u)) sr[c] = __float_as_uint(-CUDART_INF_F);
                if (!((vhi >> c) & 1u)) sr[32 + c] = __float_as_uint(-CUDART_INF_F);
            }
        }
#pragma unroll
        for (int c = 0; c < 32; c += 2) {                    // three-input maxima: half the instructions
            mxa = max3(mxa, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
            mxb = max3(mxb, __uint_as_float(sr[32 + c]), __uint_as_float(sr[33 + c]));
        }
        const float mx = fmaxf(mxa, mxb) * p.scale_log2;
        // The reference the exponents are taken against only follows the row's maximum when that has grown by more
        // than 8 (a factor 256): until then P <= 256 instead of <= 1, which costs no precision (fp32 sums, bf16 keeps
        // its relative error, the final O / l is the same quotient), and O is rescaled a few times per row instead of
        // whenever any row of the warp sees a new maximum.
        const float mnew = (mx > mrun + 8.f || mrun == -CUDART_INF_F) ? fmaxf(mrun, mx) : mrun;
        const float muse = (mnew == -CUDART_INF_F) ? 0.f : mnew;
        const float corr = ex2_approx(mrun - muse);          // 1 when the maximum did not grow, 0 at the stream's first tile
        mrun = mnew;
        // the row's P of this tile, in registers first
        // (the exponent's multiply-add and the row sum run as packed fp32 pairs: half the instructions)
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-muse, -muse);
        float2 ls0 = make_float2(0.f, 0.f), ls1 = make_float2(0.f, 0.f);
        uint4 pk[8];
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
            float2 pv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = fma2_ftz(make_float2(__uint_as_float(sr[c8 * 8 + 2 * e]), __uint_as_float(sr[c8 * 8 + 2 * e + 1])), sc2, nm2);
                pv[e] = make_float2(ex2_approx(x.x), ex2_approx(x.y));
            }
            ls0 = add2_ftz(ls0, add2_ftz(pv[0], pv[1]));
            ls1 = add2_ftz(ls1, add2_ftz(pv[2], pv[3]));
            pk[c8].x = pack_bf16(pv[0].x, pv[0].y); pk[c8].y = pack_bf16(pv[1].x, pv[1].y);
            pk[c8].z = pack_bf16(pv[2].x, pv[2].y); pk[c8].w = pack_bf16(pv[3].x, pv[3].y);
        }
        const float2 ls = add2_ftz(ls0, ls1);
        lrun = fmaf(lrun, corr, ls.x + ls.y);
        // Tree tiles are gathered by the stream two and four tiles ahead of their use, where the stage half is free
        // and this tile's P-written arrival publishes the stores before the issuing thread needs them: K of tile
        // i + 4 (its stage's K was read by S of tile i, complete), V of tile i + 2 (after O += P V of tile i - 2).
        if (i + UM_STAGES < ntiles && i + UM_STAGES >= np) {
            gather_tree(i + UM_STAGES, row, UM_ROWS_THREADS, 0, true, false);
            gather_tree(i + UM_STAGES, row, UM_ROWS_THREADS, 4, true, false);
        }
        if (i >= 2) {
            mbar_wait(bar_ev + ((i - 2) % UM_STAGES) * 8, (unsigned int)((i - 2) / UM_STAGES) & 1u, p.err);
            tc_fence_after_sync();
            if (i + 2 < ntiles && i + 2 >= np) {
                gather_tree(i + 2, row, UM_ROWS_THREADS, 0, false, true);
                gather_tree(i + 2, row, UM_ROWS_THREADS, 4, false, true);
            }
        }
        // rescale this stream's O (the load/store are warp-wide: a warp rescales if any of its rows needs it)
        if (i >= 2 && __any_sync(HS_FULL_MASK, corr != 1.f)) {
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
                unsigned int ov[32];
                tmem_ld32(tO + half * HS_HEAD_DIM + lane_off + ch * 32, ov);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * corr);
                tmem_st32(tO + half * HS_HEAD_DIM + lane_off + ch * 32, ov);
            }
            tmem_wait_st();
        }
        // P stays in tensor memory (the A operand of O += P V): this row's 64 bf16 values are 32 columns of its lane
        tmem_st32(tP + half * (ATT_BN / 2) + lane_off, reinterpret_cast<unsigned int*>(pk));
        tmem_wait_st();
        if (i + UM_STAGES >= np) fence_proxy_async_smem();   // gathered tree tiles (generic stores) -> tensor cores
        tc_fence_before_sync();
        mbar_arrive(bar_p + half * 8);
    }
    if (ntiles > 0 && warp < 8) mbar_wait(bar_done, 0u, p.err);
    __syncwarp();                                        // the issuing and producer warps reconverge (warp-aligned barriers follow)
    tc_fence_after_sync();
    // the two streams of a row are combined like two splits: weights w0, w1 on the streams' O, one (max, sum)
    if (warp < 8) { s_mx[half * ATT_BM + row] = mrun; s_lx[half * ATT_BM + row] = lrun; }
    __syncthreads();
    float w0 = 0.f, w1 = 0.f;
    if (warp < 8) {
        const float m_a = s_mx[row], m_b = s_mx[ATT_BM + row];
        mrun = fmaxf(m_a, m_b);
        const float muse = (mrun == -CUDART_INF_F) ? 0.f : mrun;
        w0 = ex2_approx(m_a - muse);
        w1 = ex2_approx(m_b - muse);
        lrun = s_lx[row] * w0 + s_lx[ATT_BM + row] * w1;
    }
    // this thread's 32 columns [half * 64 + ch * 32, + 32) of the row's combined O (a stream without tiles has no O)
    auto load_o = [&](int ch, unsigned int* ov) {
        unsigned int oa[32], ob[32];
        if (ntiles > 0) tmem_ld32(tO + lane_off + half * 64 + ch * 32, oa);
        if (ntiles > 1) tmem_ld32(tO + HS_HEAD_DIM + lane_off + half * 64 + ch * 32, ob);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            float v = 0.f;
            if (ntiles > 0) v = __uint_as_float(oa[c]) * w0;
            if (ntiles > 1) v = fmaf(__uint_as_float(ob[c]), w1, v);
            ov[c] = __float_as_uint(v);
        }
    };

    // ---- epilogue ----------------------------------------------------------------------------------------------
    if (p.nsplit == 1) {
        const float inv = lrun > 0.f ? 1.f / lrun : 0.f;
#pragma unroll 1
        for (int ch = 0; ch < 2 && warp < 8; ++ch) {
            unsigned int ov[32];
            load_o(ch, ov);
            if (orow >= 0) {
                uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)orow * HS_HEAD_DIM + half * 64 + ch * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(ov[q * 8 + 0]) * inv, __uint_as_float(ov[q * 8 + 1]) * inv);
                    pk.y = pack_bf16(__uint_as_float(ov[q * 8 + 2]) * inv, __uint_as_float(ov[q * 8 + 3]) * inv);
                    pk.z = pack_bf16(__uint_as_float(ov[q * 8 + 4]) * inv, __uint_as_float(ov[q * 8 + 5]) * inv);
                    pk.w = pack_bf16(__uint_as_float(ov[q * 8 + 6]) * inv, __uint_as_float(ov[q * 8 + 7]) * inv);
                    dst[q] = pk;
                }
            }
        }
        if (orow >= 0 && p.lse_out && half == 0) p.lse_out[orow] = (mrun + log2f(lrun)) * LN2;
    } else {
        // ---- merge across the splits of the cluster through distributed shared memory ----------------------------
        // Row rl of the block is merged by CTA owner(rl) = rl * ns / 128.  Every CTA stages its partial of every row,
        // {O / l as bf16, max, sum}, in its own shared memory and one thread PUSHES each owner's rows with a bulk
        // copy that signals the owner's mbarrier; an owner merges once all ns pieces have landed: per row the
        // splits' weights 2^(max_s - max) l_s / sum once, then out = sum_s weight_s (O_s / l_s).  (A normalised
        // partial is a convex combination of V rows, so bf16 keeps it to 2^-9 of the values' magnitude: the output
        // is bf16 anyway.)
        const int ns = p.nsplit;
        // shared memory after the tile loop: [0, UM_RECV_BYTES) partials received from the cluster (others write
        // here, so only after every CTA of the cluster has left its loop), then this CTA's own staged partial
        unsigned char* po = smem_gen;                                                // [ns][rows_max] rows of ATT_PB_STRIDE bytes
        unsigned char* stage_po = smem_gen + UM_RECV_BYTES;                          // [128] rows: own partial
        const unsigned int s_recv = smem_base, s_stage = smem_base + UM_RECV_BYTES;
        const int rows_max = (ATT_BM + ns - 1) / ns + 1;
        const int r_lo = (split * ATT_BM + ns - 1) / ns, r_hi = ((split + 1) * ATT_BM + ns - 1) / ns;   // rows this CTA owns
        long long* s_og = reinterpret_cast<long long*>(gM);               // output row of each owned row (or -1)
        float* s_wt = reinterpret_cast<float*>(gM + UM_MAP_BYTES + 1024);  // [rows owned][ATT_MAX_SPLIT] weights (s_mx / s_lx are done)
        if (tid == 0) mbar_expect_tx(bar_r, (unsigned int)(ns * (r_hi - r_lo) * ATT_PB_STRIDE));
        if (tid < r_hi - r_lo) {
            const int rg = m0 + r_lo + tid;
            long long og = -1;
            if (rg < M) {
                const int node = rg / p.G, g = rg - node * p.G;
                const int trow = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + node] : koff + node;
                og = (long long)trow * p.hq + h * p.G + g;
            }
            s_og[tid] = og;
        }
        {
            const float inv = lrun > 0.f ? 1.f / lrun : 0.f;
#pragma unroll 1
            for (int ch = 0; ch < 2 && warp < 8; ++ch) {
                unsigned int ov[32];
                load_o(ch, ov);
                uint4* dst = reinterpret_cast<uint4*>(stage_po + row * ATT_PB_STRIDE + (half * 64 + ch * 32) * 2);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(ov[q * 8 + 0]) * inv, __uint_as_float(ov[q * 8 + 1]) * inv);
                    pk.y = pack_bf16(__uint_as_float(ov[q * 8 + 2]) * inv, __uint_as_float(ov[q * 8 + 3]) * inv);
                    pk.z = pack_bf16(__uint_as_float(ov[q * 8 + 4]) * inv, __uint_as_float(ov[q * 8 + 5]) * inv);
                    pk.w = pack_bf16(__uint_as_float(ov[q * 8 + 6]) * inv, __uint_as_float(ov[q * 8 + 7]) * inv);
                    dst[q] = pk;
                }
            }
            if (warp < 4) *reinterpret_cast<float2*>(stage_po + row * ATT_PB_STRIDE + HS_HEAD_DIM * 2) = make_float2(mrun, lrun);
        }
        fence_proxy_async_smem();                            // staged rows -> visible to the copy engine
        cluster_arrive();                                    // every CTA of the cluster is done with its tiles:
        cluster_wait();                                      // its stage buffers may now receive partials
        if (tid < ns) {                                      // thread o: the rows of owner o
            const int o = tid;
            const int o_lo = (o * ATT_BM + ns - 1) / ns, o_hi = ((o + 1) * ATT_BM + ns - 1) / ns;
            if (o_hi > o_lo)
                bulk_push(cluster_map_addr(s_recv + (unsigned int)(split * rows_max) * ATT_PB_STRIDE, o),
                          s_stage + (unsigned int)o_lo * ATT_PB_STRIDE, (unsigned int)(o_hi - o_lo) * ATT_PB_STRIDE,
                          cluster_map_addr(bar_r, o));
        }
        mbar_wait(bar_r, 0u, p.err);                         // all ns pieces of this CTA's rows have landed
        cluster_arrive();                                    // (a CTA may leave only when every copy has landed everywhere)
        // the splits' weights of every owned row, once
        if (tid < r_hi - r_lo) {
            float2 ml[ATT_MAX_SPLIT];
            float Mx = -CUDART_INF_F;
#pragma unroll
            for (int s2 = 0; s2 < ATT_MAX_SPLIT; ++s2) {
                ml[s2] = make_float2(-CUDART_INF_F, 0.f);
                if (s2 < ns) ml[s2] = *reinterpret_cast<const float2*>(po + (size_t)(s2 * rows_max + tid) * ATT_PB_STRIDE + HS_HEAD_DIM * 2);
                Mx = fmaxf(Mx, ml[s2].x);
            }
            float w[ATT_MAX_SPLIT], lsum = 0.f;
#pragma unroll
            for (int s2 = 0; s2 < ATT_MAX_SPLIT; ++s2) {
                w[s2] = (ml[s2].x == -CUDART_INF_F) ? 0.f : ex2_approx(ml[s2].x - Mx) * ml[s2].y;
                lsum += w[s2];
            }
            const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
#pragma unroll
            for (int s2 = 0; s2 < ATT_MAX_SPLIT; ++s2) s_wt[tid * ATT_MAX_SPLIT + s2] = w[s2] * inv;
            const long long og = s_og[tid];
            if (og >= 0 && p.lse_out) p.lse_out[og] = (Mx + log2f(lsum)) * LN2;
        }
        if (tid < UM_SM_THREADS)                             // the softmax threads: the weights are written
            asm volatile("bar.sync 2, %0;" ::"r"(UM_SM_THREADS) : "memory");
        // items = (row, 16-byte column group of 8); every item combines one group of each split, all from local shared memory
        for (int it = tid; it < (r_hi - r_lo) * 16 && tid < UM_SM_THREADS; it += UM_SM_THREADS) {
            const int rl = it >> 4, c8 = it & 15;
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
            for (int s2 = 0; s2 < ATT_MAX_SPLIT; ++s2) {
                if (s2 < ns) {
                    const float w = s_wt[rl * ATT_MAX_SPLIT + s2];
                    const uint4 v = *reinterpret_cast<const uint4*>(po + (size_t)(s2 * rows_max + rl) * ATT_PB_STRIDE + c8 * 16);
                    acc[0] = fmaf(w, bf16_lo(v.x), acc[0]); acc[1] = fmaf(w, bf16_hi(v.x), acc[1]);
                    acc[2] = fmaf(w, bf16_lo(v.y), acc[2]); acc[3] = fmaf(w, bf16_hi(v.y), acc[3]);
                    acc[4] = fmaf(w, bf16_lo(v.z), acc[4]); acc[5] = fmaf(w, bf16_hi(v.z), acc[5]);
                    acc[6] = fmaf(w, bf16_lo(v.w), acc[6]); acc[7] = fmaf(w, bf16_hi(v.w), acc[7]);
                }
            }
            const long long og = s_og[rl];
            if (og >= 0) {
                uint4 packed;
                packed.x = pack_bf16(acc[0], acc[1]); packed.y = pack_bf16(acc[2], acc[3]);
                packed.z = pack_bf16(acc[4], acc[5]); packed.w = pack_bf16(acc[6], acc[7]);
                *reinterpret_cast<uint4*>(p.out + (size_t)og * HS_HEAD_DIM + c8 * 8) = packed;
            }
        }
        cluster_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, UM_TMEM_COLS);
}
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool make_kv_map(hs_ctx* ctx, CUtensorMap* tm, const void* base, const hs_attn_desc* d, bool head_first) {
    cuuint64_t gdim[3], gstr[2];
    cuuint32_t box[3], estr[3] = {1, 1, 1};
    gdim[0] = HS_HEAD_DIM;
    box[0] = 64;
    if (head_first) {        // (d, token, head): token stride is the smaller one
        gdim[1] = (cuuint64_t)d->kv_total; gdim[2] = (cuuint64_t)d->hkv;
        gstr[0] = (cuuint64_t)d->kv_token_stride * 2; gstr[1] = (cuuint64_t)d->kv_head_stride * 2;
        box[1] = ATT_BN; box[2] = 1;
    } else {                 // (d, head, token)
        gdim[1] = (cuuint64_t)d->hkv; gdim[2] = (cuuint64_t)d->kv_total;
        gstr[0] = (cuuint64_t)d->kv_head_stride * 2; gstr[1] = (cuuint64_t)d->kv_token_stride * 2;
        box[1] = 1; box[2] = ATT_BN;
    }
    CUresult r = ((encode_tiled_fn)ctx->encode_tiled)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                     gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// KV splits (= cluster size): the one with the fewest tile steps on the critical path, waves of CTAs (as
// many clusters of that size as the device runs at once) times tiles per CTA.  `step` = 1 tries 1..8,
// `step` = 2 only powers of two.
static int choose_splits(int base_ctas, int sm_count, int prefix_tiles, const int* cluster_cap) {
    int best = 1;
    long best_cost = 0;
    for (int s = 1; s <= ATT_MAX_SPLIT; ++s) {
        if (s > 1 && s > prefix_tiles) break;
        const long ctas = (long)base_ctas * s;
        const long cap = cluster_cap[s] > 0 ? cluster_cap[s] : sm_count;
        const long waves = (ctas + cap - 1) / cap;
        const long cost = waves * ((prefix_tiles + s - 1) / s + 2 + (s > 1 ? 2 : 0));   // + tree tiles, + merge
        if (s == 1 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

template <typename Kernel>
static void query_cluster_caps(Kernel kernel, int threads, size_t smem, int sm_count, int* cap) {
    for (int sz = 1; sz <= ATT_MAX_SPLIT; ++sz) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1, sz, sm_count);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = sz; at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, kernel, &cfg) == cudaSuccess) cap[sz] = nclusters * sz;
        else { cap[sz] = 0; (void)cudaGetLastError(); }
    }
}

hs_status hs_launch_attention(hs_ctx* ctx, const hs_pruned_tree* pruned, const hs_attn_desc* d, const void* q,
                              const void* k_tree, const void* v_tree, const void* k_cache, const void* v_cache,
                              void* out, float* lse_out, cudaStream_t stream) {
    int* cap_umma = ctx->attn_cap;                   // CTAs that run at once in clusters of s (per device = per context)
    if (!ctx->attn_ready) {
        if (cudaFuncSetAttribute(tree_attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, UM_SMEM_BYTES) !=
            cudaSuccess)
            return HS_ERR_CUDA;
        query_cluster_caps(tree_attn_umma_kernel, UM_THREADS, UM_SMEM_BYTES, ctx->sm_count, cap_umma);
        ctx->attn_ready = true;
    }
    AttnParams p;
    p.q = (const __nv_bfloat16*)q;
    p.k_tree = (const __nv_bfloat16*)k_tree;
    p.v_tree = (const __nv_bfloat16*)v_tree;
    p.out = (__nv_bfloat16*)out;
    p.lse_out = lse_out;
    p.n_keep = pruned->n_keep;
    p.keep_off = pruned->keep_off;
    p.keep_idx = pruned->keep_idx;
    p.anc_mask = (const unsigned long long*)pruned->anc_mask;
    p.status = pruned->status;
    p.node_off = d->node_off;
    p.kv_off = d->kv_off;
    p.batch = d->batch;
    p.hq = d->hq;
    p.hkv = d->hkv;
    p.G = d->hq / d->hkv;
    p.layout = d->layout;
    p.head_first = d->kv_head_stride > d->kv_token_stride;
    p.scale_log2 = d->sm_scale * LOG2E;
    p.err = ctx->counters + HS_CNT_ERROR;
    p.prefetch = (ctx->prefetch & HS_PREFETCH_KV) != 0;
    const int pairs = d->batch * d->hkv;
    const int mblocks = (p.G * d->max_nodes + ATT_BM - 1) / ATT_BM;
    const int prefix_tiles = (d->max_kv_len + ATT_BN - 1) / ATT_BN;
    p.nsplit = choose_splits(pairs * mblocks, ctx->sm_count, prefix_tiles, cap_umma);

    CUtensorMap tmK, tmV;
    memset(&tmK, 0, sizeof(tmK));
    memset(&tmV, 0, sizeof(tmV));
    if (d->kv_total > 0) {
        if (!make_kv_map(ctx, &tmK, k_cache, d, p.head_first) || !make_kv_map(ctx, &tmV, v_cache, d, p.head_first))
            return HS_ERR_CUDA;
    }
    const dim3 grid(mblocks, p.nsplit, pairs), cl(1, p.nsplit, 1);
    cudaError_t e = hs_launch(tree_attn_umma_kernel, grid, dim3(UM_THREADS), UM_SMEM_BYTES, stream, ctx->pdl, cl, p, tmK, tmV);
    return e == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
