// hs_expand_init / hs_expand_level / hs_rerank: the draft tree of Sec. 2.2 grown and reranked on the device.
//
// The candidate tree of a sequence lives in caller-owned arrays of `cap` slots in creation order (candidate 0 = the
// root, parents precede children).  One expansion level (one CTA per sequence): every frontier node gets the k most
// likely tokens of its draft row as children - the Top-K tokens and logits of that row and its log-sum-exp are
// what hs_entropy_quantify writes -, a child's value is its parent's plus its log-confidence (ln V_i = sum ln c_j),
// and the k children with the largest value (ties: created first) become the next frontier.  Reranking (one CTA
// per sequence): the N candidates with the largest value, compacted in creation order with parents re-indexed: a
// topologically ordered tree ready for the verification calls.  Ranks are found by counting, compaction by warp
// ballots and a prefix sum over the warps.
#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

#define EX_THREADS 256
#define EX_MAX_CAP 2048        // candidates per sequence the reranking holds in shared memory

__global__ void expand_init_kernel(hs_expand_state st) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    if (b >= st.batch) return;
    const size_t o = (size_t)b * st.cap;
    st.n_cand[b] = 1;
    st.parent[o] = -1; st.token[o] = -1; st.depth[o] = 0; st.logc[o] = 0.f; st.score[o] = 0.f;
    st.frontier[(size_t)b * st.top_k] = 0;
    st.n_frontier[b] = 1;
    st.status[b] = HS_OK;
}

__global__ void __launch_bounds__(EX_THREADS) expand_level_kernel(hs_expand_state st, const float* topk_val,
                                                                  const int* topk_idx, const float* row_lse, int K) {
    __shared__ float s_S[HS_MAX_TOPK * HS_MAX_TOPK];
    __shared__ int s_bad;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int k = st.top_k;
    pdl_launch_dependents();
    pdl_wait();                                    // the row statistics come from the kernel ahead
    if (st.status[b] != HS_OK) return;
    const size_t o = (size_t)b * st.cap;
    const int n0 = st.n_cand[b], nf = st.n_frontier[b];
    const int nnew = nf * k;
    if (tid == 0) s_bad = 0;
    __syncthreads();
    if (n0 + nnew > st.cap) {                      // the arrays cannot take another level
        if (tid == 0) st.status[b] = HS_ERR_SHAPE;
        return;
    }
    float S = -CUDART_INF_F;
    int par = -1, tok = -1, dep = 0;
    float lc = 0.f;
    if (tid < nnew) {
        const int j = tid / k, i = tid - j * k;
        const int row = b * k + j;
        par = st.frontier[(size_t)b * k + j];
        tok = topk_idx[(size_t)row * K + i];
        lc = topk_val[(size_t)row * K + i] - row_lse[row];
        S = st.score[o + par] + lc;
        dep = st.depth[o + par] + 1;
        if (tok < 0) s_bad = 1;                    // the row had fewer than k finite logits
        s_S[tid] = S;
    }
    __syncthreads();
    if (s_bad) {
        if (tid == 0) st.status[b] = HS_ERR_BAD_TREE;
        return;
    }
    if (tid < nnew) {
        const int c = n0 + tid;
        st.parent[o + c] = par; st.token[o + c] = tok; st.depth[o + c] = dep;
        st.logc[o + c] = lc; st.score[o + c] = S;
        int rank = 0;                              // by (value descending, creation order)
        for (int j = 0; j < nnew; ++j) rank += (s_S[j] > S || (s_S[j] == S && j < tid));
        if (rank < k) st.frontier[(size_t)b * k + rank] = c;
    }
    if (tid == 0) {
        st.n_cand[b] = n0 + nnew;
        st.n_frontier[b] = min(k, nnew);
    }
}

struct RerankParams {
    hs_expand_state st;
    const int* n_top;      // [B] or NULL
    int n_default;
    int* node_off;         // [B+1]
    int* parent;
    int* token;
    int* cand_id;
    int* depth;
};

__device__ __forceinline__ int rerank_count(const RerankParams& p, int b) {
    if (p.st.status[b] != HS_OK) return 0;
    const int want = p.n_top ? p.n_top[b] : p.n_default;
    return max(0, min(want, p.st.n_cand[b]));
}

__global__ void __launch_bounds__(EX_THREADS) rerank_kernel(const RerankParams p) {
    __shared__ float s_S[EX_MAX_CAP];
    __shared__ short s_new[EX_MAX_CAP];
    __shared__ int s_warp[EX_THREADS / 32];
    __shared__ int s_off;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    pdl_wait();
    // offset of this sequence's tree: the trees ahead of it hold min(N, candidates) nodes each
    int part = 0;
    for (int bb = tid; bb < b; bb += EX_THREADS) part += rerank_count(p, bb);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(HS_FULL_MASK, part, o);
    if (lane == 0) s_warp[warp] = part;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int w = 0; w < EX_THREADS / 32; ++w) t += s_warp[w];
        s_off = t;
    }
    __syncthreads();
    const int off = s_off;
    const int n = p.st.status[b] == HS_OK ? min(p.st.n_cand[b], EX_MAX_CAP) : 0;
    const int want = rerank_count(p, b);
    const size_t o = (size_t)b * p.st.cap;
    for (int c = tid; c < n; c += EX_THREADS) s_S[c] = p.st.score[o + c];
    __syncthreads();
    // candidates in creation order, EX_THREADS at a time; kept ones are numbered by ballot + prefix over the warps
    int base = 0;
    for (int c0 = 0; c0 < n; c0 += EX_THREADS) {
        const int c = c0 + tid;
        bool keep = false;
        if (c < n) {
            const float S = s_S[c];
            int rank = 0;
            for (int j = 0; j < n; ++j) rank += (s_S[j] > S || (s_S[j] == S && j < c));
            keep = rank < want;
        }
        const unsigned int bal = __ballot_sync(HS_FULL_MASK, keep);
        __syncthreads();                           // s_warp is reused
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = base + __popc(bal & ((1u << lane) - 1u));
        int total = 0;
        for (int w = 0; w < EX_THREADS / 32; ++w) { if (w < warp) before += s_warp[w]; total += s_warp[w]; }
        if (c < n) s_new[c] = keep ? (short)before : (short)-1;
        base += total;
    }
    __syncthreads();
    for (int c = tid; c < n; c += EX_THREADS) {
        const int i = s_new[c];
        if (i < 0) continue;
        const int par = p.st.parent[o + c];
        p.parent[off + i] = par >= 0 ? (int)s_new[par] : -1;   // (the kept set is closed under ancestors)
        p.token[off + i] = p.st.token[o + c];
        p.cand_id[off + i] = c;
        p.depth[off + i] = p.st.depth[o + c];
    }
    if (tid == 0) {
        p.node_off[b] = off;
        if (b == p.st.batch - 1) p.node_off[p.st.batch] = off + want;
    }
}

static bool state_ok(const hs_expand_state* s) {
    return s && s->batch >= 1 && s->batch <= HS_MAX_BATCH && s->top_k >= 1 && s->top_k <= HS_MAX_TOPK &&
           s->cap >= 1 + s->top_k && s->n_cand && s->parent && s->token && s->depth && s->logc && s->score &&
           s->frontier && s->n_frontier && s->status;
}

extern "C" hs_status hs_expand_init(hs_ctx* ctx, const hs_expand_state* st, hs_stream stream) {
    if (!ctx || !hs_on_device(ctx) || !state_ok(st)) return HS_ERR_INVALID_ARG;
    return hs_launch(expand_init_kernel, dim3((st->batch + 127) / 128), dim3(128), 0, (cudaStream_t)stream, ctx->pdl,
                     dim3(1, 1, 1), *st) == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

extern "C" hs_status hs_expand_level(hs_ctx* ctx, const hs_expand_state* st, const float* topk_val,
                                     const int32_t* topk_idx, const float* row_lse, int32_t topk_stride,
                                     hs_stream stream) {
    if (!ctx || !hs_on_device(ctx) || !state_ok(st) || !topk_val || !topk_idx || !row_lse) return HS_ERR_INVALID_ARG;
    if (topk_stride < st->top_k) return HS_ERR_INVALID_ARG;
    return hs_launch(expand_level_kernel, dim3(st->batch), dim3(EX_THREADS), 0, (cudaStream_t)stream, ctx->pdl,
                     dim3(1, 1, 1), *st, topk_val, topk_idx, row_lse, (int)topk_stride) == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

extern "C" hs_status hs_rerank(hs_ctx* ctx, const hs_expand_state* st, const int32_t* n_top, int32_t n_default,
                               int32_t* node_off, int32_t* parent, int32_t* token, int32_t* cand_id, int32_t* depth,
                               hs_stream stream) {
    if (!ctx || !hs_on_device(ctx) || !state_ok(st) || !node_off || !parent || !token || !cand_id || !depth)
        return HS_ERR_INVALID_ARG;
    if (st->cap > EX_MAX_CAP || (!n_top && n_default < 1)) return HS_ERR_SHAPE;
    RerankParams p;
    p.st = *st; p.n_top = n_top; p.n_default = n_default;
    p.node_off = node_off; p.parent = parent; p.token = token; p.cand_id = cand_id; p.depth = depth;
    return hs_launch(rerank_kernel, dim3(st->batch), dim3(EX_THREADS), 0, (cudaStream_t)stream, ctx->pdl, dim3(1, 1, 1), p) ==
                   cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
