// hs_stratify_prune: one CTA of 128 threads per sequence, one thread per tree node.
//
// Entropy bin -> (d', N') (Sec. 4.2-4.3), Top-N' reranking by path confidence (Sec. 2.2), then the
// surviving nodes are compacted with warp ballots and a prefix sum over the four warps, parents are
// re-indexed and each kept node gets its ancestor-or-self bit mask (the tree-attention mask).
// The CSR offset of a sequence is the sum of the kept counts of all earlier sequences.  Small batches:
// every CTA recomputes those counts itself, so no CTA waits for another and the call is one launch.
// Larger batches: a first launch counts the kept nodes of every sequence once (one warp each), the
// second sums the counts ahead of its sequence (B integers instead of B trees per CTA).
#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

struct PruneParams {
    int batch;
    const int* node_off;
    const int* parent;
    const float* score;
    const float* phi_star;
    const int* depth;
    const int* qstatus;
    hs_pruned_tree out;
    int counted;           // out.n_keep was filled by prune_count_kernel
    float th[7];
    int d_base, alpha, n_default, gamma_pct[3];
};

__device__ __forceinline__ void policy_lookup(const PruneParams& p, float phi, int& bin, int& dp, int& np) {
    bin = 0;
#pragma unroll
    for (int j = 0; j < 7; ++j) bin += (phi >= p.th[j]);
    if (bin <= 2) {
        int delta = p.alpha - bin;
        dp = p.d_base + delta;
        np = (p.gamma_pct[bin] * p.n_default + 50) / 100 + delta;
    } else {
        dp = p.d_base;
        np = p.n_default;
    }
}

// kept nodes of sequence b: min(N', nodes of depth <= d'); 0 for a sequence flagged bad
__device__ __forceinline__ int kept_count(const PruneParams& p, int b) {
    if (p.qstatus[b] != 0) return 0;
    int bin, dp, np;
    policy_lookup(p, p.phi_star[b], bin, dp, np);
    int lo = p.node_off[b], hi = p.node_off[b + 1], elig = 0;
    for (int i = lo; i < hi; ++i) elig += (p.depth[i] <= dp);
    return max(0, min(np, elig));
}

// one warp per sequence: its kept count -> out.n_keep[b]
__global__ void __launch_bounds__(128) prune_count_kernel(const PruneParams p) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
    pdl_launch_dependents();
    pdl_wait();
    if (b >= p.batch) return;
    int cnt = 0;
    if (p.qstatus[b] == 0) {
        int bin, dp, np;
        policy_lookup(p, p.phi_star[b], bin, dp, np);
        const int lo = p.node_off[b], hi = min(p.node_off[b + 1], lo + HS_MAX_NODES);
        int elig = 0;
        for (int i = lo + lane; i < hi; i += 32) elig += (p.depth[i] <= dp);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) elig += __shfl_xor_sync(HS_FULL_MASK, elig, o);
        cnt = max(0, min(np, elig));
    }
    if (lane == 0) p.out.n_keep[b] = cnt;
}

__global__ void __launch_bounds__(HS_MAX_NODES) stratify_prune_kernel(const PruneParams p) {
    __shared__ float s_S[HS_MAX_NODES];
    __shared__ int s_elig[HS_MAX_NODES];
    __shared__ int s_new[HS_MAX_NODES];
    __shared__ int s_par[HS_MAX_NODES];
    __shared__ int s_warp[4];
    __shared__ int s_off;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();                            // scores and Phi(P*) come from the kernel ahead in the stream
    const int base = p.node_off[b];
    const int n = min(p.node_off[b + 1] - base, HS_MAX_NODES);

    // offset of this sequence in the compacted arrays
    int part = 0;
    if (p.counted) {
        for (int bb = tid; bb < b; bb += HS_MAX_NODES) part += p.out.n_keep[bb];
    } else {
        for (int bb = tid; bb < b; bb += HS_MAX_NODES) part += kept_count(p, bb);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(HS_FULL_MASK, part, o);
    if (lane == 0) s_warp[warp] = part;
    __syncthreads();
    if (tid == 0) s_off = s_warp[0] + s_warp[1] + s_warp[2] + s_warp[3];
    __syncthreads();
    const int off = s_off;

    const int status = p.qstatus[b];
    int bin = 0, dp = 0, np = 0;
    policy_lookup(p, p.phi_star[b], bin, dp, np);

    int dep = 0, par = -1;
    float S = 0.f;
    bool elig = false;
    if (tid < n && status == 0) {
        dep = p.depth[base + tid];
        par = p.parent[base + tid];
        S = p.score[base + tid];
        elig = dep <= dp;
    }
    s_S[tid] = S;
    s_elig[tid] = elig;
    s_par[tid] = par;
    __syncthreads();
    // rank among eligible nodes by (S descending, index ascending)
    int rank = 0;
    if (elig) {
        for (int j = 0; j < n; ++j)
            rank += (s_elig[j] && (s_S[j] > S || (s_S[j] == S && j < tid)));
    }
    const bool keep = elig && rank < np;
    // compaction: ballot inside the warp, prefix over the four warps
    const unsigned int bal = __ballot_sync(HS_FULL_MASK, keep);
    __syncthreads();                       // s_warp is reused
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int before = __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    const int n_keep = s_warp[0] + s_warp[1] + s_warp[2] + s_warp[3];
    s_new[tid] = keep ? before : -1;
    __syncthreads();
    if (keep) {
        const int k = off + before;
        unsigned long long m0 = 0ull, m1 = 0ull;
        int a = tid;
        for (int step = 0; step <= HS_MAX_NODES && a >= 0; ++step) {   // walk to the root
            int na = s_new[a];
            if (na >= 0) {
                if (na < 64) m0 |= 1ull << na; else m1 |= 1ull << (na - 64);
            }
            a = s_par[a];
        }
        p.out.keep_idx[k] = tid;
        p.out.new_parent[k] = par >= 0 ? s_new[par] : -1;
        p.out.new_depth[k] = dep;
        p.out.keep_rank[k] = rank;
        p.out.anc_mask[2 * (size_t)k] = m0;
        p.out.anc_mask[2 * (size_t)k + 1] = m1;
    }
    if (tid == 0) {
        p.out.bin[b] = bin;
        p.out.d_prime[b] = dp;
        p.out.n_prime[b] = np;
        p.out.n_keep[b] = n_keep;
        p.out.keep_off[b] = off;
        if (b == p.batch - 1) p.out.keep_off[p.batch] = off + n_keep;
        p.out.status[b] = status;
    }
}

hs_status hs_launch_stratify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                   const hs_policy* policy, const hs_pruned_tree* out, cudaStream_t stream) {
    PruneParams p;
    p.batch = tree->batch;
    p.node_off = tree->node_off;
    p.parent = tree->parent;
    p.score = quant->score;
    p.phi_star = quant->phi_star;
    p.depth = quant->depth;
    p.qstatus = quant->status;
    p.out = *out;
    for (int i = 0; i < 7; ++i) p.th[i] = policy->thresholds[i];
    p.d_base = policy->d_base;
    p.alpha = policy->alpha;
    p.n_default = policy->n_default;
    for (int i = 0; i < 3; ++i) p.gamma_pct[i] = policy->gamma_pct[i];
    p.counted = p.batch > 32;
    if (p.counted &&
        hs_launch(prune_count_kernel, dim3((p.batch + 3) / 4), dim3(128), 0, stream, ctx->pdl, dim3(1, 1, 1), p) != cudaSuccess)
        return HS_ERR_CUDA;
    return hs_launch(stratify_prune_kernel, dim3(p.batch), dim3(HS_MAX_NODES), 0, stream, ctx->pdl, dim3(1, 1, 1), p) ==
                   cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
