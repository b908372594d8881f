// hs_stratify_prune: one CTA of 128 threads per sequence, one thread per tree node.
//
// Entropy bin -> (d', N') (Sec. 4.2-4.3), Top-N' reranking by path confidence (Sec. 2.2), then the
// surviving nodes are compacted with warp ballots and a prefix sum over the four warps, parents are
// re-indexed and each kept node gets its ancestor-or-self bit mask (the tree-attention mask).
// The CSR offset of a sequence is the sum of the kept counts of all earlier sequences.  Small batches:
// every CTA recomputes those counts itself, so no CTA waits for another and the call is one launch.
// Larger batches: a first launch counts the kept nodes of every sequence once (one warp each), the
// second sums the counts ahead of its sequence (B integers instead of B trees per CTA).
//
// hs_entropy_quantify_prune launches tree_prune_kernel instead: the tree stage (path scores, Phi, P*) and the
// pruning of a sequence in one CTA; there the kept counts are handed from CTA to CTA (release / acquire flags).
#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"
#include "tree_stage.cuh"

struct PruneParams {
    int batch;
    const int* node_off;
    const int* parent;
    const float* score;
    const float* phi_star;
    const int* depth;
    const int* qstatus;
    hs_pruned_tree out;
    int counted;           // out.n_keep was filled by a launch ahead (prune_count_kernel or budget_kernel)
    const int* n_override; // [B] node counts that replace the policy's N' (budget reallocation), or NULL
    int* base;             // [B] budget path: policy request min(N', eligible), 0 for a flagged sequence
    int* room;             // [B] budget path: eligible nodes
    const int* slo_class;  // [B] budget path
    int budget;
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

// budget path, first launch: one warp per sequence, the policy's request and the eligible nodes
__global__ void __launch_bounds__(128) budget_request_kernel(const PruneParams p) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
    pdl_launch_dependents();
    pdl_wait();
    if (b >= p.batch) return;
    int base = 0, elig = 0;
    if (p.qstatus[b] == 0) {
        int bin, dp, np;
        policy_lookup(p, p.phi_star[b], bin, dp, np);
        const int lo = p.node_off[b], hi = min(p.node_off[b + 1], lo + HS_MAX_NODES);
        for (int i = lo + lane; i < hi; i += 32) elig += (p.depth[i] <= dp);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) elig += __shfl_xor_sync(HS_FULL_MASK, elig, o);
        elig = max(elig, 1);
        base = max(1, min(np, elig));
    }
    if (lane == 0) { p.base[b] = base; p.room[b] = elig; }
}

// budget path, second launch (one CTA): App. A.8 reading - if the requests fit the budget the left-over tokens go to
// the sequences in order of SLO class (stricter first, then sequence index), each up to its eligible nodes;
// otherwise the excess is taken back in the opposite order, never below the root.  The order is found by a
// bitonic sort of (class, index) keys in shared memory, the hand-out by a running sum along that order.
#define BUDGET_THREADS 1024
__global__ void __launch_bounds__(BUDGET_THREADS) budget_kernel(const PruneParams p) {
    __shared__ unsigned int s_key[HS_MAX_BATCH];
    __shared__ int s_amt[HS_MAX_BATCH];          // what the sequence at a sorted position may take (or give back)
    __shared__ int s_red[BUDGET_THREADS / 32];
    __shared__ int s_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    pdl_wait();
    const int B = p.batch;
    int P = 32;
    while (P < B) P <<= 1;
    int part = 0;
    for (int b = tid; b < B; b += BUDGET_THREADS) part += p.base[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(HS_FULL_MASK, part, o);
    if (lane == 0) s_red[warp] = part;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int w = 0; w < BUDGET_THREADS / 32; ++w) t += s_red[w];
        s_total = t;
    }
    __syncthreads();
    const int total = s_total;
    const bool fits = total <= p.budget;
    // keys: ascending = order of service; over budget the order is reversed (loosest class, highest index first)
    for (int i = tid; i < P; i += BUDGET_THREADS) {
        unsigned int k = 0xffffffffu;
        if (i < B) {
            const unsigned int cls = (unsigned int)min(max(p.slo_class[i], 0), 0xffff);
            k = (cls << 16) | (unsigned int)i;
            if (!fits) k = 0xfffffffeu - k;
        }
        s_key[i] = k;
    }
    __syncthreads();
    for (int k = 2; k <= P; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < P / 2; t += BUDGET_THREADS) {
                const int i = 2 * t - (t & (j - 1));
                const bool up = (i & k) == 0;
                const unsigned int a = s_key[i], c = s_key[i + j];
                if ((a > c) == up) { s_key[i] = c; s_key[i + j] = a; }
            }
            __syncthreads();
        }
    auto seq_of = [&](int pos) -> int {
        unsigned int k = s_key[pos];
        if (k == 0xffffffffu) return -1;
        if (!fits) k = 0xfffffffeu - k;
        return (int)(k & 0xffffu);
    };
    for (int pos = tid; pos < P; pos += BUDGET_THREADS) {
        const int b = seq_of(pos);
        int a = 0;
        if (b >= 0 && p.base[b] > 0) a = fits ? p.room[b] - p.base[b] : p.base[b] - 1;
        s_amt[pos] = a;
    }
    __syncthreads();
    // the amount still to hand out (or take back) when the walk reaches a position = pool - sum of the amounts ahead
    const int pool = fits ? p.budget - total : total - p.budget;
    const int per = (P + BUDGET_THREADS - 1) / BUDGET_THREADS;          // consecutive positions per thread
    int mine = 0;
    for (int q = 0; q < per; ++q) { const int pos = tid * per + q; if (pos < P) mine += s_amt[pos]; }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(HS_FULL_MASK, incl, o); if (lane >= o) incl += u; }
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    int before = incl - mine;
    for (int w = 0; w < warp; ++w) before += s_red[w];
    for (int q = 0; q < per; ++q) {
        const int pos = tid * per + q;
        if (pos >= P) break;
        const int b = seq_of(pos);
        const int take = max(0, min(s_amt[pos], pool - before));
        before += s_amt[pos];
        if (b >= 0) p.out.n_keep[b] = p.base[b] == 0 ? 0 : (fits ? p.base[b] + take : p.base[b] - take);
    }
}

struct PruneSmem {
    __align__(16) float S[HS_MAX_NODES];
    int nw[HS_MAX_NODES], par[HS_MAX_NODES];
    int warp[4];
    int off;
};

// Sum of `part` over the CTA's 128 threads, the same value in every thread.
__device__ __forceinline__ int cta_sum(int part, PruneSmem& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(HS_FULL_MASK, part, o);
    __syncthreads();                       // sm.warp may still be read
    if (lane == 0) sm.warp[warp] = part;
    __syncthreads();
    return sm.warp[0] + sm.warp[1] + sm.warp[2] + sm.warp[3];
}

// Reranking and compaction of sequence b by its CTA (thread t = node t with depth `dep`, parent `par`, ln V `S`):
// Top-N' among the nodes of depth <= d' by (S descending, index ascending), ballot + prefix compaction, parents
// re-indexed, ancestor-or-self masks.  `offset_of(n_keep)` returns where the sequence starts in the compacted arrays.
template <class OffsetFn>
__device__ __forceinline__ void prune_cta(const PruneParams& p, int b, int n, int status, float phi_star, int dep,
                                          int par, float S, PruneSmem& sm, OffsetFn offset_of) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int bin = 0, dp = 0, np = 0;
    policy_lookup(p, phi_star, bin, dp, np);
    const bool elig = tid < n && status == 0 && dep <= dp;
    // rank among eligible nodes by (S descending, index ascending): a node that is not eligible takes part as NaN,
    // which compares false both ways; four scores per shared-memory read
    sm.S[tid] = elig ? S : __int_as_float(0x7fc00000);
    sm.par[tid] = par;
    __syncthreads();
    int rank = 0;
    if (elig) {
        const float4* S4 = reinterpret_cast<const float4*>(sm.S);
        for (int j = 0; j < n; j += 4) {               // (entries past n belong to threads that are not eligible)
            const float4 v = S4[j >> 2];
            rank += (v.x > S || (v.x == S && j < tid)) + (v.y > S || (v.y == S && j + 1 < tid)) +
                    (v.z > S || (v.z == S && j + 2 < tid)) + (v.w > S || (v.w == S && j + 3 < tid));
        }
    }
    const bool keep = elig && rank < (p.n_override ? p.n_override[b] : np);
    // compaction: ballot inside the warp, prefix over the four warps
    const unsigned int bal = __ballot_sync(HS_FULL_MASK, keep);
    if (lane == 0) sm.warp[warp] = __popc(bal);
    __syncthreads();
    int before = __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) before += sm.warp[w];
    const int n_keep = sm.warp[0] + sm.warp[1] + sm.warp[2] + sm.warp[3];
    sm.nw[tid] = keep ? before : -1;
    const int off = offset_of(n_keep);
    __syncthreads();                       // sm.nw is complete
    if (keep) {
        const int k = off + before;
        unsigned long long m0 = 0ull, m1 = 0ull;
        int a = tid;
        for (int step = 0; step <= HS_MAX_NODES && a >= 0; ++step) {   // walk to the root
            int na = sm.nw[a];
            if (na >= 0) {
                if (na < 64) m0 |= 1ull << na; else m1 |= 1ull << (na - 64);
            }
            a = sm.par[a];
        }
        p.out.keep_idx[k] = tid;
        p.out.new_parent[k] = par >= 0 ? sm.nw[par] : -1;
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

__global__ void __launch_bounds__(HS_MAX_NODES) stratify_prune_kernel(const PruneParams p) {
    __shared__ PruneSmem sm;
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();                            // scores and Phi(P*) come from the kernel ahead in the stream
    const int base = p.node_off[b];
    const int n = min(p.node_off[b + 1] - base, HS_MAX_NODES);
    const int status = p.qstatus[b];
    int dep = 0, par = -1;
    float S = 0.f;
    if (tid < n && status == 0) {
        dep = p.depth[base + tid];
        par = p.parent[base + tid];
        S = p.score[base + tid];
    }
    prune_cta(p, b, n, status, p.phi_star[b], dep, par, S, sm, [&](int) {
        // offset of this sequence in the compacted arrays: the kept counts of the sequences ahead
        int part = 0;
        if (p.counted) {
            for (int bb = tid; bb < b; bb += HS_MAX_NODES) part += p.out.n_keep[bb];
        } else {
            for (int bb = tid; bb < b; bb += HS_MAX_NODES) part += kept_count(p, bb);
        }
        return cta_sum(part, sm);
    });
}

// ---- tree stage and pruning in one launch ---------------------------------------------------------------------
struct TreePruneParams {
    // the tree stage's view (the names tree_stage_cta expects)
    const void* logits;
    int64_t row_stride;
    int vocab, is_bf16, prefetch;
    const int* node_off;
    const int* parent;
    const int* token;
    hs_quant_out out;
    int d_base, phi_mode, pstar_mode, entropy_mode;
    PruneParams pr;
    int* flags;       // [B] kept count + 1 of a sequence once its CTA knows it (zero between launches)
    int* done;        // CTAs that have read the counts ahead of theirs
    int* err;         // sticky device error word (a bounded wait that expired)
};

// One CTA per sequence: the tree stage, then - from shared memory and registers, without a round trip through the
// quantify outputs - bin, d', N', reranking, compaction and masks.  The offset of a sequence in the compacted arrays
// needs the kept counts of the sequences ahead, which other CTAs of this launch compute: every CTA publishes its
// count (release) and reads the counts ahead of it (acquire, bounded wait).  CTAs are started in index order and a
// CTA only waits for lower indices, so a waiting CTA never keeps the one it waits for from starting.  The CTA that
// is last to finish its reads puts flags and counter back to zero.
__global__ void __launch_bounds__(HS_MAX_NODES) tree_prune_kernel(const __grid_constant__ TreePruneParams p) {
    __shared__ TreeStageSmem tsm;
    __shared__ PruneSmem sm;
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    pdl_launch_dependents();
    const TreeStageResult t = tree_stage_cta(p, b, tsm);
    __syncthreads();                                   // tsm.phi_star
    const int n = min(max(t.n, 0), HS_MAX_NODES);
    const int status = t.bad ? HS_ERR_BAD_TREE : HS_OK;
    prune_cta(p.pr, b, n, status, t.bad ? 0.f : tsm.phi_star, t.dep, t.bad ? -1 : t.par, t.S, sm, [&](int n_keep) {
        if (p.pr.batch == 1) return 0;
        if (tid == 0) st_release_gpu(&p.flags[b], n_keep + 1);
        int part = 0;
        const unsigned long long t0 = global_timer_ns();
        for (int bb = tid; bb < b; bb += HS_MAX_NODES) {
            int v = ld_acquire_gpu(&p.flags[bb]);
            while (v == 0) {
                if (global_timer_ns() - t0 > 2000000000ull) { atomicExch(p.err, HS_ERR_TIMEOUT); v = 1; break; }
                __nanosleep(64);
                v = ld_acquire_gpu(&p.flags[bb]);
            }
            part += v - 1;
        }
        const int off = cta_sum(part, sm);             // (its barriers order every thread's reads before the arrival)
        if (tid == 0) {
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.done) : "memory");
            if (old == p.pr.batch - 1) {               // every CTA has read what it needs
                for (int bb = 0; bb < p.pr.batch; ++bb) p.flags[bb] = 0;
                *p.done = 0;
            }
        }
        return off;
    });
}

hs_status hs_launch_tree_prune(hs_ctx* ctx, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                               int64_t row_stride, int32_t vocab, const hs_policy* policy, const hs_quant_out* quant,
                               const hs_pruned_tree* out, cudaStream_t stream) {
    TreePruneParams p;
    p.logits = logits;
    p.row_stride = row_stride;
    p.vocab = vocab;
    p.is_bf16 = dtype == HS_BF16;
    p.prefetch = (ctx->prefetch & HS_PREFETCH_LOGITS) != 0;
    p.node_off = tree->node_off;
    p.parent = tree->parent;
    p.token = tree->token;
    p.out = *quant;
    p.d_base = policy->d_base;
    p.phi_mode = policy->phi_mode;
    p.pstar_mode = policy->pstar_mode;
    p.entropy_mode = policy->entropy_mode;
    PruneParams& q = p.pr;
    q.batch = tree->batch;
    q.node_off = tree->node_off;
    q.parent = tree->parent;
    q.score = quant->score;
    q.phi_star = quant->phi_star;
    q.depth = quant->depth;
    q.qstatus = quant->status;
    q.out = *out;
    for (int i = 0; i < 7; ++i) q.th[i] = policy->thresholds[i];
    q.d_base = policy->d_base;
    q.alpha = policy->alpha;
    q.n_default = policy->n_default;
    for (int i = 0; i < 3; ++i) q.gamma_pct[i] = policy->gamma_pct[i];
    q.n_override = nullptr; q.base = nullptr; q.room = nullptr; q.slo_class = nullptr; q.budget = 0;
    q.counted = 0;
    p.flags = ctx->counters + HS_CNT_PRUNE_FLAG;
    p.done = ctx->counters + HS_CNT_PRUNE_DONE;
    p.err = ctx->counters + HS_CNT_ERROR;
    return hs_launch(tree_prune_kernel, dim3(q.batch), dim3(HS_MAX_NODES), 0, stream, ctx->pdl, dim3(1, 1, 1), p) ==
                   cudaSuccess ? HS_OK : HS_ERR_CUDA;
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
    p.n_override = nullptr; p.base = nullptr; p.room = nullptr; p.slo_class = nullptr; p.budget = 0;
    p.counted = p.batch > 32;
    if (p.counted &&
        hs_launch(prune_count_kernel, dim3((p.batch + 3) / 4), dim3(128), 0, stream, ctx->pdl, dim3(1, 1, 1), p) != cudaSuccess)
        return HS_ERR_CUDA;
    return hs_launch(stratify_prune_kernel, dim3(p.batch), dim3(HS_MAX_NODES), 0, stream, ctx->pdl, dim3(1, 1, 1), p) ==
                   cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

// Sec. 4.2-4.3 with the token budget of App. A.8: request -> reallocation -> Top-N reranking with the reallocated counts.
hs_status hs_launch_stratify_prune_budget(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                          const hs_policy* policy, const int32_t* slo_class, int32_t budget,
                                          const hs_pruned_tree* out, cudaStream_t stream) {
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
    if ((size_t)2 * p.batch * sizeof(int) > ctx->scratch_bytes) return HS_ERR_WORKSPACE;
    p.base = (int*)ctx->scratch;
    p.room = p.base + p.batch;
    p.slo_class = slo_class;
    p.budget = budget;
    p.counted = 1;
    p.n_override = out->n_keep;
    if (hs_launch(budget_request_kernel, dim3((p.batch + 3) / 4), dim3(128), 0, stream, ctx->pdl, dim3(1, 1, 1), p) != cudaSuccess ||
        hs_launch(budget_kernel, dim3(1), dim3(BUDGET_THREADS), 0, stream, ctx->pdl, dim3(1, 1, 1), p) != cudaSuccess)
        return HS_ERR_CUDA;
    return hs_launch(stratify_prune_kernel, dim3(p.batch), dim3(HS_MAX_NODES), 0, stream, ctx->pdl, dim3(1, 1, 1), p) ==
                   cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
