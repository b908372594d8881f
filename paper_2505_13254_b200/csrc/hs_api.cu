// C-ABI entry points: context, argument validation, dispatch to the kernel launchers.
#include <stdlib.h>

#include <new>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

extern "C" const char* hs_status_string(hs_status s) {
    switch (s) {
        case HS_OK: return "ok";
        case HS_ERR_INVALID_ARG: return "invalid argument";
        case HS_ERR_SHAPE: return "unsupported shape";
        case HS_ERR_UNSUPPORTED: return "unsupported";
        case HS_ERR_WORKSPACE: return "workspace too small";
        case HS_ERR_CUDA: return "CUDA error";
        case HS_ERR_TIMEOUT: return "device-side wait expired";
        case HS_ERR_BAD_TREE: return "malformed tree";
        case HS_ERR_STATIC_LIMIT: return "batch exceeds the built-in scratch of the allocation-free entry point";
    }
    return "unknown status";
}

extern "C" size_t hs_workspace_bytes(int32_t max_batch, int32_t max_rows, int32_t vocab, int32_t hq, int32_t hkv) {
    if (max_batch < 1 || max_rows < 1 || vocab < 1 || hq < 1 || hkv < 1) return 0;
    size_t chunks = hs_row_chunks(vocab, HS_F32);
    // entropy pass: two partials per CTA, at most one CTA per SM (room for 1024)
    size_t quant = (size_t)2 * 1024 * HS_ROW_PARTIAL_BYTES + 256;
    // acceptance: three per-row result arrays (256-byte aligned each) + chunk partials of target and draft rows
    size_t accept = 3 * hs_align_up((size_t)max_rows * 8, 256) +
                    (size_t)2 * max_rows * chunks * HS_ACC_PARTIAL_BYTES;
    // (the attention merges its KV splits on chip: no workspace)
    size_t scratch = quant > accept ? quant : accept;
    return HS_COUNTER_BYTES + hs_align_up(scratch, 256) + 256;
}

extern "C" hs_status hs_create(hs_ctx** out, int32_t device, size_t workspace_bytes) {
    if (!out) return HS_ERR_INVALID_ARG;
    *out = nullptr;
    if (workspace_bytes < HS_COUNTER_BYTES + 256) return HS_ERR_WORKSPACE;
    int ndev = 0;
    HS_CUDA_OK(cudaGetDeviceCount(&ndev));
    if (device < 0 || device >= ndev) return HS_ERR_INVALID_ARG;
    HS_CUDA_OK(cudaSetDevice(device));
    int sm_count = 0, major = 0;
    HS_CUDA_OK(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device));
    HS_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    if (major != 10) return HS_ERR_UNSUPPORTED;                   // built for sm_100a only
    hs_ctx* c = new (std::nothrow) hs_ctx();
    if (!c) return HS_ERR_INVALID_ARG;
    c->device = device;
    c->sm_count = sm_count;
    void* p = nullptr;
    if (cudaMalloc(&p, workspace_bytes) != cudaSuccess) { delete c; return HS_ERR_CUDA; }
    c->ws = (char*)p;
    c->ws_bytes = workspace_bytes;
    c->counters = (int*)p;
    c->n_counters = HS_COUNTER_BYTES / sizeof(int);
    c->scratch = c->ws + HS_COUNTER_BYTES;
    c->scratch_bytes = workspace_bytes - HS_COUNTER_BYTES;
    if (cudaMemset(p, 0, HS_COUNTER_BYTES) != cudaSuccess) { cudaFree(p); delete c; return HS_ERR_CUDA; }
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(p); delete c; return HS_ERR_CUDA;
    }
    c->encode_tiled = fn;
    const char* no_pdl = getenv("HS_DISABLE_PDL");
    c->pdl = !(no_pdl && no_pdl[0] == '1');
    c->prefetch = 0;
    c->row_pass = HS_ROW_PASS_AUTO;
    c->attn_ready = false;
    c->walk_ready = false;
    c->quant_ready = false;
    c->rows_ready = false;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaFree(p); delete c; return HS_ERR_CUDA; }
    *out = c;
    return HS_OK;
}

extern "C" hs_status hs_destroy(hs_ctx* ctx) {
    if (!ctx) return HS_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    cudaFree(ctx->ws);
    delete ctx;
    return HS_OK;
}

// One thread waits on a barrier that nothing ever completes; the bounded wait gives up after limit_ns and
// records HS_ERR_TIMEOUT in the context's error word.
__global__ void wait_selftest_kernel(int* err, unsigned long long limit_ns) {
    __shared__ unsigned long long s_bar;
    const unsigned int bar = smem_u32(&s_bar);
    mbar_init(bar, 1);
    mbar_init_fence();
    mbar_wait_limit(bar, 0u, err, limit_ns);
}

hs_status hs_launch_wait_selftest(hs_ctx* ctx, uint64_t limit_ns, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 1, 0, stream>>>(ctx->counters + HS_CNT_ERROR, (unsigned long long)limit_ns);
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

extern "C" hs_status hs_set_prefetch(hs_ctx* ctx, int32_t flags) {
    if (!ctx || (flags & ~(HS_PREFETCH_LOGITS | HS_PREFETCH_KV))) return HS_ERR_INVALID_ARG;
    ctx->prefetch = flags;
    return HS_OK;
}

extern "C" hs_status hs_set_row_pass(hs_ctx* ctx, int32_t variant) {
    if (!ctx || variant < HS_ROW_PASS_AUTO || variant > HS_ROW_PASS_STREAM) return HS_ERR_INVALID_ARG;
    ctx->row_pass = variant;
    return HS_OK;
}

extern "C" hs_status hs_selftest_wait_timeout(hs_ctx* ctx, uint64_t limit_ns, hs_stream stream) {
    if (!ctx || !hs_on_device(ctx)) return HS_ERR_INVALID_ARG;
    if (limit_ns < 1000ull) limit_ns = 1000ull;
    if (limit_ns > 10000000ull) limit_ns = 10000000ull;
    return hs_launch_wait_selftest(ctx, limit_ns, (cudaStream_t)stream);
}

extern "C" hs_status hs_device_error(hs_ctx* ctx, int32_t* host_out) {
    if (!ctx || !host_out) return HS_ERR_INVALID_ARG;
    HS_CUDA_OK(cudaSetDevice(ctx->device));
    HS_CUDA_OK(cudaDeviceSynchronize());
    int v = 0;
    HS_CUDA_OK(cudaMemcpy(&v, ctx->counters + HS_CNT_ERROR, sizeof(int), cudaMemcpyDeviceToHost));
    if (v != 0) HS_CUDA_OK(cudaMemset(ctx->counters + HS_CNT_ERROR, 0, sizeof(int)));
    *host_out = v;
    return HS_OK;
}

static bool tree_ok(const hs_tree_batch* t) {
    return t && t->batch >= 1 && t->batch <= HS_MAX_BATCH && t->n_nodes_total >= t->batch &&
           t->n_nodes_total <= HS_MAX_ROWS && t->node_off && t->parent && t->token;
}
static bool policy_ok(const hs_policy* p) {
    if (!p || p->top_k < 1 || p->top_k > HS_MAX_TOPK || p->d_base < 0 || p->n_default < 1) return false;
    for (int i = 0; i + 1 < 7; ++i)
        if (!(p->thresholds[i] <= p->thresholds[i + 1])) return false;
    for (int i = 0; i < 3; ++i)
        if (p->gamma_pct[i] < 0) return false;
    return p->phi_mode >= 0 && p->phi_mode <= 1 && p->pstar_mode >= 0 && p->pstar_mode <= 1 &&
           p->entropy_mode >= 0 && p->entropy_mode <= 1;
}
static bool logits_ok(const void* p, hs_dtype dtype, int64_t row_stride, int32_t vocab) {
    if (!p || ((uintptr_t)p & 15)) return false;
    if (dtype != HS_F32 && dtype != HS_BF16) return false;
    int vec = dtype == HS_BF16 ? 8 : 4;
    return vocab >= 1 && row_stride >= vocab && row_stride % vec == 0;
}

extern "C" hs_status hs_entropy_quantify(hs_ctx* ctx, const hs_tree_batch* tree, const void* draft_logits,
                                         hs_dtype dtype, int64_t row_stride, int32_t vocab,
                                         const hs_policy* policy, const hs_quant_out* out, hs_stream stream) {
    if (!ctx || !out || !hs_on_device(ctx)) return HS_ERR_INVALID_ARG;
    if (!tree_ok(tree) || !policy_ok(policy) || !logits_ok(draft_logits, dtype, row_stride, vocab))
        return HS_ERR_INVALID_ARG;
    if (!out->row_max || !out->row_lse || !out->h_full || !out->i_topk || !out->i_trunc || !out->topk_val ||
        !out->topk_idx || !out->logc || !out->score || !out->phi || !out->depth || !out->pstar_node ||
        !out->phi_star || !out->status)
        return HS_ERR_INVALID_ARG;
    return hs_launch_quantify(ctx, tree, draft_logits, dtype, row_stride, vocab, policy, out, (cudaStream_t)stream);
}

static bool pruned_out_ok(const hs_pruned_tree* out) {
    return out && out->bin && out->d_prime && out->n_prime && out->n_keep && out->keep_off && out->keep_idx &&
           out->new_parent && out->new_depth && out->keep_rank && out->anc_mask && out->status;
}

extern "C" hs_status hs_entropy_quantify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const void* draft_logits,
                                               hs_dtype dtype, int64_t row_stride, int32_t vocab,
                                               const hs_policy* policy, const hs_quant_out* quant,
                                               const hs_pruned_tree* pruned, hs_stream stream) {
    if (!ctx || !quant || !hs_on_device(ctx)) return HS_ERR_INVALID_ARG;
    if (!tree_ok(tree) || !policy_ok(policy) || !logits_ok(draft_logits, dtype, row_stride, vocab))
        return HS_ERR_INVALID_ARG;
    if (!quant->row_max || !quant->row_lse || !quant->h_full || !quant->i_topk || !quant->i_trunc || !quant->topk_val ||
        !quant->topk_idx || !quant->logc || !quant->score || !quant->phi || !quant->depth || !quant->pstar_node ||
        !quant->phi_star || !quant->status || !pruned_out_ok(pruned))
        return HS_ERR_INVALID_ARG;
    hs_status st = hs_launch_quantify(ctx, tree, draft_logits, dtype, row_stride, vocab, policy, quant,
                                      (cudaStream_t)stream, false);
    if (st != HS_OK) return st;
    return hs_launch_tree_prune(ctx, tree, draft_logits, dtype, row_stride, vocab, policy, quant, pruned,
                                (cudaStream_t)stream);
}

extern "C" hs_status hs_stratify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                       const hs_policy* policy, const hs_pruned_tree* out, hs_stream stream) {
    if (!ctx || !quant || !out || !hs_on_device(ctx)) return HS_ERR_INVALID_ARG;
    if (!tree_ok(tree) || !policy_ok(policy)) return HS_ERR_INVALID_ARG;
    if (!quant->score || !quant->phi_star || !quant->depth || !quant->status) return HS_ERR_INVALID_ARG;
    if (!out->bin || !out->d_prime || !out->n_prime || !out->n_keep || !out->keep_off || !out->keep_idx ||
        !out->new_parent || !out->new_depth || !out->keep_rank || !out->anc_mask || !out->status)
        return HS_ERR_INVALID_ARG;
    return hs_launch_stratify_prune(ctx, tree, quant, policy, out, (cudaStream_t)stream);
}

extern "C" hs_status hs_stratify_prune_budget(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                              const hs_policy* policy, const int32_t* slo_class, int32_t budget,
                                              const hs_pruned_tree* out, hs_stream stream) {
    if (!ctx || !quant || !out || !slo_class || budget < 0 || !hs_on_device(ctx)) return HS_ERR_INVALID_ARG;
    if (!tree_ok(tree) || !policy_ok(policy)) return HS_ERR_INVALID_ARG;
    if (!quant->score || !quant->phi_star || !quant->depth || !quant->status) return HS_ERR_INVALID_ARG;
    if (!out->bin || !out->d_prime || !out->n_prime || !out->n_keep || !out->keep_off || !out->keep_idx ||
        !out->new_parent || !out->new_depth || !out->keep_rank || !out->anc_mask || !out->status)
        return HS_ERR_INVALID_ARG;
    return hs_launch_stratify_prune_budget(ctx, tree, quant, policy, slo_class, budget, out, (cudaStream_t)stream);
}

static bool pruned_ok(const hs_pruned_tree* p) {
    return p && p->n_keep && p->keep_off && p->keep_idx && p->new_parent && p->new_depth && p->keep_rank &&
           p->anc_mask && p->status;
}

extern "C" hs_status hs_tree_verify_attention(hs_ctx* ctx, const hs_pruned_tree* pruned, const hs_attn_desc* d,
                                              const void* q, const void* k_tree, const void* v_tree,
                                              const void* k_cache, const void* v_cache, void* out,
                                              float* lse_out, hs_stream stream) {
    if (!ctx || !d || !pruned_ok(pruned) || !q || !k_tree || !v_tree || !out || !hs_on_device(ctx))
        return HS_ERR_INVALID_ARG;
    if (d->batch < 1 || d->batch > HS_MAX_BATCH || d->max_rows < 1 || d->max_rows > HS_MAX_ROWS ||
        d->max_nodes < 1 || d->max_nodes > HS_MAX_NODES || d->kv_total < 0 || d->max_kv_len < 0 ||
        d->max_kv_len > d->kv_total || !d->kv_off)
        return HS_ERR_INVALID_ARG;
    if (d->kv_total > 0 && (!k_cache || !v_cache)) return HS_ERR_INVALID_ARG;
    if (d->layout != HS_ROWS_COMPACT && d->layout != HS_ROWS_ORIGINAL) return HS_ERR_INVALID_ARG;
    if (d->layout == HS_ROWS_ORIGINAL && !d->node_off) return HS_ERR_INVALID_ARG;
    if (d->head_dim != HS_HEAD_DIM || d->hq < 1 || d->hkv < 1 || d->hq % d->hkv != 0 || d->hq / d->hkv > 16)
        return HS_ERR_SHAPE;
    if (d->kv_total > 0 && (d->kv_token_stride % 8 != 0 || d->kv_head_stride % 8 != 0 ||
                            d->kv_token_stride < HS_HEAD_DIM || d->kv_head_stride < HS_HEAD_DIM))
        return HS_ERR_SHAPE;
    if (((uintptr_t)q | (uintptr_t)k_tree | (uintptr_t)v_tree | (uintptr_t)k_cache | (uintptr_t)v_cache |
         (uintptr_t)out) & 15)
        return HS_ERR_INVALID_ARG;
    return hs_launch_attention(ctx, pruned, d, q, k_tree, v_tree, k_cache, v_cache, out, lse_out,
                               (cudaStream_t)stream);
}

extern "C" hs_status hs_accept_path(hs_ctx* ctx, const hs_tree_batch* tree, const hs_pruned_tree* pruned,
                                    const void* target_logits, int32_t target_layout, const void* draft_logits,
                                    hs_dtype dtype, int64_t row_stride, int32_t vocab, const int32_t* mode,
                                    const float* temperature, uint64_t seed, uint64_t offset,
                                    const float* uniforms, const hs_accept_out* out, hs_stream stream) {
    if (!ctx || !out || !mode || !temperature || !hs_on_device(ctx) || (offset >> 63)) return HS_ERR_INVALID_ARG;
    if (!tree_ok(tree) || !pruned_ok(pruned) || !logits_ok(target_logits, dtype, row_stride, vocab))
        return HS_ERR_INVALID_ARG;
    if (draft_logits && ((uintptr_t)draft_logits & 15)) return HS_ERR_INVALID_ARG;
    if (target_layout != HS_ROWS_COMPACT && target_layout != HS_ROWS_ORIGINAL) return HS_ERR_INVALID_ARG;
    if (!out->accept_len || !out->path_nodes || !out->path_compact || !out->path_tokens || !out->bonus_token ||
        !out->terminal_rank || !out->status || out->path_cap < 2)
        return HS_ERR_INVALID_ARG;
    return hs_launch_accept(ctx, tree, pruned, target_logits, target_layout, draft_logits, dtype, row_stride,
                            vocab, mode, temperature, seed, offset, uniforms, out, (cudaStream_t)stream);
}

extern "C" hs_status hs_philox_uniforms(hs_ctx* ctx, uint64_t seed, uint64_t offset, const int32_t* b,
                                        const int32_t* node, const int32_t* stream_id, int32_t count,
                                        float* out, hs_stream stream) {
    if (!ctx || !b || !node || !stream_id || !out || count < 0 || !hs_on_device(ctx) || (offset >> 63))
        return HS_ERR_INVALID_ARG;
    if (count == 0) return HS_OK;
    return hs_launch_philox(seed, offset, b, node, stream_id, count, out, (cudaStream_t)stream);
}
