// Shared device/host helpers of the verification kernels (sm_100a only).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/heterospec.h"

#define HS_WARP 32
#define HS_FULL_MASK 0xffffffffu

// Context: one device, one workspace carved into fixed regions at hs_create.
struct hs_ctx {
    int device;
    int sm_count;
    size_t ws_bytes;
    char* ws;           // device workspace
    int* counters;      // device: self-resetting arrival counters (zeroed at create)
    size_t n_counters;
    char* scratch;      // device: partials region (everything after the counters)
    size_t scratch_bytes;
    void* encode_tiled; // cuTensorMapEncodeTiled entry point
    bool pdl;           // launch kernels with programmatic stream serialisation
    int row_pass;       // HS_ROW_PASS_*: kernel of the acceptance row pass
    int prefetch;       // HS_PREFETCH_* bits: inputs a kernel may fetch before its dependency wait
    bool attn_ready;    // attention kernel attributes set and cluster capacities queried on this device
    int attn_cap[9];    // CTAs of the attention kernel that run at once in clusters of s = 1..8
    bool walk_ready;    // acceptance walk kernel attributes set on this device
    bool rows_ready;    // streaming acceptance row pass: shared-memory attribute set on this device
    bool quant_ready;   // streaming entropy kernel: shared-memory attribute set on this device
};

// The context's device must be the calling thread's current device (launches go to the current device).
static inline bool hs_on_device(const hs_ctx* ctx) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == ctx->device;
}

// Kernel launch with optional programmatic-dependent-launch attribute and thread-block cluster shape.
template <typename... KArgs, typename... Args>
static inline cudaError_t hs_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t stream, bool pdl, dim3 cluster, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (cluster.x * cluster.y * cluster.z > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = cluster.x;
        attr[na].val.clusterDim.y = cluster.y;
        attr[na].val.clusterDim.z = cluster.z;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

#define HS_CUDA_OK(call)                                   \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return HS_ERR_CUDA;        \
    } while (0)

static inline size_t hs_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- warp helpers --------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(HS_FULL_MASK, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(HS_FULL_MASK, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(HS_FULL_MASK, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long w = __shfl_xor_sync(HS_FULL_MASK, v, o);
        v = w > v ? w : v;
    }
    return v;
}

// Order-preserving key: larger logit first, then lower index.  key(a) > key(b) iff a ranks
// before b in (value descending, index ascending).
__device__ __forceinline__ unsigned int float_order_bits(float f) {
    unsigned int u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float order_bits_float(unsigned int b) {
    unsigned int u = (b & 0x80000000u) ? (b & 0x7fffffffu) : ~b;
    return __uint_as_float(u);
}
__device__ __forceinline__ unsigned long long make_key(float v, int idx) {
    return ((unsigned long long)float_order_bits(v) << 32) | (unsigned int)(~(unsigned int)idx);
}
__device__ __forceinline__ float key_value(unsigned long long k) { return order_bits_float((unsigned int)(k >> 32)); }
__device__ __forceinline__ int key_index(unsigned long long k) { return (int)(~(unsigned int)(k & 0xffffffffu)); }

// bf16 pair (packed in 32 bits) -> two floats, exact
__device__ __forceinline__ float bf16_lo(unsigned int p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(unsigned int p) { return __uint_as_float(p & 0xffff0000u); }

// loads that bypass L1 (values written by other CTAs of the same launch)
__device__ __forceinline__ float ld_cg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ int ld_cg_i(const int* p) { return __ldcg(p); }

// Row of the logits / attention arrays that holds kept node i of sequence b.
__device__ __forceinline__ int kept_row(int layout, const int* node_off, const int* keep_off,
                                        const int* keep_idx, int b, int i) {
    int k = keep_off[b] + i;
    return layout == HS_ROWS_ORIGINAL ? node_off[b] + keep_idx[k] : k;
}

// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0,k1) -> first output word.
__device__ __forceinline__ unsigned int philox4x32_10_x0(unsigned int c0, unsigned int c1, unsigned int c2,
                                                         unsigned int c3, unsigned int k0, unsigned int k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        unsigned int hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        unsigned int hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        unsigned int n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}
__device__ __forceinline__ float philox_uniform(unsigned long long seed, unsigned long long offset, int b,
                                                int node, int stream_id) {
    // counter = (offset low word, b, node, stream + 2 * offset high word), key = seed
    unsigned int x0 = philox4x32_10_x0((unsigned int)offset, (unsigned int)b, (unsigned int)node,
                                       (unsigned int)stream_id + 2u * (unsigned int)(offset >> 32),
                                       (unsigned int)seed, (unsigned int)(seed >> 32));
    return (float)(x0 >> 8) * 5.9604644775390625e-8f;  // 2^-24
}

// ---- launchers implemented in the kernel files ---------------------------------------------
hs_status hs_launch_quantify(hs_ctx* ctx, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                             int64_t row_stride, int32_t vocab, const hs_policy* policy,
                             const hs_quant_out* out, cudaStream_t stream, bool with_tree_stage = true);
hs_status hs_launch_tree_prune(hs_ctx* ctx, const hs_tree_batch* tree, const void* logits, hs_dtype dtype,
                               int64_t row_stride, int32_t vocab, const hs_policy* policy, const hs_quant_out* quant,
                               const hs_pruned_tree* out, cudaStream_t stream);
hs_status hs_launch_stratify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                   const hs_policy* policy, const hs_pruned_tree* out, cudaStream_t stream);
hs_status hs_launch_stratify_prune_budget(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                          const hs_policy* policy, const int32_t* slo_class, int32_t budget,
                                          const hs_pruned_tree* out, cudaStream_t stream);
hs_status hs_launch_attention(hs_ctx* ctx, const hs_pruned_tree* pruned, const hs_attn_desc* desc,
                              const void* q, const void* k_tree, const void* v_tree, const void* k_cache,
                              const void* v_cache, void* out, float* lse_out, cudaStream_t stream);
hs_status hs_launch_accept(hs_ctx* ctx, const hs_tree_batch* tree, const hs_pruned_tree* pruned,
                           const void* target_logits, int32_t target_layout, const void* draft_logits,
                           hs_dtype dtype, int64_t row_stride, int32_t vocab, const int32_t* mode,
                           const float* temperature, uint64_t seed, uint64_t offset, const float* uniforms,
                           const hs_accept_out* out, cudaStream_t stream);
hs_status hs_launch_wait_selftest(hs_ctx* ctx, uint64_t limit_ns, cudaStream_t stream);
hs_status hs_launch_philox(uint64_t seed, uint64_t offset, const int32_t* b, const int32_t* node,
                           const int32_t* stream_id, int32_t count, float* out, cudaStream_t stream);
