// hs_tree_verify_attention (Sec. 2.2, tree-mask attention).
//
// tree_attn_split_kernel  CTA = (block of 128 query rows, KV split, sequence x kv-head).  The GQA group
//     times the kept tree nodes forms the dense M dimension: query row r = node * G + g.  KV prefix
//     tiles of 64 keys are brought into 128-byte-swizzled shared memory by TMA (cp.async.bulk.tensor,
//     double buffered, mbarrier completion); the <= 128 tree keys are gathered with plain loads
//     because their rows may be indirect.  S = Q K^T and O += P V run on the tensor cores with fp32
//     accumulation; the softmax is the online (running max / running sum) form in base 2.  Prefix
//     columns are fully visible, tree column j is visible to row r iff bit j of the ancestor mask
//     of r's node is set.
// tree_attn_combine_kernel  merges the per-split (max, sum, O) partials of a row into the bf16 output.
#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"

#define ATT_THREADS 256
#define ATT_BM 128
#define ATT_BN 64
#define ATT_TILE_BYTES (ATT_BN * HS_HEAD_DIM * 2)   // 16 KiB: one K or V tile
#define ATT_STAGE_BYTES (2 * ATT_TILE_BYTES)
#define ATT_SMEM_BYTES (2 * ATT_STAGE_BYTES + 1024 + 64)
#define ATT_WAIT_LIMIT (1 << 24)
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
    int batch, hq, hkv, G, layout, nsplit, mpad, head_first;
    float scale_log2;
    float* part_o;      // [pair][split][mpad][128]
    float2* part_ml;    // [pair][split][mpad] {running max (base 2), running sum}
    int* err;
};

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ unsigned int smem_u32(const void* p) { return (unsigned int)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned int bar, unsigned int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned int bar, unsigned int bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned int bar, unsigned int parity) {
    unsigned int ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after ATT_WAIT_LIMIT polls and records HS_ERR_TIMEOUT; never spins forever.
__device__ __forceinline__ void mbar_wait(unsigned int bar, unsigned int parity, int* err) {
    for (int i = 0; i < ATT_WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return;
    atomicExch(err, (int)HS_ERR_TIMEOUT);
}
__device__ __forceinline__ void tma_load_3d(unsigned int dst, const CUtensorMap* tm, int c0, int c1, int c2,
                                            unsigned int bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4(unsigned int addr, unsigned int& r0, unsigned int& r1, unsigned int& r2,
                                        unsigned int& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(unsigned int addr, unsigned int& r0, unsigned int& r1, unsigned int& r2,
                                          unsigned int& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const unsigned int* a, unsigned int b0, unsigned int b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ unsigned int pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned int*>(&v);
}
// byte offset of (key row, 16-byte chunk 0..15 of the 128 d's) inside a swizzled 64x128 bf16 tile
__device__ __forceinline__ unsigned int tile_off(int key, int chunk) {
    return (unsigned int)((chunk >> 3) * (ATT_TILE_BYTES / 2) + key * 128 + (((chunk & 7) ^ (key & 7)) << 4));
}

// tiles of a sequence and the share of one split; identical in both kernels
__device__ __forceinline__ void split_range(int L, int nk, int nsplit, int split, int& t_prefix, int& t_total,
                                            int& t0, int& t1) {
    t_prefix = (L + ATT_BN - 1) / ATT_BN;
    t_total = t_prefix + (nk + ATT_BN - 1) / ATT_BN;
    int per = (t_total + nsplit - 1) / nsplit;
    t0 = min(split * per, t_total);
    t1 = min(t0 + per, t_total);
}

__global__ void __launch_bounds__(ATT_THREADS, 1)
tree_attn_split_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair = blockIdx.z, b = pair / p.hkv, h = pair % p.hkv;
    const int split = blockIdx.y;
    const int nk = (p.status[b] == 0) ? p.n_keep[b] : 0;
    const int M = nk * p.G;
    const int m0 = blockIdx.x * ATT_BM;
    if (m0 >= M) return;
    const int koff = p.keep_off[b];
    const int kv0 = p.kv_off[b];
    const int L = p.kv_off[b + 1] - kv0;
    int t_prefix, t_total, t0, t1;
    split_range(L, nk, p.nsplit, split, t_prefix, t_total, t0, t1);
    if (t0 >= t1) return;

    const unsigned int smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const unsigned int bar0 = smem_base + 2 * ATT_STAGE_BYTES;
    unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // ---- query fragments (A operand, 16 rows x 128 d per warp) straight from global memory --------
    const int gid = lane >> 2, qd = (lane & 3) * 2;
    const int r0 = m0 + warp * 16 + gid, r1 = r0 + 8;
    unsigned int qf[8][4];
    unsigned long long mk[2][2] = {{0ull, 0ull}, {0ull, 0ull}};
    int orow[2] = {-1, -1};           // output row (token row * hq + head) of r0 / r1, -1 = padding
    {
        const int rr[2] = {r0, r1};
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const int r = rr[x];
            const unsigned int* src = nullptr;
            if (r < M) {
                const int node = r / p.G, g = r % p.G;
                const int trow = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + node] : koff + node;
                orow[x] = trow * p.hq + h * p.G + g;
                src = reinterpret_cast<const unsigned int*>(p.q + (size_t)orow[x] * HS_HEAD_DIM);
                mk[x][0] = p.anc_mask[2 * (size_t)(koff + node)];
                mk[x][1] = p.anc_mask[2 * (size_t)(koff + node) + 1];
            }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qf[ks][x] = src ? __ldg(src + (ks * 16 + qd) / 2) : 0u;
                qf[ks][x + 2] = src ? __ldg(src + (ks * 16 + 8 + qd) / 2) : 0u;
            }
        }
    }

    float oacc[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
    float mrun[2] = {-CUDART_INF_F, -CUDART_INF_F};
    float lrun[2] = {0.f, 0.f};

    // ---- tile loader -----------------------------------------------------------------------------------
    auto issue = [&](int tile, int stage) {
        const unsigned int sK = smem_base + stage * ATT_STAGE_BYTES, sV = sK + ATT_TILE_BYTES;
        if (tile < t_prefix) {
            if (tid == 0) {
                const unsigned int bar = bar0 + stage * 8;
                const int tok = kv0 + tile * ATT_BN;
                mbar_expect_tx(bar, ATT_STAGE_BYTES);
                if (p.head_first) {      // tensor dims (d, token, head)
                    tma_load_3d(sK, &tmK, 0, tok, h, bar);
                    tma_load_3d(sK + ATT_TILE_BYTES / 2, &tmK, 64, tok, h, bar);
                    tma_load_3d(sV, &tmV, 0, tok, h, bar);
                    tma_load_3d(sV + ATT_TILE_BYTES / 2, &tmV, 64, tok, h, bar);
                } else {                 // tensor dims (d, head, token)
                    tma_load_3d(sK, &tmK, 0, h, tok, bar);
                    tma_load_3d(sK + ATT_TILE_BYTES / 2, &tmK, 64, h, tok, bar);
                    tma_load_3d(sV, &tmV, 0, h, tok, bar);
                    tma_load_3d(sV + ATT_TILE_BYTES / 2, &tmV, 64, h, tok, bar);
                }
            }
        } else {
            // tree keys/values: gathered rows, 16-byte loads, swizzled stores (2 x 1024 chunks / 256 threads)
            unsigned char* gK = smem_gen + stage * ATT_STAGE_BYTES;
            unsigned char* gV = gK + ATT_TILE_BYTES;
            const int j0 = (tile - t_prefix) * ATT_BN;
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const int c = tid + it * ATT_THREADS;       // 0..1023
                const int key = c >> 4, chunk = c & 15;
                const int j = j0 + key;
                uint4 kvv = make_uint4(0, 0, 0, 0), vvv = make_uint4(0, 0, 0, 0);
                if (j < nk) {
                    const int trow = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + j] : koff + j;
                    const size_t off = ((size_t)trow * p.hkv + h) * HS_HEAD_DIM + chunk * 8;
                    kvv = __ldg(reinterpret_cast<const uint4*>(p.k_tree + off));
                    vvv = __ldg(reinterpret_cast<const uint4*>(p.v_tree + off));
                }
                *reinterpret_cast<uint4*>(gK + tile_off(key, chunk)) = kvv;
                *reinterpret_cast<uint4*>(gV + tile_off(key, chunk)) = vvv;
            }
        }
    };

    unsigned int phase[2] = {0u, 0u};
    issue(t0, 0);
    if (t0 >= t_prefix) __syncthreads();
    for (int tile = t0; tile < t1; ++tile) {
        const int stage = (tile - t0) & 1;
        if (tile + 1 < t1) issue(tile + 1, stage ^ 1);
        if (tile < t_prefix) {
            mbar_wait(bar0 + stage * 8, phase[stage], p.err);
            phase[stage] ^= 1u;
        }
        const unsigned int sK = smem_base + stage * ATT_STAGE_BYTES, sV = sK + ATT_TILE_BYTES;

        // ---- S = Q K^T (16 x 64 per warp) -----------------------------------------------------------------
        float sacc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
            const int key = nt * 8 + (lane & 7);
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                unsigned int b0, b1, b2, b3;
                ldsm_x4(sK + tile_off(key, kp * 4 + (lane >> 3)), b0, b1, b2, b3);
                mma_bf16(sacc[nt], qf[2 * kp], b0, b1);
                mma_bf16(sacc[nt], qf[2 * kp + 1], b2, b3);
            }
        }
        // ---- scale, mask, online softmax ---------------------------------------------------------------------
        const bool is_tree = tile >= t_prefix;
        const int col0 = is_tree ? (tile - t_prefix) * ATT_BN : tile * ATT_BN;
        const int limit = is_tree ? nk : L;
        float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
        // a tree tile of 64 keys lies inside one 64-bit word of the ancestor mask
        const unsigned long long mw[2] = {col0 == 0 ? mk[0][0] : mk[0][1], col0 == 0 ? mk[1][0] : mk[1][1]};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int cl = nt * 8 + qd + (e & 1);
                const int col = col0 + cl;
                const int x = e >> 1;
                bool vis = col < limit;
                if (is_tree && vis) vis = (mw[x] >> cl) & 1ull;
                const float sv = vis ? sacc[nt][e] * p.scale_log2 : -CUDART_INF_F;
                sacc[nt][e] = sv;
                mx[x] = fmaxf(mx[x], sv);
            }
        }
        float corr[2], muse[2];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            mx[x] = fmaxf(mx[x], __shfl_xor_sync(HS_FULL_MASK, mx[x], 1));
            mx[x] = fmaxf(mx[x], __shfl_xor_sync(HS_FULL_MASK, mx[x], 2));
            const float mnew = fmaxf(mrun[x], mx[x]);
            muse[x] = (mnew == -CUDART_INF_F) ? 0.f : mnew;
            corr[x] = ex2(mrun[x] - muse[x]);
            mrun[x] = mnew;
            lrun[x] *= corr[x];
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            oacc[i][0] *= corr[0]; oacc[i][1] *= corr[0];
            oacc[i][2] *= corr[1]; oacc[i][3] *= corr[1];
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pv = ex2(sacc[nt][e] - muse[e >> 1]);
                sacc[nt][e] = pv;
                lrun[e >> 1] += pv;
            }
        }
        // ---- O += P V ---------------------------------------------------------------------------------------------
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            unsigned int pa[4];
            pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
            pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
            pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
            pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
            const int key = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
            for (int dc = 0; dc < 8; ++dc) {
                unsigned int b0, b1, b2, b3;
                ldsm_x4_t(sV + tile_off(key, dc * 2 + (lane >> 4)), b0, b1, b2, b3);
                mma_bf16(oacc[2 * dc], pa, b0, b1);
                mma_bf16(oacc[2 * dc + 1], pa, b2, b3);
            }
        }
        __syncthreads();     // the stage may be refilled; generic tree-tile stores become visible
    }

    // ---- epilogue --------------------------------------------------------------------------------------------------
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        lrun[x] += __shfl_xor_sync(HS_FULL_MASK, lrun[x], 1);
        lrun[x] += __shfl_xor_sync(HS_FULL_MASK, lrun[x], 2);
    }
    const int rr[2] = {r0, r1};
    if (p.nsplit == 1) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            if (orow[x] < 0) continue;
            const float inv = lrun[x] > 0.f ? 1.f / lrun[x] : 0.f;
            __nv_bfloat16* dst = p.out + (size_t)orow[x] * HS_HEAD_DIM;
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *reinterpret_cast<unsigned int*>(dst + i * 8 + qd) =
                    pack_bf16(oacc[i][2 * x] * inv, oacc[i][2 * x + 1] * inv);
            if (p.lse_out && (lane & 3) == 0) p.lse_out[orow[x]] = (mrun[x] + log2f(lrun[x])) * LN2;
        }
    } else {
        const size_t pbase = ((size_t)pair * p.nsplit + split) * p.mpad;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            if (orow[x] < 0) continue;
            float* dst = p.part_o + (pbase + rr[x]) * HS_HEAD_DIM;
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *reinterpret_cast<float2*>(dst + i * 8 + qd) = make_float2(oacc[i][2 * x], oacc[i][2 * x + 1]);
            if ((lane & 3) == 0) p.part_ml[pbase + rr[x]] = make_float2(mrun[x], lrun[x]);
        }
    }
}

// one warp per (sequence, kv head, query row); lane owns 4 of the 128 output values
__global__ void __launch_bounds__(256) tree_attn_combine_kernel(const AttnParams p) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int pair = blockIdx.y, b = pair / p.hkv, h = pair % p.hkv;
    const int nk = (p.status[b] == 0) ? p.n_keep[b] : 0;
    if (r >= nk * p.G) return;
    const int L = p.kv_off[b + 1] - p.kv_off[b];
    const int koff = p.keep_off[b];
    const int node = r / p.G, g = r % p.G;
    const int trow = (p.layout == HS_ROWS_ORIGINAL) ? p.node_off[b] + p.keep_idx[koff + node] : koff + node;
    const size_t orow = (size_t)trow * p.hq + h * p.G + g;
    float M = -CUDART_INF_F;
    for (int s = 0; s < p.nsplit; ++s) {
        int tp, tt, t0, t1;
        split_range(L, nk, p.nsplit, s, tp, tt, t0, t1);
        if (t0 >= t1) break;
        M = fmaxf(M, p.part_ml[((size_t)pair * p.nsplit + s) * p.mpad + r].x);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float lsum = 0.f;
    for (int s = 0; s < p.nsplit; ++s) {
        int tp, tt, t0, t1;
        split_range(L, nk, p.nsplit, s, tp, tt, t0, t1);
        if (t0 >= t1) break;
        const size_t pb = ((size_t)pair * p.nsplit + s) * p.mpad + r;
        const float2 ml = p.part_ml[pb];
        const float w = (ml.x == -CUDART_INF_F) ? 0.f : ex2(ml.x - M);
        const float4 o = *reinterpret_cast<const float4*>(p.part_o + pb * HS_HEAD_DIM + lane * 4);
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        lsum += w * ml.y;
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + orow * HS_HEAD_DIM + lane * 4) = packed;
    if (p.lse_out && lane == 0) p.lse_out[orow] = (M + log2f(lsum)) * LN2;
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

hs_status hs_launch_attention(hs_ctx* ctx, const hs_pruned_tree* pruned, const hs_attn_desc* d, const void* q,
                              const void* k_tree, const void* v_tree, const void* k_cache, const void* v_cache,
                              void* out, float* lse_out, cudaStream_t stream) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(tree_attn_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ATT_SMEM_BYTES) != cudaSuccess)
            return HS_ERR_CUDA;
        attr_set = true;
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
    p.mpad = p.G * d->max_nodes;
    p.head_first = d->kv_head_stride > d->kv_token_stride;
    p.scale_log2 = d->sm_scale * LOG2E;
    p.err = ctx->counters + HS_CNT_ERROR;
    const int pairs = d->batch * d->hkv;
    const int mblocks = (p.mpad + ATT_BM - 1) / ATT_BM;
    const int tiles_max = (d->max_kv_len + ATT_BN - 1) / ATT_BN + (d->max_nodes + ATT_BN - 1) / ATT_BN;
    int nsplit = (ctx->sm_count + pairs * mblocks - 1) / (pairs * mblocks);
    if (nsplit > tiles_max) nsplit = tiles_max;
    if (nsplit < 1) nsplit = 1;
    const size_t per_split = (size_t)pairs * p.mpad * (HS_HEAD_DIM * sizeof(float) + sizeof(float2));
    while (nsplit > 1 && per_split * nsplit + 256 > ctx->scratch_bytes) --nsplit;
    p.nsplit = nsplit;
    p.part_o = (float*)ctx->scratch;
    p.part_ml = (float2*)(ctx->scratch + hs_align_up((size_t)pairs * nsplit * p.mpad * HS_HEAD_DIM * sizeof(float), 256));

    CUtensorMap tmK, tmV;
    memset(&tmK, 0, sizeof(tmK));
    memset(&tmV, 0, sizeof(tmV));
    if (d->kv_total > 0) {
        if (!make_kv_map(ctx, &tmK, k_cache, d, p.head_first) || !make_kv_map(ctx, &tmV, v_cache, d, p.head_first))
            return HS_ERR_CUDA;
    }
    dim3 grid(mblocks, nsplit, pairs);
    tree_attn_split_kernel<<<grid, ATT_THREADS, ATT_SMEM_BYTES, stream>>>(p, tmK, tmV);
    if (cudaGetLastError() != cudaSuccess) return HS_ERR_CUDA;
    if (nsplit > 1) {
        dim3 cgrid((p.mpad + 7) / 8, pairs);
        tree_attn_combine_kernel<<<cgrid, 256, 0, stream>>>(p);
        if (cudaGetLastError() != cudaSuccess) return HS_ERR_CUDA;
    }
    return HS_OK;
}
