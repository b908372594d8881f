// hs_cart_fit: training of the entropy stratifier on the device (Sec. 4.2, Eq. 2).
//
// One feature (x = Phi(P*)) and one target (y = Terminal Confidence Rank): the samples are sorted by x once (bitonic
// network: chunks of 1024 in shared memory, wider exchanges in global memory), running sums of y and y^2 in double
// precision follow, and then every layer of the tree scores all split positions of all its nodes in parallel from
// the running sums - a node is a contiguous range of the sorted samples, a split at position i costs
//     L = nL / N * (SyyL - SyL^2 / nL) + nR / N * (SyyR - SyR^2 / nR)           (Eq. 2)
// - and takes, per node, the position with the smallest L (ties: the smallest), between distinct feature values
// only.  The threshold is the midpoint of the two neighbouring feature values.
#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

#define CT_THREADS 256
#define CT_CHUNK 1024
#define CT_MAX_DEPTH 6
#define CT_SPLIT_BLOCKS 64          // blocks that share the split positions of one node

// key = (order-preserving bits of x) : (bits of y); padding keys are all ones and sort to the end
__global__ void cart_pack_kernel(const float* x, const float* y, int n, int P, unsigned long long* keys) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= P) return;
    keys[i] = i < n ? (((unsigned long long)float_order_bits(x[i]) << 32) | __float_as_uint(y[i])) : ~0ull;
}

__device__ __forceinline__ void cmp_swap(unsigned long long& a, unsigned long long& b, bool up) {
    if ((a > b) == up) { const unsigned long long t = a; a = b; b = t; }
}

// all exchange distances below CT_CHUNK of the merge step of width k (k >= 2), inside shared memory;
// with k <= CT_CHUNK and first == true the chunk is sorted from scratch
__global__ void __launch_bounds__(CT_CHUNK / 2) cart_sort_chunk_kernel(unsigned long long* keys, int k_lo, int k_hi) {
    __shared__ unsigned long long s[CT_CHUNK];
    const int tid = threadIdx.x;
    const size_t base = (size_t)blockIdx.x * CT_CHUNK;
    s[tid] = keys[base + tid];
    s[tid + CT_CHUNK / 2] = keys[base + tid + CT_CHUNK / 2];
    __syncthreads();
    for (int k = k_lo; k <= k_hi; k <<= 1) {
        for (int j = min(k >> 1, CT_CHUNK / 2); j > 0; j >>= 1) {
            const int i = 2 * tid - (tid & (j - 1));           // lower index of this thread's pair
            const bool up = (((base + i) & (size_t)k) == 0);
            cmp_swap(s[i], s[i + j], up);
            __syncthreads();
        }
    }
    keys[base + tid] = s[tid];
    keys[base + tid + CT_CHUNK / 2] = s[tid + CT_CHUNK / 2];
}

// one exchange distance j >= CT_CHUNK of the merge step of width k, in global memory
__global__ void cart_sort_global_kernel(unsigned long long* keys, int P, int j, int k) {
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (size_t)P / 2) return;
    const size_t i = 2 * t - (t & (size_t)(j - 1));
    const bool up = ((i & (size_t)k) == 0);
    unsigned long long a = keys[i], b = keys[i + j];
    if ((a > b) == up) { keys[i] = b; keys[i + j] = a; }
}

// running sums: block-wise inclusive scans of y and y^2 (double), the blocks' totals, their scan, the offsets
__global__ void __launch_bounds__(CT_THREADS) cart_scan_blocks_kernel(const unsigned long long* keys, int n, double* sy,
                                                                      double* syy, double* blk) {
    __shared__ double s_a[CT_THREADS], s_b[CT_THREADS];
    const int tid = threadIdx.x;
    const int i = blockIdx.x * CT_THREADS + tid;
    double a = 0.0, b = 0.0;
    if (i < n) { a = (double)__uint_as_float((unsigned int)keys[i]); b = a * a; }
    s_a[tid] = a; s_b[tid] = b;
    __syncthreads();
    for (int o = 1; o < CT_THREADS; o <<= 1) {
        double ua = 0.0, ub = 0.0;
        if (tid >= o) { ua = s_a[tid - o]; ub = s_b[tid - o]; }
        __syncthreads();
        s_a[tid] += ua; s_b[tid] += ub;
        __syncthreads();
    }
    if (i < n) { sy[i + 1] = s_a[tid]; syy[i + 1] = s_b[tid]; }          // (exclusive sums: entry i = samples before i)
    if (tid == CT_THREADS - 1) { blk[2 * blockIdx.x] = s_a[tid]; blk[2 * blockIdx.x + 1] = s_b[tid]; }
    if (i == 0) { sy[0] = 0.0; syy[0] = 0.0; }
}
__global__ void cart_scan_totals_kernel(double* blk, int nblk) {     // one thread: the blocks' totals in order
    double a = 0.0, b = 0.0;
    for (int i = 0; i < nblk; ++i) {
        const double ta = blk[2 * i], tb = blk[2 * i + 1];
        blk[2 * i] = a; blk[2 * i + 1] = b;
        a += ta; b += tb;
    }
}
__global__ void __launch_bounds__(CT_THREADS) cart_scan_add_kernel(int n, double* sy, double* syy, const double* blk) {
    const int i = blockIdx.x * CT_THREADS + threadIdx.x;
    if (i < n) { sy[i + 1] += blk[2 * blockIdx.x]; syy[i + 1] += blk[2 * blockIdx.x + 1]; }
}

struct CartLevel {
    const unsigned long long* keys;
    const double* sy;
    const double* syy;
    const int* bnd;        // [nodes + 1] node boundaries (positions in the sorted order) of this layer
    int* bnd_next;         // [2 * nodes + 1]
    double* part_l;        // [nodes][CT_SPLIT_BLOCKS] best loss of a block
    int* part_i;           // [nodes][CT_SPLIT_BLOCKS] its position
    float* thresholds;     // [2^depth - 1] ascending
    int* status;
    int nodes, level, depth;
};

__device__ __forceinline__ float key_x(unsigned long long k) { return order_bits_float((unsigned int)(k >> 32)); }

__global__ void __launch_bounds__(CT_THREADS) cart_split_scan_kernel(const CartLevel c) {
    __shared__ double s_l[CT_THREADS];
    __shared__ int s_i[CT_THREADS];
    const int node = blockIdx.y, tid = threadIdx.x;
    const int lo = c.bnd[node], hi = c.bnd[node + 1];
    const double N = (double)(hi - lo);
    double best = CUDART_INF;
    int best_i = 0x7fffffff;
    const double sy_lo = c.sy[lo], syy_lo = c.syy[lo], sy_hi = c.sy[hi], syy_hi = c.syy[hi];
    for (int i = lo + 1 + blockIdx.x * CT_THREADS + tid; i < hi; i += CT_SPLIT_BLOCKS * CT_THREADS) {
        if (!(key_x(c.keys[i - 1]) < key_x(c.keys[i]))) continue;       // a threshold lies between distinct values
        const double nl = (double)(i - lo), nr = (double)(hi - i);
        const double yl = c.sy[i] - sy_lo, yyl = c.syy[i] - syy_lo;
        const double yr = sy_hi - c.sy[i], yyr = syy_hi - c.syy[i];
        const double l = nl / N * (yyl - yl * yl / nl) + nr / N * (yyr - yr * yr / nr);
        if (l < best) { best = l; best_i = i; }                          // (ascending i: the first minimum stays)
    }
    s_l[tid] = best; s_i[tid] = best_i;
    __syncthreads();
    for (int o = CT_THREADS / 2; o > 0; o >>= 1) {
        if (tid < o) {
            const double l2 = s_l[tid + o];
            const int i2 = s_i[tid + o];
            if (l2 < s_l[tid] || (l2 == s_l[tid] && i2 < s_i[tid])) { s_l[tid] = l2; s_i[tid] = i2; }
        }
        __syncthreads();
    }
    if (tid == 0) { c.part_l[node * CT_SPLIT_BLOCKS + blockIdx.x] = s_l[0]; c.part_i[node * CT_SPLIT_BLOCKS + blockIdx.x] = s_i[0]; }
}

__global__ void cart_split_pick_kernel(const CartLevel c) {            // one thread per node
    const int node = blockIdx.x * blockDim.x + threadIdx.x;
    if (node >= c.nodes) return;
    double best = CUDART_INF;
    int best_i = 0x7fffffff;
    for (int b = 0; b < CT_SPLIT_BLOCKS; ++b) {
        const double l = c.part_l[node * CT_SPLIT_BLOCKS + b];
        const int i = c.part_i[node * CT_SPLIT_BLOCKS + b];
        if (l < best || (l == best && i < best_i)) { best = l; best_i = i; }
    }
    const int lo = c.bnd[node], hi = c.bnd[node + 1];
    // position of this node's threshold in the ascending list: in-order index of the node
    const int slot = (2 * node + 1) * (1 << (c.depth - 1 - c.level)) - 1;
    if (best_i == 0x7fffffff) {                      // a single feature value: the node cannot be split
        *c.status = HS_ERR_SHAPE;
        c.thresholds[slot] = CUDART_NAN_F;
        best_i = hi;
    } else {
        c.thresholds[slot] = (float)(0.5 * ((double)key_x(c.keys[best_i - 1]) + (double)key_x(c.keys[best_i])));
    }
    c.bnd_next[2 * node] = lo;
    c.bnd_next[2 * node + 1] = best_i;
    if (node == c.nodes - 1) c.bnd_next[2 * c.nodes] = hi;
}

__global__ void cart_init_kernel(int* bnd, int n, int* status) { bnd[0] = 0; bnd[1] = n; *status = HS_OK; }

static int next_pow2(int n) { int p = CT_CHUNK; while (p < n) p <<= 1; return p; }

extern "C" size_t hs_cart_workspace_bytes(int32_t n) {
    if (n < 2) return 0;
    const size_t P = next_pow2(n);
    return HS_COUNTER_BYTES + P * 8 + 2 * ((size_t)n + 1) * 8 + 2 * (((size_t)n + CT_THREADS - 1) / CT_THREADS) * 8 +
           2 * (2 << CT_MAX_DEPTH) * 4 + (1 << CT_MAX_DEPTH) * CT_SPLIT_BLOCKS * 12 + 4096;
}

extern "C" hs_status hs_cart_fit(hs_ctx* ctx, const float* x, const float* y, int32_t n, int32_t depth,
                                 float* thresholds, int32_t* status, hs_stream stream_) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ctx || !hs_on_device(ctx) || !x || !y || !thresholds || !status) return HS_ERR_INVALID_ARG;
    if (depth < 1 || depth > CT_MAX_DEPTH || n < (1 << depth) || n > (1 << 26)) return HS_ERR_SHAPE;
    const int P = next_pow2(n);
    const int nblk = (n + CT_THREADS - 1) / CT_THREADS;
    // workspace: keys | sy | syy | block totals | two boundary arrays | per-block minima
    size_t o = 0;
    auto take = [&](size_t bytes) { char* p = ctx->scratch + o; o += hs_align_up(bytes, 256); return p; };
    unsigned long long* keys = (unsigned long long*)take((size_t)P * 8);
    double* sy = (double*)take(((size_t)n + 1) * 8);
    double* syy = (double*)take(((size_t)n + 1) * 8);
    double* blk = (double*)take((size_t)nblk * 16);
    int* bnd_a = (int*)take((2 << CT_MAX_DEPTH) * 4);
    int* bnd_b = (int*)take((2 << CT_MAX_DEPTH) * 4);
    double* part_l = (double*)take((size_t)(1 << CT_MAX_DEPTH) * CT_SPLIT_BLOCKS * 8);
    int* part_i = (int*)take((size_t)(1 << CT_MAX_DEPTH) * CT_SPLIT_BLOCKS * 4);
    if (o > ctx->scratch_bytes) return HS_ERR_WORKSPACE;

    cart_pack_kernel<<<(P + 255) / 256, 256, 0, stream>>>(x, y, n, P, keys);
    cart_sort_chunk_kernel<<<P / CT_CHUNK, CT_CHUNK / 2, 0, stream>>>(keys, 2, CT_CHUNK);
    for (int k = 2 * CT_CHUNK; k <= P; k <<= 1) {
        for (int j = k >> 1; j >= CT_CHUNK; j >>= 1)
            cart_sort_global_kernel<<<(P / 2 + 255) / 256, 256, 0, stream>>>(keys, P, j, k);
        cart_sort_chunk_kernel<<<P / CT_CHUNK, CT_CHUNK / 2, 0, stream>>>(keys, k, k);
    }
    cart_scan_blocks_kernel<<<nblk, CT_THREADS, 0, stream>>>(keys, n, sy, syy, blk);
    cart_scan_totals_kernel<<<1, 1, 0, stream>>>(blk, nblk);
    cart_scan_add_kernel<<<nblk, CT_THREADS, 0, stream>>>(n, sy, syy, blk);
    cart_init_kernel<<<1, 1, 0, stream>>>(bnd_a, n, status);
    for (int level = 0; level < depth; ++level) {
        CartLevel c;
        c.keys = keys; c.sy = sy; c.syy = syy;
        c.bnd = (level & 1) ? bnd_b : bnd_a;
        c.bnd_next = (level & 1) ? bnd_a : bnd_b;
        c.part_l = part_l; c.part_i = part_i; c.thresholds = thresholds; c.status = status;
        c.nodes = 1 << level; c.level = level; c.depth = depth;
        cart_split_scan_kernel<<<dim3(CT_SPLIT_BLOCKS, c.nodes), CT_THREADS, 0, stream>>>(c);
        cart_split_pick_kernel<<<1, 64, 0, stream>>>(c);
    }
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
