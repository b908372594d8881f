// hs_accept_path: the row pass (one of two kernels) and, with draft logits, the walk.
//
// accept_rows_kernel   vocabulary pass over the target row of every kept node (arg-max with lowest
//                      index on ties; for sampling sequences also max and sum e^((x-max)/T)) and
//                      over the draft row of every kept internal node of a sampling sequence.
//                      A CTA per 32 KiB chunk of a row, all 16-byte loads in flight at once (launches
//                      with few rows); the chunks of a row merge in the shared memory of a thread-block
//                      cluster, or through partials and an arrival counter where the grid is too large
//                      for clusters to pay.
// accept_stream_kernel the same pass for launches with many rows: one persistent CTA per SM, a producer
//                      warp and a ring of shared-memory slots (see the comment ahead of the kernel).
//                      Greedy sequences and sequences with deterministic proposals finish in the row
//                      pass: the CTA that completes a sequence's last target row walks its tree
//                      (greedy_walk, deterministic_walk).
// accept_walk_kernel   one thread-block cluster per sequence walks the tree from the root.
//                      Greedy (temperature 0): follow the child whose token is the arg-max.
//                      Sampling (Sec. 2.1): test siblings in index order with u < min(1, r/q); the
//                      residual after k rejections is max(p - c_k q, 0) / W_k with c_0 = 0, W_0 = 1,
//                      c_(k+1) = c_k + W_k, W_k = sum_v max(p_v - c_k q_v, 0), so a rejection costs
//                      one vocabulary-wide sum, split over the CTAs of the cluster and exchanged
//                      through distributed shared memory.  The bonus token is drawn by inverse CDF
//                      in token order.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

namespace cg = cooperative_groups;

#define LOG2E 1.4426950408889634f
#define WALK_CLUSTER 16       // (larger than the portable 8: the launcher asks for it)
#define WALK_THREADS 512

struct RowOut {           // per kept node, in the workspace
    int* tgt_arg;         // arg-max token of the target row
    float2* tgt_ms;       // {max, sum e^((x-max)/T)} of the target row
    float2* drf_ms;       // same for the draft row (internal nodes of sampling sequences)
};

struct AcceptParams {
    const void* target;
    const void* draft;
    int64_t row_stride;
    int vocab, nvec, chunks, chunk_vecs, is_bf16, have_draft;
    int batch, n_nodes_total, target_layout, part_rows;
    const int* node_off;
    const int* token;
    hs_pruned_tree pr;
    const int* mode;
    const float* temperature;
    unsigned long long seed, offset;
    const float* uniforms;
    hs_accept_out out;
    RowOut ro;
    uint4* partials;      // [2][max_rows][chunks] {key lo, key hi, max, sum}
    int* row_cnt;
    int* seq_cnt;         // [batch] merged target rows of a sequence (zero between launches)
    int clustered;        // chunk kernel: the chunks of a row form a thread-block cluster and merge through shared memory
    int staged;           // the walk may stage row slices in shared memory by bulk copies (16-byte aligned rows)
    int* err;             // sticky device error word (a bounded wait that expired)
};

__device__ __forceinline__ float ex2a(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <bool BF16>
__device__ __forceinline__ void unpack_v(const uint4& v, float* x) {
    if (BF16) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    } else {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
}

// Greedy acceptance of sequence b by one whole CTA (Sec. 5, temperature 0): from the root, move to the kept
// child whose token is the arg-max of the current node's target row until no child matches; the bonus
// token is the arg-max where the walk stops.  tgt_arg was written by other CTAs: read it past L1.
// The two walks below are run by the first HS_ROW_THREADS threads of a CTA (the whole CTA of the chunk kernel, half
// of the consumer warps of the streaming kernel), which meet on a barrier of their own.
__device__ __forceinline__ void walk_sync() { named_bar_sync(2, HS_ROW_THREADS); }

__device__ void greedy_walk(const AcceptParams& p, int b) {
    __shared__ int s_arg[HS_MAX_NODES], s_next[HS_MAX_NODES], s_orig[HS_MAX_NODES];
    const int tid = threadIdx.x, nthr = HS_ROW_THREADS;
    const int koff = p.pr.keep_off[b];
    const int nk = min(p.pr.n_keep[b], HS_MAX_NODES);
    const int nbase = p.node_off[b];
    const int cap = p.out.path_cap;
    // Every kept node's parent, token and its row's arg-max in one round trip; the walk itself then runs in shared
    // memory: node j continues the path of its parent iff its token is the parent's arg-max, and of several such
    // children (duplicate tokens among siblings) the one with the lowest index does.
    int my_par = -1, my_tok = -1;
    if (tid < nk) {
        my_par = p.pr.new_parent[koff + tid];
        const int orig = p.pr.keep_idx[koff + tid];
        s_arg[tid] = __ldcg(&p.ro.tgt_arg[koff + tid]);
        s_orig[tid] = orig;
        s_next[tid] = 0x7fffffff;
        my_tok = p.token[nbase + orig];
    }
    for (int j = tid; j < cap; j += nthr) {
        p.out.path_nodes[b * cap + j] = -1;
        p.out.path_compact[b * cap + j] = -1;
        p.out.path_tokens[b * cap + j] = -1;
    }
    walk_sync();
    if (tid > 0 && tid < nk && my_par >= 0 && my_par < tid && my_tok == s_arg[my_par]) atomicMin(&s_next[my_par], tid);
    walk_sync();
    if (tid == 0) {
        int cur = 0, len = 0;
        for (int step = 0; step < nk; ++step) {
            if (len < cap) {
                p.out.path_compact[b * cap + len] = cur;
                p.out.path_nodes[b * cap + len] = s_orig[cur];
            }
            const int nxt = s_next[cur];
            if (nxt == 0x7fffffff) break;
            if (len < cap) p.out.path_tokens[b * cap + len] = s_arg[cur];
            cur = nxt;
            ++len;
        }
        p.out.accept_len[b] = len;
        p.out.bonus_token[b] = s_arg[cur];
        p.out.terminal_rank[b] = p.pr.keep_rank[koff + cur];
        p.out.status[b] = HS_OK;
    }
}

__device__ __forceinline__ float load_logit(const void* base, int is_bf16, size_t off);

// Acceptance of sequence b with deterministic proposals by one whole CTA (Sec. 2.1 with a point-mass proposal per
// candidate): at node cur with p = softmax(target row / T) the kept children are tried in index order; child x
// with token t is accepted iff u_x < min(1, p_t / W), W = 1 - (mass of the tokens rejected at this node so far); a
// rejection removes t.  When no candidate is left the bonus token is drawn by inverse CDF in token order from p
// without the rejected tokens (running sums in double, one contiguous run of tokens per thread).
__device__ __noinline__ void deterministic_walk(const AcceptParams& p, int b) {
    __shared__ int s_par[HS_MAX_NODES], s_tok[HS_MAX_NODES], s_rej[HS_MAX_NODES];
    __shared__ float s_pt[HS_MAX_NODES], s_u[HS_MAX_NODES];     // p(token of node j | its parent), its accept uniform
    __shared__ double s_scan[HS_ROW_THREADS / 32];
    __shared__ double s_phase[64];
    __shared__ double s_wp[64][HS_ROW_THREADS / 32];     // per (phase, warp) sums of pass 1
    __shared__ int s_pick[2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = HS_ROW_THREADS;
    const int koff = p.pr.keep_off[b];
    const int nk = min(p.pr.n_keep[b], HS_MAX_NODES);
    const int nbase = p.node_off[b];
    const int cap = p.out.path_cap;
    for (int j = tid; j < cap; j += nthr) {
        p.out.path_nodes[b * cap + j] = -1;
        p.out.path_compact[b * cap + j] = -1;
        p.out.path_tokens[b * cap + j] = -1;
    }
    for (int j = tid; j < nk; j += nthr) {
        s_par[j] = p.pr.new_parent[koff + j];
        s_tok[j] = p.token[nbase + p.pr.keep_idx[koff + j]];
    }
    walk_sync();
    const float invT = LOG2E / p.temperature[b];
    const size_t esz = p.is_bf16 ? 2 : 4;
    // every candidate's probability under its parent's target row and its uniform, all nodes at once (one round
    // trip instead of one per sibling test); the walk below then runs from shared memory
    for (int j = 1 + tid; j < nk; j += nthr) {
        const int par = s_par[j];
        const int orig = p.pr.keep_idx[koff + j];
        float pt = 0.f;
        if (par >= 0 && par < nk) {
            const int prow_i = p.target_layout == HS_ROWS_ORIGINAL ? nbase + p.pr.keep_idx[koff + par] : koff + par;
            const char* row = (const char*)p.target + (size_t)prow_i * p.row_stride * esz;
            const float2 ms = __ldcg(&p.ro.tgt_ms[koff + par]);      // written by another CTA of this launch
            pt = exp2f((fmaxf(load_logit(row, p.is_bf16, s_tok[j]), -1e30f) - ms.x) * invT) * (1.f / ms.y);
        }
        s_pt[j] = pt;
        s_u[j] = p.uniforms ? p.uniforms[nbase + orig] : philox_uniform(p.seed, p.offset, b, orig, 0);
    }
    walk_sync();
    int cur = 0, len = 0, bonus = -1;
    for (int step = 0; step < nk; ++step) {
        if (tid == 0 && len < cap) {
            p.out.path_compact[b * cap + len] = cur;
            p.out.path_nodes[b * cap + len] = p.pr.keep_idx[koff + cur];
        }
        const int orig_cur = p.pr.keep_idx[koff + cur];
        const int trow = p.target_layout == HS_ROWS_ORIGINAL ? nbase + orig_cur : koff + cur;
        const char* prow = (const char*)p.target + (size_t)trow * p.row_stride * esz;
        const float2 pms = __ldcg(&p.ro.tgt_ms[koff + cur]);      // written by another CTA of this launch
        const float pm = pms.x, ips = 1.f / pms.y;
        double W = 1.0;
        int nrej = 0, accepted = -1;
        for (int j = cur + 1; j < nk; ++j) {                     // siblings in index order (every thread the same)
            if (s_par[j] != cur) continue;
            const int t = s_tok[j];
            float pt = s_pt[j];
            for (int k = 0; k < nrej; ++k)                       // a token rejected at this node has left the residual
                if (s_rej[k] == t) pt = 0.f;
            const float a = fminf(1.f, pt / (float)W);
            if (s_u[j] < a) { accepted = j; break; }
            const double W_next = W - (double)pt;
            if (!(W_next > 0.0)) { nrej = 0; W = 1.0; break; }  // nothing left: fall back to p
            walk_sync();                                     // (every thread walks the same way)
            if (tid == 0) s_rej[nrej] = t;
            walk_sync();
            ++nrej;
            W = W_next;
        }
        if (accepted >= 0) {
            if (tid == 0 && len < cap) p.out.path_tokens[b * cap + len] = s_tok[accepted];
            cur = accepted;
            ++len;
            continue;
        }
        // ---- the bonus token: inverse CDF over the vocabulary without the rejected tokens -------------------
        // The row is taken in phases of nthr * 4 vectors; in a phase thread t owns 4 consecutive 16-byte vectors (all
        // loads in flight together), so token order is (phase, thread, token).  Pass 1 sums
        // every phase; then the phase that holds the crossing is summed again and scanned.
        const float ufin = p.uniforms ? p.uniforms[p.n_nodes_total + b] : philox_uniform(p.seed, p.offset, b, 0, 1);
        if (tid == 0) { s_pick[0] = 0x7fffffff; s_pick[1] = -1; }
        walk_sync();                                         // s_rej, s_pick
        const int ve = p.is_bf16 ? 8 : 4;
        const int phase_vecs = nthr * 4;
        // (at most 64 phases: the launcher refuses vocabularies of more than 32 chunks = 64 phases)
        const int nph = min((p.nvec + phase_vecs - 1) / phase_vecs, 64);
        // masses of this thread's 4 vectors of phase ph (0 past the vocabulary and for rejected tokens)
        auto phase_mass = [&](int ph, float (&m)[4][8]) {
            uint4 d[4];
            const int vbase = ph * phase_vecs + tid * 4;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                d[q] = (vbase + q < p.nvec) ? __ldg((const uint4*)prow + vbase + q) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float x[8];
                if (p.is_bf16) unpack_v<true>(d[q], x); else unpack_v<false>(d[q], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int tok = (vbase + q) * ve + e;
                    const bool in = e < ve && vbase + q < p.nvec && tok < p.vocab;
                    m[q][e] = in ? exp2f((fmaxf(x[e], -1e30f) - pm) * invT) * ips : 0.f;
                }
            }
            for (int k = 0; k < nrej; ++k) {                     // few: the siblings rejected at this node
                const int rv = s_rej[k] / ve - vbase;
                if (rv >= 0 && rv < 4) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (q == rv && e == s_rej[k] % ve) m[q][e] = 0.f;
                }
            }
        };
        int last_pos = -1;
#pragma unroll 2
        for (int ph = 0; ph < nph; ++ph) {
            float m[4][8];
            phase_mass(ph, m);
            double mine = 0.0;
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    mine += (double)m[q][e];
                    if (m[q][e] > 0.f) last_pos = ((ph * phase_vecs + tid * 4 + q) * ve + e);
                }
            const double w = warp_sum_d(mine);
            if (lane == 0) s_wp[ph][warp] = w;           // (no barrier per phase: the loads of the next one go out)
        }
        walk_sync();
        for (int ph = tid; ph < nph; ph += nthr) {
            double t = 0.0;
            for (int w2 = 0; w2 < nthr / 32; ++w2) t += s_wp[ph][w2];
            s_phase[ph] = t;
        }
        walk_sync();
        double total = 0.0;
        for (int ph = 0; ph < nph; ++ph) total += s_phase[ph];
        const double goal = (double)ufin * total;
        int phx = -1;                                            // first phase whose running total exceeds the goal
        double before_ph = 0.0;
        for (int ph = 0; ph < nph; ++ph) {
            if (before_ph + s_phase[ph] > goal) { phx = ph; break; }
            before_ph += s_phase[ph];
        }
        if (phx >= 0) {
            float m[4][8];
            phase_mass(phx, m);
            double mine = 0.0;
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 8; ++e) mine += (double)m[q][e];
            double incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(HS_FULL_MASK, incl, o);
                if (lane >= o) incl += up;
            }
            if (lane == 31) s_scan[warp] = incl;
            walk_sync();
            double run = before_ph + (incl - mine);
            for (int w2 = 0; w2 < warp; ++w2) run += s_scan[w2];
            if (run <= goal && run + mine > goal) {              // the crossing lies in this thread's tokens
                bool found = false;
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        run += (double)m[q][e];
                        if (!found && run > goal) {
                            found = true;
                            atomicMin(&s_pick[0], (phx * phase_vecs + tid * 4 + q) * ve + e);
                        }
                    }
            }
        }
        if (last_pos >= 0) atomicMax(&s_pick[1], last_pos);
        walk_sync();
        bonus = s_pick[0] != 0x7fffffff ? s_pick[0] : max(s_pick[1], 0);
        break;
    }
    if (tid == 0) {
        p.out.accept_len[b] = len;
        p.out.bonus_token[b] = bonus;
        p.out.terminal_rank[b] = p.pr.keep_rank[koff + cur];
        p.out.status[b] = HS_OK;
    }
}

template <bool BF16>
__global__ void __launch_bounds__(HS_ROW_THREADS, 4) accept_rows_kernel(const __grid_constant__ AcceptParams p) {
    constexpr int VE = BF16 ? 8 : 4;
    constexpr int VPT = HS_ROW_VPT;
    __shared__ float s_w[8][2];
    __shared__ unsigned long long s_key[8];
    __shared__ __align__(16) uint4 s_cl[8];       // clustered launch, first CTA of a row: the chunks' results
    __shared__ int s_flag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x, k = blockIdx.y, which = blockIdx.z;   // which: 0 target, 1 draft
    pdl_launch_dependents();
    // First half of a cluster barrier: when it completes every CTA of the row's cluster runs, and its shared memory may
    // be written from outside.  (The CTAs of a cluster take every early exit below together: same row, same sequence.)
    if (p.clustered) cluster_arrive();
    pdl_wait();                            // the pruned tree and the logits come from upstream
    // sequences that kept nothing (flagged upstream) get their empty result from CTA (0, b, 0)
    if (chunk == 0 && which == 0 && k < p.batch && (p.pr.n_keep[k] <= 0 || p.pr.status[k] != 0)) {
        const int cap = p.out.path_cap;
        for (int j = tid; j < cap; j += HS_ROW_THREADS) {
            p.out.path_nodes[k * cap + j] = -1;
            p.out.path_compact[k * cap + j] = -1;
            p.out.path_tokens[k * cap + j] = -1;
        }
        if (tid == 0) {
            p.out.accept_len[k] = 0; p.out.bonus_token[k] = -1; p.out.terminal_rank[k] = -1;
            p.out.status[k] = p.pr.status[k] != 0 ? p.pr.status[k] : HS_ERR_BAD_TREE;
        }
    }
    if (k >= p.pr.keep_off[p.batch]) return;
    int lo = 0, hi = p.batch;                     // sequence of kept node k
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (p.pr.keep_off[mid] <= k) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int i = k - p.pr.keep_off[b];
    const int nk = p.pr.n_keep[b];
    const int md = p.mode[b];
    const bool sampling = md != HS_ACCEPT_GREEDY;          // the row's normaliser is needed
    if (which == 1) {
        if (md != HS_ACCEPT_REJECTION) return;
        int internal = 0;                         // does kept node i have a kept child?
        for (int j = i + 1 + tid; j < nk; j += HS_ROW_THREADS)
            internal |= (p.pr.new_parent[p.pr.keep_off[b] + j] == i);
        if (!__syncthreads_or(internal)) return;
    }
    const int orig_row = p.node_off[b] + p.pr.keep_idx[k];
    const int row = which == 1 ? orig_row : (p.target_layout == HS_ROWS_ORIGINAL ? orig_row : k);
    const char* rowp = (const char*)(which == 1 ? p.draft : p.target) + (size_t)row * p.row_stride * (BF16 ? 2 : 4);
    const int v0 = chunk * p.chunk_vecs;
    const int v1 = min(v0 + p.chunk_vecs, p.nvec);

    uint4 d[VPT];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        int v = v0 + tid + j * HS_ROW_THREADS;
        if (v < v1) {
            d[j] = __ldcs((const uint4*)(rowp) + v);
        } else {
            unsigned int ninf = BF16 ? 0xff80ff80u : 0xff800000u;
            d[j] = make_uint4(ninf, ninf, ninf, ninf);
        }
    }
    // per-thread best (value, lowest index)
    float tmax = -CUDART_INF_F;
    int targ = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        float x[8];
        unpack_v<BF16>(d[j], x);
        int base = (v0 + tid + j * HS_ROW_THREADS) * VE;
#pragma unroll
        for (int e = 0; e < VE; ++e) {
            bool in = base + e < p.vocab;
            if (in && x[e] > tmax) { tmax = x[e]; targ = base + e; }   // ascending index: strict > keeps the lowest
        }
    }
    unsigned long long key = (targ == 0x7fffffff) ? 0ull : make_key(tmax, targ);
    key = warp_max_u64(key);
    float s = 0.f;
    if (sampling) {
        const float invT = LOG2E / p.temperature[b];
        const float nml = (tmax == -CUDART_INF_F) ? 0.f : -tmax * invT;
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            float x[8];
            unpack_v<BF16>(d[j], x);
            int base = (v0 + tid + j * HS_ROW_THREADS) * VE;
#pragma unroll
            for (int e = 0; e < VE; ++e)
                if (base + e < p.vocab) s += ex2a(fmaf(fmaxf(x[e], -1e30f), invT, nml));
        }
        float wm = warp_max(tmax);
        float f = (tmax == -CUDART_INF_F) ? 0.f : ex2a((tmax - wm) * invT);
        s = warp_sum(s * f);
        if (lane == 0) { s_w[warp][0] = wm; s_w[warp][1] = s; }
    }
    if (lane == 0) s_key[warp] = key;
    __syncthreads();
    if (p.clustered) cluster_wait();
    if (tid == 0) {
        unsigned long long best = s_key[0];
        for (int w = 1; w < 8; ++w) best = s_key[w] > best ? s_key[w] : best;
        float M = -CUDART_INF_F, S = 0.f;
        if (sampling) {
            const float invT = LOG2E / p.temperature[b];
            for (int w = 0; w < 8; ++w) M = fmaxf(M, s_w[w][0]);
            for (int w = 0; w < 8; ++w)
                S += (s_w[w][0] == -CUDART_INF_F) ? 0.f : s_w[w][1] * ex2a((s_w[w][0] - M) * invT);
        }
        if (p.clustered) {
            // the chunk's result goes into slot `chunk` of the first CTA of the row's cluster (posted stores through
            // distributed shared memory; the cluster barrier below makes them visible there)
            const unsigned int dst = cluster_map_addr(smem_u32(&s_cl[chunk]), 0);
            asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"((unsigned int)best),
                         "r"((unsigned int)(best >> 32)), "r"(__float_as_uint(M)), "r"(__float_as_uint(S)) : "memory");
            s_flag = (chunk == 0);
        } else {
            p.partials[((size_t)which * p.part_rows + k) * p.chunks + chunk] =
                make_uint4((unsigned int)best, (unsigned int)(best >> 32), __float_as_uint(M), __float_as_uint(S));
            // one release-acquire arrival at device scope: this thread's partial is visible to whoever arrives last,
            // and the last one (then, behind the barrier below, its whole CTA) sees all of them
            int* cnt = &p.row_cnt[which * HS_MAX_ROWS + k];
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(cnt) : "memory");
            s_flag = (old == p.chunks - 1);
            if (s_flag) *cnt = 0;
        }
    }
    if (p.clustered) {
        cluster_arrive();
        cluster_wait();
    } else {
        __syncthreads();
    }
    if (!s_flag) return;
    if (warp == 0) {
    // the CTA that merges the row (chunks <= 32, one lane per chunk)
    unsigned long long ck = 0ull;
    float cm = -CUDART_INF_F, cs = 0.f;
    if (lane < p.chunks) {
        const uint4 q = p.clustered ? s_cl[lane] : __ldcg(&p.partials[((size_t)which * p.part_rows + k) * p.chunks + lane]);
        ck = ((unsigned long long)q.y << 32) | q.x;
        cm = __uint_as_float(q.z);
        cs = __uint_as_float(q.w);
    }
    unsigned long long best = warp_max_u64(ck);
    float M = warp_max(cm), S = 0.f;
    if (sampling) {
        const float invT = LOG2E / p.temperature[b];
        S = warp_sum((cm == -CUDART_INF_F) ? 0.f : cs * ex2a((cm - M) * invT));
    }
    if (lane == 0) {
        if (which == 0) {
            p.ro.tgt_arg[k] = key_index(best);
            p.ro.tgt_ms[k] = make_float2(M, S);
        } else {
            p.ro.drf_ms[k] = make_float2(M, S);
        }
    }
    }
    // ---- greedy sequences finish here: the last target row of a sequence to be merged walks its tree ------
    if (md == HS_ACCEPT_REJECTION && !p.have_draft && which == 0 && i == 0) {
        // rejection sampling needs the draft distribution: the caller passed none
        const int cap = p.out.path_cap;
        for (int j = tid; j < cap; j += HS_ROW_THREADS) {
            p.out.path_nodes[b * cap + j] = -1;
            p.out.path_compact[b * cap + j] = -1;
            p.out.path_tokens[b * cap + j] = -1;
        }
        if (tid == 0) {
            p.out.accept_len[b] = 0; p.out.bonus_token[b] = -1; p.out.terminal_rank[b] = -1;
            p.out.status[b] = HS_ERR_INVALID_ARG;
        }
    }
    if (which != 0 || md == HS_ACCEPT_REJECTION) return;
    __syncthreads();
    if (tid == 0) {                                // (the thread that wrote the row's merged result)
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(&p.seq_cnt[b]) : "memory");
        s_flag = (old == nk - 1);
        if (s_flag) p.seq_cnt[b] = 0;
    }
    __syncthreads();
    if (s_flag) {
        if (md == HS_ACCEPT_GREEDY) greedy_walk(p, b);
        else deterministic_walk(p, b);
    }
}

// ================================================================================================================
// The row pass as a stream (launches whose rows do not fit the latency-bound regime of the chunk kernel)
// ================================================================================================================
// The rows to read - the target row of every kept node, then the draft row of every kept internal node of a
// sequence in rejection mode - form one stream of 16-byte vectors that is cut into equal contiguous shares, one per
// CTA, one CTA per SM.  Which rows those are is only known on the device (the pruned tree comes from the kernel
// ahead), so every CTA derives the list itself: a bit per kept node for "needs its draft row", a prefix of the bit
// counts, the share bounds from the total.  A producer warp looks the rows of the share up (32 at a time, one per
// lane) and brings them on chip in items of up to 32 KiB (bulk copies into a ring of shared-memory slots); sixteen
// consumer warps reduce each item in one pass: arg-max with the lowest index on ties (packed bf16 maxima with a
// 16-bit position code per half-lane, decoded once per row segment) and, for sampling sequences, max and
// sum e^((x-max)/T).  A row that lies in several shares leaves partials; the last share to arrive merges them.
// Sequences that finish in the row pass (greedy, deterministic proposals) are walked after the CTA's share by the
// CTA that merged their last target row.
#define AS_CONSUMERS 512
#define AS_NW (AS_CONSUMERS / 32)
#define AS_THREADS (AS_CONSUMERS + 32)
#define AS_ITEM_VECS 2048
#define AS_VPT (AS_ITEM_VECS / AS_CONSUMERS)
#define AS_SLOTS 5
#define AS_MAX_SEGS 32
#define AS_ROW_RING 64
#define AS_SMEM_BYTES (AS_SLOTS * AS_ITEM_VECS * 16 + 128)
#define AS_MIN_BYTES ((size_t)48 << 20)       // smaller launches go to the chunk kernel

struct WorkRow {          // one row of the stream, as looked up by the producer warp
    const char* ptr;
    int k;                // kept node (index into the compacted arrays)
    int b;                // its sequence
    int which;            // 0 target row, 1 draft row
    int mode;
    float invT;           // log2(e) / temperature
    int nk;               // kept nodes of the sequence
};

template <bool BF16>
__global__ void __launch_bounds__(AS_THREADS, 1) accept_stream_kernel(const __grid_constant__ AcceptParams p) {
    constexpr int VE = BF16 ? 8 : 4;
    constexpr int NWORDS = HS_MAX_ROWS / 32;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ unsigned long long s_full[AS_SLOTS], s_empty[AS_SLOTS];
    __shared__ unsigned int s_bits[NWORDS];          // kept node -> its draft row is part of the stream
    __shared__ int s_pref[NWORDS + 1];               // set bits ahead of each word
    __shared__ WorkRow s_rows[AS_ROW_RING];
    __shared__ unsigned long long s_wkey[2][AS_NW];
    __shared__ float2 s_wms[2][AS_NW];
    __shared__ unsigned short s_pending[HS_MAX_BATCH];   // sequences this CTA has to walk
    __shared__ int s_npending;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned int slots0 = (smem_u32(s_dyn) + 127u) & ~127u;
    const unsigned char* slots_gen = s_dyn + (slots0 - smem_u32(s_dyn));
    const size_t esz = BF16 ? 2 : 4;

    if (tid == 0) {
        for (int s = 0; s < AS_SLOTS; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), AS_NW);
        }
        mbar_init_fence();
        s_npending = 0;
    }
    for (int i = tid; i < NWORDS; i += AS_THREADS) s_bits[i] = 0u;
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();                            // the pruned tree and the logits come from upstream

    // ---- the rows of the stream --------------------------------------------------------------------------------
    const int T = min(p.pr.keep_off[p.batch], p.part_rows);
    if (p.have_draft) {
        for (int b = warp; b < p.batch; b += AS_THREADS / 32) {
            if (p.mode[b] != HS_ACCEPT_REJECTION) continue;
            const int koff = p.pr.keep_off[b], nk = p.pr.n_keep[b];
            for (int j = 1 + lane; j < nk; j += 32) {
                const int par = p.pr.new_parent[koff + j];
                const int k = koff + par;
                if (par >= 0 && par < j && k < T) atomicOr(&s_bits[k >> 5], 1u << (k & 31));
            }
        }
    }
    // sequences that kept nothing (flagged upstream) and sequences in rejection mode without draft logits get their
    // result here, shared out over the warps of the grid
    for (int b = blockIdx.x * (AS_THREADS / 32) + warp; b < p.batch; b += gridDim.x * (AS_THREADS / 32)) {
        const int st = p.pr.status[b];
        const bool empty = p.pr.n_keep[b] <= 0 || st != 0;
        const bool nodraft = !empty && p.mode[b] == HS_ACCEPT_REJECTION && !p.have_draft;
        if (empty || nodraft) {
            const int cap = p.out.path_cap;
            for (int j = lane; j < cap; j += 32) {
                p.out.path_nodes[b * cap + j] = -1;
                p.out.path_compact[b * cap + j] = -1;
                p.out.path_tokens[b * cap + j] = -1;
            }
            if (lane == 0) {
                p.out.accept_len[b] = 0; p.out.bonus_token[b] = -1; p.out.terminal_rank[b] = -1;
                p.out.status[b] = empty ? (st != 0 ? st : HS_ERR_BAD_TREE) : HS_ERR_INVALID_ARG;
            }
        }
    }
    __syncthreads();
    if (warp == 0) {
        constexpr int WPL = NWORDS / 32;
        int c = 0;
#pragma unroll
        for (int i = 0; i < WPL; ++i) c += __popc(s_bits[lane * WPL + i]);
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(HS_FULL_MASK, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - c;
#pragma unroll
        for (int i = 0; i < WPL; ++i) {
            s_pref[lane * WPL + i] = run;
            run += __popc(s_bits[lane * WPL + i]);
        }
        if (lane == 31) s_pref[NWORDS] = run;
    }
    __syncthreads();
    const int W = T + s_pref[NWORDS];
    const long long total = (long long)W * p.nvec;
    long long per = (total + gridDim.x - 1) / gridDim.x;
    per = max(per, (long long)((p.nvec + (AS_MAX_SEGS - 2) - 1) / (AS_MAX_SEGS - 2)));   // a row in at most AS_MAX_SEGS shares
    per = max(per, (long long)AS_ITEM_VECS);
    const long long g0 = (long long)blockIdx.x * per, g1 = min(g0 + per, total);
    if (g0 >= g1) return;
    const int w_first = (int)(g0 / p.nvec), w_last = (int)((g1 - 1) / p.nvec);

    auto lookup = [&](int w) -> WorkRow {
        WorkRow r;
        if (w < T) {
            r.k = w; r.which = 0;
        } else {
            const int rnk = w - T;                        // the rnk-th set bit
            int lo = 0, hi = NWORDS;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s_pref[mid] <= rnk) lo = mid; else hi = mid;
            }
            r.k = lo * 32 + (int)__fns(s_bits[lo], 0, rnk - s_pref[lo] + 1);
            r.which = 1;
        }
        int lo = 0, hi = p.batch;                         // the last b with keep_off[b] <= k (skips empty sequences)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.pr.keep_off[mid] <= r.k) lo = mid; else hi = mid;
        }
        r.b = lo;
        r.nk = p.pr.n_keep[lo];
        r.mode = p.mode[lo];
        r.invT = LOG2E / p.temperature[lo];
        const int orig_row = p.node_off[lo] + p.pr.keep_idx[r.k];
        const int row = r.which == 1 ? orig_row : (p.target_layout == HS_ROWS_ORIGINAL ? orig_row : r.k);
        r.ptr = (const char*)(r.which == 1 ? p.draft : p.target) + (size_t)row * p.row_stride * esz;
        return r;
    };

    if (warp == AS_NW) {
        // ---- producer warp: lane 0 walks the share item by item; all lanes look rows up, 32 rows at a time ---------
        long long g = g0;
        int it = 0, slot = 0;
        unsigned int epar = 1u;              // parity of the slot's `empty` barrier before its first completion
        for (int w = w_first; w <= w_last; ++w) {
            const int rl = w - w_first;
            if ((rl & 31) == 0) {
                // (the consumers are at most AS_SLOTS + 1 rows behind: the other half of the ring)
                if (w + lane <= w_last) s_rows[(rl + lane) % AS_ROW_RING] = lookup(w + lane);
                __syncwarp();
            }
            if (lane == 0) {
                const char* ptr = s_rows[rl % AS_ROW_RING].ptr;
                const long long row_g0 = (long long)w * p.nvec;
                int v = (int)(g - row_g0);
                const int v_end = (int)(min(g1, row_g0 + p.nvec) - row_g0);
                while (v < v_end) {
                    const int len = min(AS_ITEM_VECS, v_end - v);
                    if (it >= AS_SLOTS) mbar_wait(smem_u32(&s_empty[slot]), epar, p.err);
                    const unsigned int bar = smem_u32(&s_full[slot]);
                    // (the arrival below also publishes the row table to the consumers that wait on this barrier)
                    mbar_expect_tx(bar, (unsigned int)len * 16u);
                    bulk_load(slots0 + (unsigned int)slot * (AS_ITEM_VECS * 16), ptr + (size_t)v * 16, (unsigned int)len * 16u, bar);
                    v += len;
                    ++it;
                    if (++slot == AS_SLOTS) { slot = 0; epar ^= 1u; }
                }
                g = row_g0 + v_end;
            }
            __syncwarp();
        }
        return;
    }

    // ---- consumers -------------------------------------------------------------------------------------------------
    const unsigned int ninf = BF16 ? 0xff80ff80u : 0xff800000u;
    int cslot = 0;                 // slot of the next item and the parity of its `full` barrier (the producer fills
    unsigned int cpar = 0u;        // the slots round-robin in the same order)
    int seg = 0;
    long long g = g0;
    while (g < g1) {
        // ---- one segment: the part of this share inside row w of the stream --------------------------------------
        const int w = (int)(g / p.nvec);
        const long long row_g0 = (long long)w * p.nvec;
        const int sv0 = (int)(g - row_g0);
        const int sv1 = (int)(min(g1, row_g0 + p.nvec) - row_g0);
        mbar_wait(smem_u32(&s_full[cslot]), cpar, p.err);      // the row's first item; the row table entry with it
        const WorkRow r = s_rows[(w - w_first) % AS_ROW_RING];
        const bool sampling = r.mode != HS_ACCEPT_GREEDY;      // the row's normaliser is needed
        const bool want_arg = r.which == 0;
        unsigned int bm = ninf, bc = 0u;      // bf16: running maximum and position code of the two half-lanes
        float m_f = -CUDART_INF_F;            // f32: running maximum and its position code
        unsigned int c_f = 0u;
        float m_t = -CUDART_INF_F;            // maximum the sums are relative to
        float2 s2 = make_float2(0.f, 0.f);
        int it = 0;
        for (int v = sv0; v < sv1; ++it) {
            const int len = min(AS_ITEM_VECS, sv1 - v);
            const int slot = cslot;
            mbar_wait(smem_u32(&s_full[slot]), cpar, p.err);
            if (++cslot == AS_SLOTS) { cslot = 0; cpar ^= 1u; }
            const uint4* st = reinterpret_cast<const uint4*>(slots_gen + (size_t)slot * (AS_ITEM_VECS * 16));
            uint4 d[AS_VPT];
            if (len == AS_ITEM_VECS) {
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) d[j] = st[tid + j * AS_CONSUMERS];
            } else {
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) {
                    const int vl = tid + j * AS_CONSUMERS;
                    d[j] = (vl < len) ? st[vl] : make_uint4(ninf, ninf, ninf, ninf);
                }
            }
            if (v + len == p.nvec && p.nvec * VE != p.vocab) {                // the row's last vector runs past vocab
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) {
                    if (v + tid + j * AS_CONSUMERS == p.nvec - 1) {
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
            // maxima (target rows: with the position of the first occurrence; items, vectors and words are taken in
            // ascending token order and only a strictly larger value replaces the running one)
            if (BF16) {
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) {
                    const unsigned int* wd = reinterpret_cast<const unsigned int*>(&d[j]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const __nv_bfloat162 x2 = *reinterpret_cast<const __nv_bfloat162*>(&wd[q]);
                        const __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&bm);
                        if (want_arg) {
                            const unsigned int gt = __hgt2_mask(x2, m2);
                            const unsigned int cc = ((unsigned int)(it << 4 | j << 2 | q)) * 0x00010001u;
                            bc = (bc & ~gt) | (cc & gt);
                        }
                        const __nv_bfloat162 n2 = __hmax2(m2, x2);
                        bm = *reinterpret_cast<const unsigned int*>(&n2);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) {
                    const unsigned int* wd = reinterpret_cast<const unsigned int*>(&d[j]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float x = __uint_as_float(wd[e]);
                        if (x > m_f) { m_f = x; c_f = (unsigned int)(it << 4 | j << 2 | e); }
                    }
                }
            }
            if (sampling) {
                const float imax = BF16 ? fmaxf(bf16_lo(bm), bf16_hi(bm)) : m_f;
                if (imax > m_t) {                     // the thread's maximum grows: rescale its sum
                    const float f = (m_t == -CUDART_INF_F) ? 0.f : ex2a((m_t - imax) * r.invT);
                    s2.x *= f; s2.y *= f;
                    m_t = imax;
                }
                const float nml = (m_t == -CUDART_INF_F) ? 0.f : -m_t * r.invT;
                const float2 l2 = make_float2(r.invT, r.invT), n2 = make_float2(nml, nml);
                const unsigned int floor2 = 0xf149f149u;  // bf16 pair of -1e30: keeps 0 * x finite for x = -inf
#pragma unroll
                for (int j = 0; j < AS_VPT; ++j) {
                    const unsigned int* wd = reinterpret_cast<const unsigned int*>(&d[j]);
                    if (BF16) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const __nv_bfloat162 cl = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&wd[q]),
                                                             *reinterpret_cast<const __nv_bfloat162*>(&floor2));
                            const unsigned int cw = *reinterpret_cast<const unsigned int*>(&cl);
                            const float2 t = fma2_ftz(make_float2(bf16_lo(cw), bf16_hi(cw)), l2, n2);
                            s2 = add2_ftz(s2, make_float2(ex2a(t.x), ex2a(t.y)));
                        }
                    } else {
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const float2 x = make_float2(fmaxf(__uint_as_float(wd[2 * q]), -1e30f),
                                                         fmaxf(__uint_as_float(wd[2 * q + 1]), -1e30f));
                            const float2 t = fma2_ftz(x, l2, n2);
                            s2 = add2_ftz(s2, make_float2(ex2a(t.x), ex2a(t.y)));
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
            v += len;
        }
        // ---- end of the segment: the thread's candidates become (value, lowest index) keys ------------------------
        unsigned long long key = 0ull;
        if (want_arg) {
            if (BF16) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float val = h ? bf16_hi(bm) : bf16_lo(bm);
                    const unsigned int code = (bc >> (16 * h)) & 0xffffu;
                    if (val > -CUDART_INF_F) {
                        const int vec = sv0 + (int)(code >> 4) * AS_ITEM_VECS + tid + (int)((code >> 2) & 3u) * AS_CONSUMERS;
                        const unsigned long long kk = make_key(val, vec * 8 + 2 * (int)(code & 3u) + h);
                        key = kk > key ? kk : key;
                    }
                }
            } else if (m_f > -CUDART_INF_F) {
                const int vec = sv0 + (int)(c_f >> 4) * AS_ITEM_VECS + tid + (int)((c_f >> 2) & 3u) * AS_CONSUMERS;
                key = make_key(m_f, vec * 4 + (int)(c_f & 3u));
            }
            key = warp_max_u64(key);
        }
        float wm = -CUDART_INF_F, ws = 0.f;
        if (sampling) {
            wm = warp_max(m_t);
            const float f = (m_t == -CUDART_INF_F) ? 0.f : ex2a((m_t - wm) * r.invT);
            ws = warp_sum((s2.x + s2.y) * f);
        }
        if (lane == 0) { s_wkey[seg & 1][warp] = key; s_wms[seg & 1][warp] = make_float2(wm, ws); }
        named_bar_sync(1, AS_CONSUMERS);
        if (warp == 0) {
            // the other warps are already on their way to the next segment
            unsigned long long best = warp_max_u64(lane < AS_NW ? s_wkey[seg & 1][lane] : 0ull);
            const float2 ms = lane < AS_NW ? s_wms[seg & 1][lane] : make_float2(-CUDART_INF_F, 0.f);
            float M = warp_max(ms.x);
            float S = sampling ? warp_sum(ms.x == -CUDART_INF_F ? 0.f : ms.y * ex2a((ms.x - M) * r.invT)) : 0.f;
            const int c_first = (int)(row_g0 / per);
            const int nseg = (int)((row_g0 + p.nvec - 1) / per) - c_first + 1;
            bool mine = true;                     // this warp holds the row's final result
            if (nseg > 1) {
                // a share holds at most two partial rows: the one that began in an earlier share, the one that goes on
                auto slot_of = [&](int c) { return 2 * c + (row_g0 < (long long)c * per ? 0 : 1); };
                int last = 0;
                if (lane == 0) {
                    p.partials[slot_of(blockIdx.x)] =
                        make_uint4((unsigned int)best, (unsigned int)(best >> 32), __float_as_uint(M), __float_as_uint(S));
                    // one release-acquire arrival at device scope: the partial is visible to whoever arrives last
                    int old;
                    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(&p.row_cnt[w]) : "memory");
                    last = old == nseg - 1;
                    if (last) p.row_cnt[w] = 0;
                }
                mine = __shfl_sync(HS_FULL_MASK, last, 0) != 0;
                if (mine) {
                    unsigned long long ck = 0ull;
                    float cm = -CUDART_INF_F, cs = 0.f;
                    if (lane < nseg) {
                        const uint4 q = __ldcg(&p.partials[slot_of(c_first + lane)]);
                        ck = ((unsigned long long)q.y << 32) | q.x;
                        cm = __uint_as_float(q.z);
                        cs = __uint_as_float(q.w);
                    }
                    best = warp_max_u64(ck);
                    M = warp_max(cm);
                    S = sampling ? warp_sum(cm == -CUDART_INF_F ? 0.f : cs * ex2a((cm - M) * r.invT)) : 0.f;
                }
            }
            if (mine && lane == 0) {
                if (r.which == 0) {
                    p.ro.tgt_arg[r.k] = key_index(best);
                    p.ro.tgt_ms[r.k] = make_float2(M, S);
                    if (r.mode != HS_ACCEPT_REJECTION) {
                        // greedy sequences and deterministic proposals finish in this kernel: the CTA that completes a
                        // sequence's last target row walks its tree once its own share is done
                        int old;
                        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(&p.seq_cnt[r.b]) : "memory");
                        if (old == r.nk - 1) {
                            p.seq_cnt[r.b] = 0;
                            s_pending[s_npending++] = (unsigned short)r.b;
                        }
                    }
                } else {
                    p.ro.drf_ms[r.k] = make_float2(M, S);
                }
            }
        }
        ++seg;
        g = row_g0 + sv1;
    }
    named_bar_sync(1, AS_CONSUMERS);          // warp 0 has finished its last row: the list of walks is complete
    if (tid < HS_ROW_THREADS) {
        const int npend = s_npending;
        for (int i = 0; i < npend; ++i) {
            const int b = s_pending[i];
            if (p.mode[b] == HS_ACCEPT_GREEDY) greedy_walk(p, b);
            else deterministic_walk(p, b);
            walk_sync();                       // the walks' shared arrays are free again
        }
    }
}

// ---- the walk ----------------------------------------------------------------------------------

__device__ __forceinline__ float load_logit(const void* base, int is_bf16, size_t off) {
    return is_bf16 ? __bfloat162float(((const __nv_bfloat16*)base)[off]) : ((const float*)base)[off];
}

// This CTA's slice of the current node's target row p and draft row q: vectors [v0, v0 + nv) of the row, read
// through pointers to shared memory (staged by bulk copies) or to the rows themselves.
struct RowSlice {
    const uint4* p;
    const uint4* q;       // NULL when only p is there
    int v0, nv;
};

// All-gather of one 64-bit value per CTA over the cluster: warp 0 of every CTA stores its value into slot `rank` of the
// exchange buffer of all WALK_CLUSTER CTAs (posted stores through distributed shared memory, lane r to CTA r), one
// cluster barrier makes them visible, every CTA then reads its own copy.  The buffers alternate from one exchange to
// the next (s_x[xch & 1]), so one barrier per exchange is enough: a buffer is written again only two exchanges later,
// after a barrier that every CTA reaches with its reads done.  `v` must be valid in warp 0.
__device__ __forceinline__ void cluster_allgather(unsigned long long v, unsigned long long (*s_x)[WALK_CLUSTER],
                                                  unsigned int& xch, unsigned int rank) {
    unsigned long long* buf = s_x[xch & 1u];
    ++xch;
    if (threadIdx.x < WALK_CLUSTER) {
        const unsigned int remote = cluster_map_addr(smem_u32(&buf[rank]), threadIdx.x);
        asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(remote), "l"(v) : "memory");
    }
    cluster_arrive();
    cluster_wait();
}

// Sum over this CTA's share of the vocabulary of max(p_v - c q_v, 0), then over the cluster.
// Every CTA returns the same value (fixed summation order).
__device__ double cluster_residual_sum(const AcceptParams& p, unsigned int rank, const RowSlice& rs,
                                       float pm, float ips, float qm, float iqs, float invT,
                                       float c, double* s_part, unsigned long long (*s_x)[WALK_CLUSTER], unsigned int& xch) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ve = p.is_bf16 ? 8 : 4;
    float acc = 0.f;
    for (int v = tid; v < rs.nv; v += WALK_THREADS) {
        uint4 a = rs.p[v], bq = rs.q[v];
        float x[8], y[8];
        if (p.is_bf16) { unpack_v<true>(a, x); unpack_v<true>(bq, y); }
        else { unpack_v<false>(a, x); unpack_v<false>(bq, y); }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            if (e < ve && (rs.v0 + v) * ve + e < p.vocab) {
                float pv = exp2f((fmaxf(x[e], -1e30f) - pm) * invT) * ips;
                float qv = exp2f((fmaxf(y[e], -1e30f) - qm) * invT) * iqs;
                acc += fmaxf(pv - c * qv, 0.f);
            }
        }
    }
    double w = warp_sum_d((double)acc);
    if (lane == 0) s_part[warp] = w;
    __syncthreads();
    double t = 0.0;
    if (warp == 0) {                                   // the warps' sums in a fixed order, known to every lane of warp 0
        for (int i = 0; i < WALK_THREADS / 32; ++i) t += s_part[i];
    }
    const unsigned long long* got = s_x[xch & 1u];
    cluster_allgather((unsigned long long)__double_as_longlong(t), s_x, xch, rank);
    double tot = 0.0;
    for (unsigned int r = 0; r < WALK_CLUSTER; ++r) tot += __longlong_as_double((long long)got[r]);
    return tot;
}

// Inverse-CDF draw from max(p - c q, 0) in token order: smallest j whose running sum exceeds
// u * total; if rounding leaves none, the last token with positive mass.  rs.q may be NULL (c = 0).
// A CTA covers the tokens of its slice, a thread a contiguous run of them; running sums in double.
__device__ int cluster_inverse_cdf(const AcceptParams& p, unsigned int rank, const RowSlice& rs,
                                   float pm, float ips, float qm, float iqs, float invT,
                                   float c, float u, double* s_scan, unsigned long long (*s_x)[WALK_CLUSTER],
                                   unsigned int& xch, int* s_pick) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ve = p.is_bf16 ? 8 : 4;
    const int c0 = rs.v0 * ve, c1 = min(c0 + rs.nv * ve, p.vocab);
    const int seg = (max(c1 - c0, 0) + WALK_THREADS - 1) / WALK_THREADS;
    const int t0 = min(c0 + tid * seg, c1), t1 = min(t0 + seg, c1);
    auto mass = [&](int j) -> float {
        float pv = exp2f((fmaxf(load_logit(rs.p, p.is_bf16, j - c0), -1e30f) - pm) * invT) * ips;
        if (rs.q == nullptr) return pv;
        float qv = exp2f((fmaxf(load_logit(rs.q, p.is_bf16, j - c0), -1e30f) - qm) * invT) * iqs;
        return fmaxf(pv - c * qv, 0.f);
    };
    double mine = 0.0;
    int last_pos = -1;
    for (int j = t0; j < t1; ++j) {
        float r = mass(j);
        mine += (double)r;
        if (r > 0.f) last_pos = j;
    }
    if (tid == 0) { s_pick[0] = 0x7fffffff; s_pick[1] = -1; }
    // exclusive scan over the CTA's threads: inclusive shuffle scan inside a warp, then the warps' totals in order
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(HS_FULL_MASK, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    double wbefore = 0.0, ctot = 0.0;
#pragma unroll
    for (int w = 0; w < WALK_THREADS / 32; ++w) {
        const double t = s_scan[w];
        if (w < warp) wbefore += t;
        ctot += t;
    }
    const unsigned long long* got = s_x[xch & 1u];
    cluster_allgather((unsigned long long)__double_as_longlong(ctot), s_x, xch, rank);
    double before = 0.0, total = 0.0;
    for (unsigned int r = 0; r < WALK_CLUSTER; ++r) {
        const double v = __longlong_as_double((long long)got[r]);
        if (r < rank) before += v;
        total += v;
    }
    const double goal = (double)u * total;
    double run = before + wbefore + (incl - mine);
    if (run <= goal && run + mine > goal) {          // the crossing lies in this thread's segment
        for (int j = t0; j < t1; ++j) {
            run += (double)mass(j);
            if (run > goal) { atomicMin(&s_pick[0], j); break; }
        }
    }
    if (last_pos >= 0) atomicMax(&s_pick[1], last_pos);
    __syncthreads();
    // the CTAs' (crossing, last positive token) pairs, one 64-bit word each
    const unsigned long long mine2 = ((unsigned long long)(unsigned int)s_pick[0] << 32) | (unsigned int)s_pick[1];
    const unsigned long long* got2 = s_x[xch & 1u];
    cluster_allgather(mine2, s_x, xch, rank);
    int pick = 0x7fffffff, lastp = -1;
    for (unsigned int r = 0; r < WALK_CLUSTER; ++r) {
        pick = min(pick, (int)(unsigned int)(got2[r] >> 32));
        lastp = max(lastp, (int)(unsigned int)(got2[r] & 0xffffffffu));
    }
    return pick != 0x7fffffff ? pick : max(lastp, 0);
}

__global__ void __cluster_dims__(WALK_CLUSTER, 1, 1) __launch_bounds__(WALK_THREADS, 1)
accept_walk_kernel(const AcceptParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) unsigned char s_rows[];    // staged: this CTA's slices of p and q, `per` vectors each
    __shared__ unsigned long long s_bar;
    __shared__ double s_part[WALK_THREADS / 32];
    __shared__ double s_scan[WALK_THREADS / 32];
    __shared__ unsigned long long s_x[2][WALK_CLUSTER];    // all-gather buffers of the cluster exchanges
    unsigned int xch = 0;                  // exchanges through s_cta so far
    __shared__ int s_pick[2];
    const int tid = threadIdx.x;
    const int b = blockIdx.x / WALK_CLUSTER;
    const unsigned int rank = cluster.block_rank();
    pdl_launch_dependents();
    pdl_wait();                            // arg-max and normalisers come from the row pass
    const int koff = p.pr.keep_off[b];
    const int nk = p.pr.n_keep[b];
    const int nbase = p.node_off[b];
    const int cap = p.out.path_cap;
    const bool sampling = p.mode[b] == HS_ACCEPT_REJECTION;
    const size_t esz = p.is_bf16 ? 2 : 4;

    if (!sampling && nk > 0 && p.pr.status[b] == 0) return;      // greedy sequences were finished by the row pass
    if (rank == 0) {
        for (int j = tid; j < cap; j += WALK_THREADS) {
            p.out.path_nodes[b * cap + j] = -1;
            p.out.path_compact[b * cap + j] = -1;
            p.out.path_tokens[b * cap + j] = -1;
        }
    }
    if (nk <= 0 || p.pr.status[b] != 0) {
        if (rank == 0 && tid == 0) {
            p.out.accept_len[b] = 0; p.out.bonus_token[b] = -1; p.out.terminal_rank[b] = -1;
            p.out.status[b] = p.pr.status[b] != 0 ? p.pr.status[b] : HS_ERR_BAD_TREE;
        }
        return;
    }
    // This CTA's slice of a row: vectors [v0, v0 + nv).  The rows of the node the walk stands on are brought into
    // shared memory once (one bulk copy each, only when a residual or the final draw needs them) and serve every
    // rejection at that node and the final draw.
    const int per = (p.nvec + WALK_CLUSTER - 1) / WALK_CLUSTER;
    RowSlice rs;
    rs.v0 = rank * per;
    rs.nv = max(min(rs.v0 + per, p.nvec) - rs.v0, 0);
    rs.p = nullptr; rs.q = nullptr;
    const unsigned int bar = smem_u32(&s_bar);
    if (tid == 0 && p.staged) { mbar_init(bar, 1); mbar_init_fence(); }
    unsigned int stage_n = 0;
    int staged_node = -1;
    bool staged_q = false;
    auto stage = [&](int node, const char* prow, const char* qrow) {      // qrow may be NULL: only p
        if (staged_node == node && (staged_q || qrow == nullptr)) {
            if (qrow == nullptr) rs.q = nullptr;
            return;
        }
        staged_node = node; staged_q = qrow != nullptr;
        if (!p.staged) {
            rs.p = (const uint4*)prow + rs.v0;
            rs.q = qrow ? (const uint4*)qrow + rs.v0 : nullptr;
            return;
        }
        __syncthreads();                   // nobody still reads the rows of the previous node
        if (tid == 0) {
            const unsigned int bytes = (unsigned int)rs.nv * 16u;
            mbar_expect_tx(bar, qrow ? 2u * bytes : bytes);
            if (bytes) {
                bulk_load(smem_u32(s_rows), (const uint4*)prow + rs.v0, bytes, bar);
                if (qrow) bulk_load(smem_u32(s_rows) + (unsigned int)per * 16u, (const uint4*)qrow + rs.v0, bytes, bar);
            }
        }
        mbar_wait(bar, stage_n & 1u, p.err);
        ++stage_n;
        rs.p = (const uint4*)s_rows;
        rs.q = qrow ? (const uint4*)s_rows + per : nullptr;
    };
    // Every candidate's probability under its parent's target and draft row, its uniform and the normalisers of its
    // own rows, for all kept nodes at once (three dependent round trips in all instead of three per visited node);
    // the walk below then runs from shared memory until a rejection needs a vocabulary-wide residual sum.  Every CTA
    // of the cluster fetches the same values and takes the same decisions.
    __shared__ int s_par[HS_MAX_NODES], s_tok[HS_MAX_NODES], s_orig[HS_MAX_NODES];
    __shared__ float s_pt[HS_MAX_NODES], s_qt[HS_MAX_NODES], s_u[HS_MAX_NODES];
    __shared__ float2 s_pms[HS_MAX_NODES];
    // Also per node: its first (lowest-index) kept child and whether that child, tested first (residual = p), is
    // accepted - the common step of the walk then costs two shared-memory reads.
    __shared__ int s_first[HS_MAX_NODES];
    __shared__ unsigned char s_acc0[HS_MAX_NODES];
    const float T = p.temperature[b];
    const float invT = LOG2E / T;
    const int nkc = min(nk, HS_MAX_NODES);
    for (int j = tid; j < nkc; j += WALK_THREADS) s_first[j] = 0x7fffffff;
    __syncthreads();
    for (int j = tid; j < nkc; j += WALK_THREADS) {
        const int par = p.pr.new_parent[koff + j];
        const int orig = p.pr.keep_idx[koff + j];
        const int tok = p.token[nbase + orig];
        s_par[j] = par; s_tok[j] = tok; s_orig[j] = orig;
        s_pms[j] = p.ro.tgt_ms[koff + j];
        float pt = 0.f, qt = 0.f;
        if (par >= 0 && par < nkc) {
            const int porig = p.pr.keep_idx[koff + par];
            const int trow = p.target_layout == HS_ROWS_ORIGINAL ? nbase + porig : koff + par;
            const char* prow = (const char*)p.target + (size_t)trow * p.row_stride * esz;
            const char* qrow = (const char*)p.draft + (size_t)(nbase + porig) * p.row_stride * esz;
            const float2 pms = p.ro.tgt_ms[koff + par], qms = p.ro.drf_ms[koff + par];
            pt = exp2f((fmaxf(load_logit(prow, p.is_bf16, tok), -1e30f) - pms.x) * invT) * (1.f / pms.y);
            qt = exp2f((fmaxf(load_logit(qrow, p.is_bf16, tok), -1e30f) - qms.x) * invT) * (1.f / qms.y);
        }
        s_pt[j] = pt; s_qt[j] = qt;
        const float u = p.uniforms ? p.uniforms[nbase + orig] : philox_uniform(p.seed, p.offset, b, orig, 0);
        s_u[j] = u;
        // (the same expressions as in the sibling loop below with c = 0, W = 1: the same decision, bit for bit)
        const float r0 = fmaxf(pt - 0.f * qt, 0.f) / 1.f;
        const float a0 = qt > 0.f ? fminf(1.f, r0 / qt) : 1.f;
        s_acc0[j] = (par >= 0 && par < j && u < a0) ? 1 : 0;
        if (par >= 0 && par < j) atomicMin(&s_first[par], j);
    }
    __syncthreads();
    int cur = 0, len = 0, bonus = -1;
    {
        for (int step = 0; step < nkc; ++step) {
            if (rank == 0 && tid == 0 && len < cap) {
                p.out.path_compact[b * cap + len] = cur;
                p.out.path_nodes[b * cap + len] = s_orig[cur];
            }
            {
                const int j1 = s_first[cur];
                if (j1 != 0x7fffffff && s_acc0[j1]) {            // the first child is accepted: no residual is needed
                    if (rank == 0 && tid == 0 && len < cap) p.out.path_tokens[b * cap + len] = s_tok[j1];
                    cur = j1;
                    ++len;
                    continue;
                }
            }
            const int trow = p.target_layout == HS_ROWS_ORIGINAL ? nbase + s_orig[cur] : koff + cur;
            const int drow = nbase + s_orig[cur];
            const char* prow = (const char*)p.target + (size_t)trow * p.row_stride * esz;
            const char* qrow = (const char*)p.draft + (size_t)drow * p.row_stride * esz;
            const float2 pms = s_pms[cur];
            const float pm = pms.x, ips = 1.f / pms.y;
            float qm = 0.f, iqs = 0.f;
            bool have_q = false;
            float c = 0.f;
            double W = 1.0;
            int accepted = -1;
            bool tested = false;
            // the kept children of cur as bit masks (every warp finds them with four ballots instead of a serial scan)
            unsigned int kids[HS_MAX_NODES / 32];
#pragma unroll
            for (int w = 0; w < HS_MAX_NODES / 32; ++w) {
                const int j = w * 32 + (tid & 31);
                kids[w] = __ballot_sync(HS_FULL_MASK, j > cur && j < nkc && s_par[j] == cur);
            }
            for (;;) {                                           // siblings in index order
                int j = -1;
#pragma unroll
                for (int w = HS_MAX_NODES / 32 - 1; w >= 0; --w)
                    if (kids[w]) j = w * 32 + __ffs(kids[w]) - 1;
                if (j < 0) break;
#pragma unroll
                for (int w = 0; w < HS_MAX_NODES / 32; ++w)
                    if (j >> 5 == w) kids[w] &= kids[w] - 1;
                tested = true;
                const float pt = s_pt[j], qt = s_qt[j];
                const float r = fmaxf(pt - c * qt, 0.f) / (float)W;
                const float a = qt > 0.f ? fminf(1.f, r / qt) : 1.f;
                if (s_u[j] < a) { accepted = j; break; }
                if (!have_q) {
                    const float2 qms = p.ro.drf_ms[koff + cur];
                    qm = qms.x; iqs = 1.f / qms.y; have_q = true;
                }
                const float c_next = c + (float)W;
                stage(cur, prow, qrow);
                const double W_next = cluster_residual_sum(p, rank, rs, pm, ips, qm, iqs, invT,
                                                           c_next, s_part, s_x, xch);
                if (!(W_next > 0.0)) { c = 0.f; W = 1.0; tested = false; break; }   // p == q: fall back to p
                c = c_next; W = W_next;
            }
            if (accepted >= 0) {
                if (rank == 0 && tid == 0 && len < cap) p.out.path_tokens[b * cap + len] = s_tok[accepted];
                cur = accepted;
                ++len;
                continue;
            }
            const float ufin = p.uniforms ? p.uniforms[p.n_nodes_total + b] : philox_uniform(p.seed, p.offset, b, 0, 1);
            stage(cur, prow, (tested && c > 0.f) ? qrow : nullptr);
            bonus = cluster_inverse_cdf(p, rank, rs, pm, ips, qm, iqs,
                                        invT, c, ufin, s_scan, s_x, xch, s_pick);
            break;
        }
    }
    // (every store into a CTA's exchange buffers precedes a barrier that CTA takes part in: it may leave now)
    if (rank == 0 && tid == 0) {
        p.out.accept_len[b] = len;
        p.out.bonus_token[b] = bonus;
        p.out.terminal_rank[b] = p.pr.keep_rank[koff + cur];
        p.out.status[b] = HS_OK;
    }
}

__global__ void philox_kernel(unsigned long long seed, unsigned long long offset, const int* b, const int* node,
                              const int* stream_id, int count, float* out) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = philox_uniform(seed, offset, b[i], node[i], stream_id[i]);
}

hs_status hs_launch_philox(uint64_t seed, uint64_t offset, const int32_t* b, const int32_t* node,
                           const int32_t* stream_id, int32_t count, float* out, cudaStream_t stream) {
    philox_kernel<<<(count + 255) / 256, 256, 0, stream>>>(seed, offset, b, node, stream_id, count, out);
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

hs_status hs_launch_accept(hs_ctx* ctx, const hs_tree_batch* tree, const hs_pruned_tree* pruned,
                           const void* target_logits, int32_t target_layout, const void* draft_logits,
                           hs_dtype dtype, int64_t row_stride, int32_t vocab, const int32_t* mode,
                           const float* temperature, uint64_t seed, uint64_t offset, const float* uniforms,
                           const hs_accept_out* out, cudaStream_t stream) {
    AcceptParams p;
    const int ve = hs_vec_elems(dtype);
    p.target = target_logits;
    p.draft = draft_logits ? draft_logits : target_logits;   // only read by sampling sequences
    p.row_stride = row_stride;
    p.vocab = vocab;
    p.nvec = (vocab + ve - 1) / ve;
    p.chunks = hs_row_chunks(vocab, dtype);
    if (p.chunks > 32) return HS_ERR_SHAPE;
    p.chunk_vecs = (p.nvec + p.chunks - 1) / p.chunks;
    p.is_bf16 = dtype == HS_BF16;
    p.have_draft = draft_logits != nullptr;
    p.batch = tree->batch;
    p.n_nodes_total = tree->n_nodes_total;
    p.target_layout = target_layout;
    p.node_off = tree->node_off;
    p.token = tree->token;
    p.pr = *pruned;
    p.mode = mode;
    p.temperature = temperature;
    p.seed = seed;
    p.offset = offset;
    p.uniforms = uniforms;
    p.out = *out;
    int rows = tree->n_nodes_total;                // upper bound of kept nodes
    if (out->max_kept_rows > 0 && out->max_kept_rows < rows) rows = out->max_kept_rows;
    size_t o = 0;
    p.ro.tgt_arg = (int*)(ctx->scratch + o); o += hs_align_up((size_t)rows * sizeof(int), 256);
    p.ro.tgt_ms = (float2*)(ctx->scratch + o); o += hs_align_up((size_t)rows * sizeof(float2), 256);
    p.ro.drf_ms = (float2*)(ctx->scratch + o); o += hs_align_up((size_t)rows * sizeof(float2), 256);
    p.partials = (uint4*)(ctx->scratch + o);
    p.part_rows = rows;
    // (chunk kernel: a partial per chunk of a row; streaming kernel: two per share, one share per SM)
    o += max((size_t)2 * rows * p.chunks, (size_t)2 * ctx->sm_count) * sizeof(uint4);
    if (o > ctx->scratch_bytes) return HS_ERR_WORKSPACE;
    p.row_cnt = ctx->counters + HS_CNT_ACC_ROW;
    p.seq_cnt = ctx->counters + HS_CNT_ACC_SEQ;
    p.err = ctx->counters + HS_CNT_ERROR;
    p.staged = 0;
    p.clustered = 0;
    // without draft logits every sequence must be greedy: no draft rows to scan and no sampling walk
    cudaError_t e;
    const bool streamed = ctx->row_pass == HS_ROW_PASS_STREAM ||
                          (ctx->row_pass == HS_ROW_PASS_AUTO && (size_t)rows * p.nvec * 16 >= AS_MIN_BYTES);
    if (streamed) {
        // enough rows to be bound by memory traffic: one persistent CTA per SM streams them
        if (!ctx->rows_ready) {
            if (cudaFuncSetAttribute(accept_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AS_SMEM_BYTES) != cudaSuccess ||
                cudaFuncSetAttribute(accept_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AS_SMEM_BYTES) != cudaSuccess)
                return HS_ERR_CUDA;
            ctx->rows_ready = true;
        }
        e = dtype == HS_BF16
            ? hs_launch(accept_stream_kernel<true>, dim3(ctx->sm_count), dim3(AS_THREADS), AS_SMEM_BYTES, stream, ctx->pdl, dim3(1, 1, 1), p)
            : hs_launch(accept_stream_kernel<false>, dim3(ctx->sm_count), dim3(AS_THREADS), AS_SMEM_BYTES, stream, ctx->pdl, dim3(1, 1, 1), p);
    } else {
        // up to eight chunks per row (the portable cluster size): the CTAs of a row are one cluster, and the row is
        // merged in the shared memory of its first CTA instead of through partials and a counter in global memory
        // - while the whole grid is resident at once (four CTAs per SM): with more CTAs the clusters wait for eight free
        // slots in one GPC and the pass gets slower than with independent CTAs
        p.clustered = p.chunks > 1 && p.chunks <= 8 &&
                      (size_t)p.chunks * rows * (p.have_draft ? 2 : 1) * 2 <= (size_t)7 * ctx->sm_count;
        dim3 grid(p.chunks, rows, p.have_draft ? 2 : 1), cl(p.clustered ? p.chunks : 1, 1, 1);
        e = dtype == HS_BF16
            ? hs_launch(accept_rows_kernel<true>, grid, dim3(HS_ROW_THREADS), 0, stream, ctx->pdl, cl, p)
            : hs_launch(accept_rows_kernel<false>, grid, dim3(HS_ROW_THREADS), 0, stream, ctx->pdl, cl, p);
    }
    if (e != cudaSuccess) return HS_ERR_CUDA;
    if (!p.have_draft) return HS_OK;
    // the cluster shape of the walk is fixed at compile time (__cluster_dims__); its two row slices in shared memory
    const size_t esz = dtype == HS_BF16 ? 2 : 4;
    const size_t walk_smem = 2 * (size_t)((p.nvec + WALK_CLUSTER - 1) / WALK_CLUSTER) * 16;
    p.staged = ((uintptr_t)p.target % 16 == 0) && ((uintptr_t)p.draft % 16 == 0) && ((size_t)row_stride * esz % 16 == 0) &&
               walk_smem <= 160 * 1024;
    if (!ctx->walk_ready) {                  // per device (= per context): more than 48 KiB of shared memory, 16-CTA clusters
        if (cudaFuncSetAttribute(accept_walk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(accept_walk_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
            return HS_ERR_CUDA;
        ctx->walk_ready = true;
    }
    e = hs_launch(accept_walk_kernel, dim3(p.batch * WALK_CLUSTER), dim3(WALK_THREADS), p.staged ? walk_smem : 0, stream,
                  ctx->pdl, dim3(1, 1, 1), p);
    return e == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
