// Tree stage of one sequence by one CTA of HS_MAX_NODES (128) threads, one thread per node: path confidence
// ln V_i (Sec. 2.2), cumulative meta-path Top-K entropy Phi (Eq. 1), the operational path P* (Sec. 4.1).
// Shared by the kernel that follows the entropy pass and by the kernel that goes on to prune the tree.
#pragma once

#include <math_constants.h>

#include "hs_common.cuh"
#include "hs_layout.h"
#include "hs_ptx.cuh"

struct TreeStageSmem {
    float logc[HS_MAX_NODES], I[HS_MAX_NODES], phi[HS_MAX_NODES];
    int par[HS_MAX_NODES];
    unsigned long long best[4];
    int maxd[4];
    float phi_star;
};

struct TreeStageResult {   // of the calling thread's node (thread t = node t)
    int n;                 // nodes of the sequence
    bool bad;              // the sequence was flagged (empty, too large or malformed); its outputs are written
    int par, dep;
    float S;               // ln V of the node
};

// P needs: logits, row_stride, vocab, is_bf16, node_off, parent, token, out (hs_quant_out), d_base, phi_mode,
// pstar_mode, entropy_mode, prefetch.  Calls griddepcontrol.wait once (the row statistics come from the launch ahead;
// with `prefetch` the tree and the token logits, inputs of the call, are fetched before that wait).
template <class P>
__device__ __forceinline__ TreeStageResult tree_stage_cta(const P& p, int b, TreeStageSmem& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    TreeStageResult r;
    if (!p.prefetch) pdl_wait();
    const int base = p.node_off[b];
    const int n = p.node_off[b + 1] - base;
    r.n = n;
    int bad = (n > HS_MAX_NODES || n <= 0);
    int par = -1, tok = 0;
    if (!bad && tid < n) {
        par = p.parent[base + tid];
        tok = p.token[base + tid];
        if (tid == 0) bad = (par != -1);
        else bad = (par < 0 || par >= tid || tok < 0 || tok >= p.vocab);
    }
    float lv = 0.f;
    if (!bad && tid < n && tid > 0) {
        const size_t off = (size_t)(base + par) * p.row_stride + tok;
        lv = p.is_bf16 ? __bfloat162float(((const __nv_bfloat16*)p.logits)[off]) : ((const float*)p.logits)[off];
    }
    if (p.prefetch) pdl_wait();
    bad = __syncthreads_or(bad);
    r.bad = bad != 0;
    r.par = par; r.dep = 0; r.S = 0.f;
    if (bad) {
        for (int i = tid; i < n; i += blockDim.x) {
            p.out.logc[base + i] = 0.f; p.out.score[base + i] = 0.f; p.out.phi[base + i] = 0.f;
            p.out.depth[base + i] = 0;
        }
        if (tid == 0) { p.out.status[b] = HS_ERR_BAD_TREE; p.out.pstar_node[b] = 0; p.out.phi_star[b] = 0.f; }
        return r;
    }
    if (tid < n) {
        sm.logc[tid] = tid > 0 ? lv - p.out.row_lse[base + par] : 0.f;
        sm.I[tid] = p.entropy_mode == 0 ? p.out.i_topk[base + tid] : p.out.i_trunc[base + tid];
        sm.par[tid] = par;
    }
    __syncthreads();
    float S = 0.f, Phi = 0.f;
    int dep = 0;
    if (tid < n) {
        int a = tid;
        while (a > 0) {
            const int pa = sm.par[a];
            S += sm.logc[a];
            Phi += sm.I[pa];
            a = pa;
            ++dep;
        }
        if (p.phi_mode == 1) Phi += sm.I[tid];
        sm.phi[tid] = Phi;
        p.out.logc[base + tid] = sm.logc[tid];
        p.out.score[base + tid] = S;
        p.out.phi[base + tid] = Phi;
        p.out.depth[base + tid] = dep;
    }
    r.dep = dep; r.S = S;
    // deepest level, then P* among the nodes of depth min(d_base, deepest)
    int md = dep;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) md = max(md, __shfl_xor_sync(HS_FULL_MASK, md, o));
    if (lane == 0) sm.maxd[warp] = md;
    __syncthreads();
    md = max(max(sm.maxd[0], sm.maxd[1]), max(sm.maxd[2], sm.maxd[3]));
    const int t_eval = min(p.d_base, md);
    unsigned long long key = 0ull;
    if (tid < n && dep == t_eval) key = make_key(p.pstar_mode == 0 ? sm.logc[tid] : S, tid);
    key = warp_max_u64(key);
    if (lane == 0) sm.best[warp] = key;
    __syncthreads();
    if (tid == 0) {
        unsigned long long best = sm.best[0];
        for (int w = 1; w < 4; ++w) best = sm.best[w] > best ? sm.best[w] : best;
        const int node = key_index(best);
        sm.phi_star = sm.phi[node];
        p.out.pstar_node[b] = node;
        p.out.phi_star[b] = sm.phi[node];
        p.out.status[b] = HS_OK;
    }
    return r;
}
