/*
 * heterospec.h - C ABI of the B200 (sm_100a) draft-tree verification library.
 *
 * One verification step of HeteroSpec (arXiv 2505.13254) is four calls, in this order:
 *
 *   hs_entropy_quantify       Sec. 4.1, Eq. 1: Top-K entropy of every draft distribution, the
 *                             cumulative meta-path entropy Phi of every tree path, the path
 *                             confidence V_i of Sec. 2.2 (in log form) and Phi(P*).
 *   hs_stratify_prune         Sec. 4.2-4.3: entropy bin -> speculative depth d' and Top-N';
 *                             Top-N' reranking of the tree (Sec. 2.2), compaction, tree mask.
 *   hs_tree_verify_attention  Sec. 2.2: tree-mask attention of the kept tokens over the accepted
 *                             prefix (KV cache) and their own ancestors.
 *   hs_accept_path            Sec. 2.1 / Sec. 5: greedy (temperature 0) or rejection-sampling
 *                             acceptance of the longest path, plus the bonus token.
 *
 * Conventions
 *   - A batch holds B independent sequences in CSR form.  Sequence b owns the tree nodes
 *     node_off[b] .. node_off[b+1]-1; inside a sequence nodes are numbered 0..n-1 in topological
 *     order (parent index < own index); node 0 is the root = the last accepted token (depth 0).
 *     A sequence has at most HS_MAX_NODES nodes.
 *   - Row r of a logits matrix is the next-token distribution AFTER node r.
 *   - Every data pointer is DEVICE memory owned by the caller unless a comment says "host".
 *     The small descriptor structs (hs_tree_batch, hs_policy, ...) are host structs read during
 *     the call.  The library owns only the workspace created by hs_create.
 *   - All four step calls enqueue work on the caller's stream and return without synchronising.
 *     `stream` is a cudaStream_t passed as void* (NULL = default stream).  A context serves one
 *     stream at a time (its workspace is shared by the calls); the device of the context must be
 *     the current device of the calling thread, otherwise the call returns HS_ERR_INVALID_ARG.
 *   - Kernels are launched with programmatic stream serialisation: their prologue may overlap the
 *     tail of the kernel ahead of them in the stream.  By default every read of caller memory comes
 *     after the dependency wait, so inputs written by the preceding kernel (the draft model's LM
 *     head, a cache append) are always complete.  hs_set_prefetch relaxes this per input class.
 *   - Errors: a bad argument or shape returns a non-zero hs_status and launches nothing.
 *     Data-dependent problems (malformed tree, token out of range) set status[b] != 0 on the
 *     device; later steps skip such a sequence (n_keep = 0, accept_len = 0).  Kernels never trap.
 *   - Results are deterministic: the same inputs give bit-identical outputs.
 */
#ifndef HETEROSPEC_H
#define HETEROSPEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HS_MAX_NODES 128 /* nodes per sequence (two 64-bit words of tree mask) */
#define HS_MAX_TOPK 16   /* K of the Top-K entropy */
#define HS_HEAD_DIM 128  /* the only supported attention head size */

typedef struct hs_ctx hs_ctx;
typedef void* hs_stream;

typedef enum {
    HS_OK = 0,
    HS_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum */
    HS_ERR_SHAPE = 2,       /* size outside the supported range */
    HS_ERR_UNSUPPORTED = 3,
    HS_ERR_WORKSPACE = 4,   /* workspace given to hs_create is too small for this call */
    HS_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed */
    HS_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (device status word) */
    HS_ERR_BAD_TREE = 7,    /* device status word: malformed tree or token out of range */
    HS_ERR_STATIC_LIMIT = 8 /* hs_entropy_quantify_static: batch larger than the built-in scratch array */
} hs_status;

typedef enum { HS_F32 = 0, HS_BF16 = 1 } hs_dtype;
/* GREEDY: Sec. 5 (temperature 0).  REJECTION: Sec. 2.1, candidates sampled from the draft distribution q.
 * DETERMINISTIC: Sec. 2.1 with a point-mass proposal per candidate (drafts that propose fixed tokens, e.g. their
 * top-k): candidate x is accepted with probability r(token of x), a rejection removes that token from r. */
typedef enum { HS_ACCEPT_GREEDY = 0, HS_ACCEPT_REJECTION = 1, HS_ACCEPT_DETERMINISTIC = 2 } hs_accept_mode;
/* Layout of per-kept-node rows (q, k_tree, v_tree, out, target logits):
 *   COMPACT  row keep_off[b] + i           belongs to kept node i of sequence b
 *   ORIGINAL row node_off[b] + keep_idx[.] belongs to it (rows indexed by drafted node id) */
typedef enum { HS_ROWS_COMPACT = 0, HS_ROWS_ORIGINAL = 1 } hs_row_layout;

const char* hs_status_string(hs_status s);

/* Bytes of workspace that cover every call on batches of at most `max_rows` tree nodes in total,
 * `max_batch` sequences, `hq` query heads and a vocabulary of `vocab`. */
size_t hs_workspace_bytes(int32_t max_batch, int32_t max_rows, int32_t vocab, int32_t hq, int32_t hkv);

/* Creates a context on `device` and allocates `workspace_bytes` of device memory (the only
 * allocation the library makes).  hs_destroy frees it. */
hs_status hs_create(hs_ctx** ctx, int32_t device, size_t workspace_bytes);
hs_status hs_destroy(hs_ctx* ctx);

/* Inputs a kernel may start to fetch BEFORE it waits for the kernel ahead of it in the stream (see
 * "Conventions").  Set a bit only if that input is complete before the call is enqueued, i.e. it is
 * not written by the immediately preceding kernel of the stream: typically true for the KV cache
 * prefix (appended a step earlier), true for logits only if something else separates producer and
 * call.  Default 0: nothing is read early. */
#define HS_PREFETCH_LOGITS 1   /* draft logits and tree arrays (parent, token, node_off) of hs_entropy_quantify */
#define HS_PREFETCH_KV 2       /* k_cache / v_cache of hs_tree_verify_attention */
hs_status hs_set_prefetch(hs_ctx* ctx, int32_t flags);

/* Which kernel hs_accept_path reads the vocabulary rows with (a tuning knob; the paper has no counterpart).  Both give
 * the same results.  HS_ROW_PASS_CHUNK: one small CTA per 32 KiB of a row, all loads in flight at once - shortest
 * latency when the rows of a step are few.  HS_ROW_PASS_STREAM: one persistent CTA per SM with a producer warp and
 * a ring of shared-memory slots - highest bandwidth when the rows of a step exceed what is in flight at once.
 * HS_ROW_PASS_AUTO (default): the stream from 48 MiB of rows (upper bound of kept rows x row bytes), else chunks. */
#define HS_ROW_PASS_AUTO 0
#define HS_ROW_PASS_CHUNK 1
#define HS_ROW_PASS_STREAM 2
hs_status hs_set_row_pass(hs_ctx* ctx, int32_t variant);

/* Reads and clears the context's sticky device error word into *host_out (host pointer): HS_OK, or
 * HS_ERR_TIMEOUT if a kernel gave up a bounded wait since the last call.  Synchronises the device. */
hs_status hs_device_error(hs_ctx* ctx, int32_t* host_out);

/* Self-test of the bounded device-side wait (no counterpart in the paper): one thread waits on a
 * barrier that nothing completes, gives up after `limit_ns` nanoseconds (clamped to 1 us .. 10 ms)
 * and records HS_ERR_TIMEOUT in the context's error word, which hs_device_error then returns.  The
 * kernel always terminates; the context stays usable. */
hs_status hs_selftest_wait_timeout(hs_ctx* ctx, uint64_t limit_ns, hs_stream stream);

/* ---- descriptors -------------------------------------------------------------------------- */

typedef struct {
    int32_t batch;           /* B >= 1 */
    int32_t n_nodes_total;   /* node_off[B] (host copy) */
    const int32_t* node_off; /* [B+1] */
    const int32_t* parent;   /* [n_nodes_total] parent inside the sequence, -1 for the root */
    const int32_t* token;    /* [n_nodes_total] token id of the node (root: ignored) */
} hs_tree_batch;

/* Policy of Sec. 4.2-4.3.  The paper trains the seven thresholds offline and does not print
 * them, so they are an input.  bin = number of thresholds <= Phi(P*).  Bins 0..2:
 * Delta = alpha - bin, d' = d_base + Delta, N' = round(gamma_pct[bin] * n_default / 100) + Delta;
 * bins 3..7: d' = d_base, N' = n_default. */
typedef struct {
    float thresholds[7]; /* ascending */
    int32_t d_base;
    int32_t alpha;        /* ceil(depth / 2) in the paper (Table 3) */
    int32_t n_default;
    int32_t top_k;        /* 1 .. HS_MAX_TOPK */
    int32_t gamma_pct[3]; /* 30, 60, 100 in the paper */
    int32_t phi_mode;     /* 0: Phi sums the rows the path's tokens were drawn from; 1: + own row */
    int32_t pstar_mode;   /* 0: P* by the final token's confidence; 1: by the path confidence */
    int32_t entropy_mode; /* 0: Top-K probabilities renormalised to 1; 1: vocabulary softmax */
} hs_policy;

/* Outputs of hs_entropy_quantify.  Per row r (= tree node): */
typedef struct {
    float* row_max;    /* [N] maximum logit */
    float* row_lse;    /* [N] log-sum-exp */
    float* h_full;     /* [N] Shannon entropy of softmax(row), nats */
    float* i_topk;     /* [N] entropy of the renormalised Top-K probabilities (Eq. 1 inner sum) */
    float* i_trunc;    /* [N] -sum over the Top-K of p ln p, p the vocabulary softmax */
    float* topk_val;   /* [N*K] the K largest logits, descending; ties: lowest index first */
    int32_t* topk_idx; /* [N*K] their token ids */
    float* logc;       /* [N] ln c_n: draft log-probability of the node's token (root 0) */
    float* score;      /* [N] S = sum of logc root..n = ln V_i (Sec. 2.2) */
    float* phi;        /* [N] cumulative Top-K entropy of the path root..n (Eq. 1) */
    int32_t* depth;    /* [N] */
    int32_t* pstar_node; /* [B] end node of P* (Sec. 4.1) */
    float* phi_star;   /* [B] Phi(P*) */
    int32_t* status;   /* [B] 0 or HS_ERR_BAD_TREE */
} hs_quant_out;

/* Outputs of hs_stratify_prune.  M = total kept nodes <= N. */
typedef struct {
    int32_t* bin;        /* [B] entropy bin 0..7 */
    int32_t* d_prime;    /* [B] */
    int32_t* n_prime;    /* [B] N' of the policy (before clamping to the eligible nodes) */
    int32_t* n_keep;     /* [B] kept nodes = min(N', nodes of depth <= d') */
    int32_t* keep_off;   /* [B+1] prefix sum of n_keep */
    int32_t* keep_idx;   /* [N] original node id of kept node, ascending per sequence */
    int32_t* new_parent; /* [N] parent among the kept nodes, -1 root */
    int32_t* new_depth;  /* [N] */
    int32_t* keep_rank;  /* [N] rank of the node by (S descending, index ascending) */
    uint64_t* anc_mask;  /* [N*2] bit j of (word j/64): kept node j is this node or an ancestor */
    int32_t* status;     /* [B] copied from the quantify status */
} hs_pruned_tree;

typedef struct {
    int32_t batch;
    int32_t max_rows;      /* upper bound of kept nodes in total (host): e.g. n_nodes_total */
    int32_t max_nodes;     /* upper bound of kept nodes per sequence (host), <= HS_MAX_NODES */
    int32_t kv_total;      /* tokens in the KV cache arrays = kv_off[B] (host copy) */
    int32_t max_kv_len;    /* longest prefix (host) */
    int32_t hq, hkv;       /* query heads, key/value heads; hq % hkv == 0, hq/hkv <= 16 */
    int32_t head_dim;      /* HS_HEAD_DIM */
    int32_t layout;        /* hs_row_layout of q, k_tree, v_tree, out, lse_out */
    const int32_t* node_off; /* [B+1] needed for HS_ROWS_ORIGINAL, else may be NULL */
    const int32_t* kv_off; /* [B+1] prefix of sequence b = cache tokens kv_off[b]..kv_off[b+1]-1 */
    int64_t kv_token_stride; /* elements between consecutive tokens of the cache, multiple of 8 */
    int64_t kv_head_stride;  /* elements between consecutive kv heads, multiple of 8 */
    float sm_scale;        /* 1/sqrt(head_dim) */
} hs_attn_desc;

typedef struct {
    int32_t* accept_len;   /* [B] number of accepted draft tokens */
    int32_t* path_nodes;   /* [B*path_cap] original node ids root..terminal, -1 padded */
    int32_t* path_compact; /* [B*path_cap] the same nodes as kept-node indices */
    int32_t* path_tokens;  /* [B*path_cap] tokens of the accepted nodes (slot 0 = first accepted) */
    int32_t* bonus_token;  /* [B] token emitted after the accepted path */
    int32_t* terminal_rank;/* [B] confidence rank of the terminal node (Terminal Confidence Rank) */
    int32_t* status;       /* [B] */
    int32_t path_cap;      /* slots per sequence, > deepest kept node */
    int32_t max_kept_rows; /* host: upper bound of the kept nodes of the whole batch, 0 = n_nodes_total; sizes the grid */
} hs_accept_out;

/* ---- the four steps ----------------------------------------------------------------------- */

/* Sec. 4.1, Eq. 1.  draft_logits: [n_nodes_total rows] of `vocab` values, row stride in elements
 * (multiple of 8 for bf16, 4 for f32; base 16-byte aligned).  Reads every row once. */
hs_status hs_entropy_quantify(hs_ctx* ctx, const hs_tree_batch* tree, const void* draft_logits,
                              hs_dtype dtype, int64_t row_stride, int32_t vocab,
                              const hs_policy* policy, const hs_quant_out* out, hs_stream stream);

/* No counterpart in the paper: hs_entropy_quantify for callers that must not allocate device memory
 * (a process whose memory is owned by one arena fixed at start-up, a component that is forbidden
 * cudaMalloc after initialisation).  It needs no hs_ctx and calls no cudaMalloc, cudaFree or other
 * allocating routine: its scratch (chunk partials and arrival counters) is one array built into the
 * library, about 580 KB that every GPU loading the library holds until the process exits.  Same
 * arguments, outputs and results as hs_entropy_quantify, on the CURRENT device.
 *   Limits: n_nodes_total <= HS_STATIC_MAX_ROWS, batch <= HS_STATIC_MAX_BATCH, vocab <= 262144 (bf16) or
 *   131072 (f32); anything larger returns HS_ERR_STATIC_LIMIT and launches nothing.
 *   The first call on a device looks up the array's device address (once per device, with that device
 *   current); make that first call outside any stream capture.
 *   All calls share the one array: it keeps the previous call's contents (the counters are cleared on the
 *   stream before each launch), and two calls whose kernels overlap on the GPU - different streams, or
 *   different threads - race on it.  Serialise them. */
#define HS_STATIC_MAX_ROWS 256
#define HS_STATIC_MAX_BATCH 64
hs_status hs_entropy_quantify_static(const hs_tree_batch* tree, const void* draft_logits, hs_dtype dtype,
                                     int64_t row_stride, int32_t vocab, const hs_policy* policy,
                                     const hs_quant_out* out, hs_stream stream);

/* hs_entropy_quantify and hs_stratify_prune (Sec. 4.1 - 4.3, reranking of Sec. 2.2) as one call of two launches
 * instead of three: the kernel that computes the tree scores of a sequence goes on to prune it, from shared memory
 * and registers.  Arguments, outputs (all of `quant` and all of `pruned` are written) and error behaviour are those
 * of the two calls made one after the other; the budgeted variant has no fused form.  Device pointers; enqueues on
 * `stream` and returns. */
hs_status hs_entropy_quantify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const void* draft_logits,
                                    hs_dtype dtype, int64_t row_stride, int32_t vocab, const hs_policy* policy,
                                    const hs_quant_out* quant, const hs_pruned_tree* pruned, hs_stream stream);

/* Sec. 4.2-4.3 and the reranking of Sec. 2.2.  Reads score, phi_star, depth, status of `quant`. */
hs_status hs_stratify_prune(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                            const hs_policy* policy, const hs_pruned_tree* out, hs_stream stream);

/* hs_stratify_prune under a token budget (App. A.8: "hardware budget", the tokens one forward pass of the target
 * model may process, shared by the batch).  The paper names the goal - Top-N pruning frees budget on low-entropy
 * requests, which is handed to requests with stricter service-level objectives - but no algorithm; this call
 * implements: every sequence first asks for min(N', nodes of depth <= d'); if the requests fit `budget`, the
 * tokens left over go to the sequences in order of slo_class[b] (device [B]; smaller = stricter = served first,
 * ties by sequence index), each up to its nodes of depth <= d'; otherwise the excess is taken back in the
 * opposite order, never below the root.  The reallocated counts replace N' in the Top-N reranking (n_keep
 * reports them, n_prime still the policy's N'); the sum of n_keep is at most max(budget, B). */
hs_status hs_stratify_prune_budget(hs_ctx* ctx, const hs_tree_batch* tree, const hs_quant_out* quant,
                                   const hs_policy* policy, const int32_t* slo_class, int32_t budget,
                                   const hs_pruned_tree* out, hs_stream stream);

/* Sec. 2.2 tree-mask attention.  q, out: [rows][hq][128] bf16; k_tree, v_tree: [rows][hkv][128]
 * bf16 (keys/values of the kept tree tokens, already position-encoded); k_cache, v_cache: bf16
 * with the strides of `desc`; lse_out (nullable): [rows][hq] float, natural-log normaliser.
 * Kept node i of a sequence sees the whole prefix and the tree tokens j with anc_mask bit j. */
hs_status hs_tree_verify_attention(hs_ctx* ctx, const hs_pruned_tree* pruned, const hs_attn_desc* desc,
                                   const void* q, const void* k_tree, const void* v_tree,
                                   const void* k_cache, const void* v_cache, void* out,
                                   float* lse_out, hs_stream stream);

/* Sec. 2.1 (sampling) and Sec. 5 (temperature 0).  target_logits rows follow `target_layout`;
 * draft_logits rows are always indexed by original node id (as given to hs_entropy_quantify) and
 * are read only by sequences in rejection mode; a caller without such sequences passes NULL (a
 * rejection-mode sequence then gets status HS_ERR_INVALID_ARG) and saves a launch.  mode[b]: hs_accept_mode;
 * temperature[b] > 0 for the two sampling modes, applied to both models.  Uniforms: Philox4x32-10 with key = seed, counter =
 * (low word of offset, b, original node id, stream + 2 * (high word of offset)) with stream 0 = accept test of
 * that node, 1 = final draw (node 0); offset < 2^63; u = (x0 >> 8) * 2^-24.
 * Sibling candidates that carry the same token: the first in index order is the candidate, a later one
 * is tested against the residual like any other (greedy: the lowest index is taken).
 * path_cap: slots per sequence in path_*; a path longer than path_cap - 1 tokens is still walked and
 * accept_len reports its true length, only the first path_cap entries are stored.
 * If `uniforms` is not NULL it overrides the generator:
 * uniforms[node_off[b] + node] for accept tests and uniforms[n_nodes_total + b] for the final draw. */
hs_status hs_accept_path(hs_ctx* ctx, const hs_tree_batch* tree, const hs_pruned_tree* pruned,
                         const void* target_logits, int32_t target_layout, const void* draft_logits,
                         hs_dtype dtype, int64_t row_stride, int32_t vocab, const int32_t* mode,
                         const float* temperature, uint64_t seed, uint64_t offset,
                         const float* uniforms, const hs_accept_out* out, hs_stream stream);

/* Philox4x32-10 uniforms exactly as hs_accept_path draws them, written to out[count] for
 * counters (offset, b[i], node[i], stream[i]) - for cross-checking the generator by value. */
hs_status hs_philox_uniforms(hs_ctx* ctx, uint64_t seed, uint64_t offset, const int32_t* b,
                             const int32_t* node, const int32_t* stream_id, int32_t count,
                             float* out, hs_stream stream);

/* ---- the step ahead of verification: growing and reranking the draft tree ------------------------ */

/* Candidate tree of Sec. 2.2 ("Expansion"), all arrays DEVICE memory owned by the caller.  Sequence b owns slots
 * b * cap .. b * cap + n_cand[b] - 1 in creation order (candidate 0 = the root, parents precede children).
 * cap >= 1 + top_k + (levels - 1) * top_k^2 holds a tree of that many levels. */
typedef struct {
    int32_t batch;
    int32_t cap;          /* slots per sequence; hs_rerank takes at most 2048 */
    int32_t top_k;        /* children per expanded node = width of the frontier, 1 .. HS_MAX_TOPK */
    int32_t* n_cand;      /* [B] candidates so far */
    int32_t* parent;      /* [B*cap] candidate id of the parent, -1 for the root */
    int32_t* token;       /* [B*cap] */
    int32_t* depth;       /* [B*cap] */
    float* logc;          /* [B*cap] ln c: log-confidence of the token under its parent's draft row */
    float* score;         /* [B*cap] ln V_i = sum of logc along the path */
    int32_t* frontier;    /* [B*top_k] candidates the draft model is run on next, best first */
    int32_t* n_frontier;  /* [B] */
    int32_t* status;      /* [B] 0, HS_ERR_SHAPE (cap exhausted) or HS_ERR_BAD_TREE (a row with fewer than top_k finite logits) */
} hs_expand_state;

/* Sec. 2.2: the tree holds the root only, the frontier is the root. */
hs_status hs_expand_init(hs_ctx* ctx, const hs_expand_state* st, hs_stream stream);

/* Sec. 2.2 "Expansion", one level (Sec. 4.3: called d' = d_base + Delta times): row b * top_k + j of the three
 * statistics arrays belongs to the draft row after frontier[b * top_k + j] - exactly what hs_entropy_quantify
 * writes to topk_val / topk_idx (row stride topk_stride >= top_k, best first) and row_lse for those rows.  Every
 * frontier node gets its top_k tokens as children (value = parent's + ln c); the top_k children with the
 * largest value, ties to the one created first, are the next frontier. */
hs_status hs_expand_level(hs_ctx* ctx, const hs_expand_state* st, const float* topk_val, const int32_t* topk_idx,
                          const float* row_lse, int32_t topk_stride, hs_stream stream);

/* Sec. 2.2 "Reranking" (Sec. 4.3: with N' in place of N): the n_top[b] (NULL: n_default) candidates with the
 * largest value, root included, as a tree in creation order: node_off[B+1], and per kept node its parent among
 * the kept nodes, token, candidate id and depth (arrays of at least sum of min(N, n_cand) entries).  The result is
 * an hs_tree_batch for the verification calls. */
hs_status hs_rerank(hs_ctx* ctx, const hs_expand_state* st, const int32_t* n_top, int32_t n_default,
                    int32_t* node_off, int32_t* parent, int32_t* token, int32_t* cand_id, int32_t* depth,
                    hs_stream stream);

/* ---- training of the stratifier ------------------------------------------------------------------- */

/* Sec. 4.2, Eq. 2: CART regression on one feature.  x[n] = Phi(P*) of n verified trees (phi_star of
 * hs_entropy_quantify), y[n] = their Terminal Confidence Rank (terminal_rank of hs_accept_path, as floats), both
 * DEVICE arrays.  Every layer splits every node at the threshold s that minimises
 *   L(s) = sum over {left, right} of |D_j| / |D| * sum over D_j of (y - mean_j)^2
 * over the midpoints between consecutive distinct feature values (ties: the smallest s).  thresholds (device,
 * 2^depth - 1 floats) receives the thresholds in ascending order: with depth = 3 they are hs_policy.thresholds.
 * status (device, one int): 0, or HS_ERR_SHAPE if some node held a single feature value (its threshold is NaN).
 * 1 <= depth <= 6, 2^depth <= n <= 2^26.  Needs hs_cart_workspace_bytes(n) of context workspace. */
size_t hs_cart_workspace_bytes(int32_t n);
hs_status hs_cart_fit(hs_ctx* ctx, const float* x, const float* y, int32_t n, int32_t depth, float* thresholds,
                      int32_t* status, hs_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* HETEROSPEC_H */
