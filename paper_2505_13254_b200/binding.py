"""ctypes binding of ``libheterospec.so``: argument marshalling only.

Every function has the name and the meaning of the C entry point in ``include/heterospec.h``;
torch tensors provide device memory and the current CUDA stream, nothing is computed here.
A missing library or a non-zero status raises: there is no fallback path.
"""

from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

HS_MAX_NODES = 128
HS_MAX_TOPK = 16
HS_F32, HS_BF16 = 0, 1
HS_ACCEPT_GREEDY, HS_ACCEPT_REJECTION, HS_ACCEPT_DETERMINISTIC = 0, 1, 2
HS_ROWS_COMPACT, HS_ROWS_ORIGINAL = 0, 1
HS_PREFETCH_LOGITS, HS_PREFETCH_KV = 1, 2
HS_ROW_PASS_AUTO, HS_ROW_PASS_CHUNK, HS_ROW_PASS_STREAM = 0, 1, 2
HS_ERR_INVALID_ARG, HS_ERR_SHAPE, HS_ERR_WORKSPACE, HS_ERR_TIMEOUT, HS_ERR_BAD_TREE = 1, 2, 4, 6, 7

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libheterospec.so")
_lib = None

i32p, f32p, u64p, vp = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p   # device pointers travel as integers


class _TreeBatch(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_nodes_total", C.c_int32), ("node_off", i32p), ("parent", i32p),
                ("token", i32p)]


class _Policy(C.Structure):
    _fields_ = [("thresholds", C.c_float * 7), ("d_base", C.c_int32), ("alpha", C.c_int32),
                ("n_default", C.c_int32), ("top_k", C.c_int32), ("gamma_pct", C.c_int32 * 3),
                ("phi_mode", C.c_int32), ("pstar_mode", C.c_int32), ("entropy_mode", C.c_int32)]


class _QuantOut(C.Structure):
    _fields_ = [(n, vp) for n in ("row_max", "row_lse", "h_full", "i_topk", "i_trunc", "topk_val", "topk_idx",
                                  "logc", "score", "phi", "depth", "pstar_node", "phi_star", "status")]


class _PrunedTree(C.Structure):
    _fields_ = [(n, vp) for n in ("bin", "d_prime", "n_prime", "n_keep", "keep_off", "keep_idx", "new_parent",
                                  "new_depth", "keep_rank", "anc_mask", "status")]


class _AttnDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("max_rows", C.c_int32), ("max_nodes", C.c_int32), ("kv_total", C.c_int32),
                ("max_kv_len", C.c_int32), ("hq", C.c_int32), ("hkv", C.c_int32), ("head_dim", C.c_int32),
                ("layout", C.c_int32), ("node_off", i32p), ("kv_off", i32p), ("kv_token_stride", C.c_int64),
                ("kv_head_stride", C.c_int64), ("sm_scale", C.c_float)]


class _ExpandState(C.Structure):
    _fields_ = [("batch", C.c_int32), ("cap", C.c_int32), ("top_k", C.c_int32)] + \
               [(n, vp) for n in ("n_cand", "parent", "token", "depth", "logc", "score", "frontier", "n_frontier", "status")]


class _AcceptOut(C.Structure):
    _fields_ = [(n, vp) for n in ("accept_len", "path_nodes", "path_compact", "path_tokens", "bonus_token",
                                  "terminal_rank", "status")] + [("path_cap", C.c_int32), ("max_kept_rows", C.c_int32)]


EXPORTS = ("hs_status_string", "hs_workspace_bytes", "hs_create", "hs_destroy", "hs_device_error", "hs_entropy_quantify",
           "hs_stratify_prune", "hs_tree_verify_attention", "hs_accept_path", "hs_philox_uniforms",
           "hs_entropy_quantify_static", "hs_set_prefetch", "hs_set_row_pass", "hs_entropy_quantify_prune", "hs_selftest_wait_timeout", "hs_expand_init",
           "hs_expand_level", "hs_rerank", "hs_cart_fit", "hs_cart_workspace_bytes", "hs_stratify_prune_budget")


def lib() -> C.CDLL:
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2505_13254_b200.build`")
        L = C.CDLL(_LIB_PATH)
        L.hs_status_string.restype = C.c_char_p
        L.hs_status_string.argtypes = [C.c_int]
        L.hs_workspace_bytes.restype = C.c_size_t
        L.hs_workspace_bytes.argtypes = [C.c_int32] * 5
        L.hs_create.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.c_size_t]
        L.hs_destroy.argtypes = [C.c_void_p]
        L.hs_device_error.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        L.hs_set_prefetch.argtypes = [C.c_void_p, C.c_int32]
        L.hs_set_row_pass.argtypes = [C.c_void_p, C.c_int32]
        L.hs_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_uint64, vp]
        L.hs_entropy_quantify.argtypes = [C.c_void_p, C.POINTER(_TreeBatch), vp, C.c_int, C.c_int64, C.c_int32,
                                          C.POINTER(_Policy), C.POINTER(_QuantOut), vp]
        L.hs_entropy_quantify_prune.argtypes = [C.c_void_p, C.POINTER(_TreeBatch), vp, C.c_int, C.c_int64, C.c_int32,
                                                C.POINTER(_Policy), C.POINTER(_QuantOut), C.POINTER(_PrunedTree), vp]
        L.hs_entropy_quantify_static.argtypes = [C.POINTER(_TreeBatch), vp, C.c_int, C.c_int64, C.c_int32,
                                                 C.POINTER(_Policy), C.POINTER(_QuantOut), vp]
        L.hs_stratify_prune.argtypes = [C.c_void_p, C.POINTER(_TreeBatch), C.POINTER(_QuantOut),
                                        C.POINTER(_Policy), C.POINTER(_PrunedTree), vp]
        L.hs_stratify_prune_budget.argtypes = [C.c_void_p, C.POINTER(_TreeBatch), C.POINTER(_QuantOut),
                                               C.POINTER(_Policy), vp, C.c_int32, C.POINTER(_PrunedTree), vp]
        L.hs_tree_verify_attention.argtypes = [C.c_void_p, C.POINTER(_PrunedTree), C.POINTER(_AttnDesc), vp, vp, vp,
                                               vp, vp, vp, vp, vp]
        L.hs_accept_path.argtypes = [C.c_void_p, C.POINTER(_TreeBatch), C.POINTER(_PrunedTree), vp, C.c_int32, vp,
                                     C.c_int, C.c_int64, C.c_int32, vp, vp, C.c_uint64, C.c_uint64, vp,
                                     C.POINTER(_AcceptOut), vp]
        L.hs_expand_init.argtypes = [C.c_void_p, C.POINTER(_ExpandState), vp]
        L.hs_expand_level.argtypes = [C.c_void_p, C.POINTER(_ExpandState), vp, vp, vp, C.c_int32, vp]
        L.hs_rerank.argtypes = [C.c_void_p, C.POINTER(_ExpandState), vp, C.c_int32, vp, vp, vp, vp, vp, vp]
        L.hs_cart_workspace_bytes.restype = C.c_size_t
        L.hs_cart_workspace_bytes.argtypes = [C.c_int32]
        L.hs_cart_fit.argtypes = [C.c_void_p, vp, vp, C.c_int32, C.c_int32, vp, vp, vp]
        L.hs_philox_uniforms.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, vp, vp, vp, C.c_int32, vp, vp]
        for name in EXPORTS:
            if name not in ("hs_status_string", "hs_workspace_bytes", "hs_cart_workspace_bytes"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class HsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().hs_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != 0:
        raise HsError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def hs_device_error(ctx: "Context") -> int:
    v = C.c_int32(0)
    _check(lib().hs_device_error(ctx.handle, C.byref(v)), "hs_device_error")
    return int(v.value)


def hs_set_prefetch(ctx: "Context", flags: int) -> None:
    _check(lib().hs_set_prefetch(ctx.handle, flags), "hs_set_prefetch")


def hs_set_row_pass(ctx: "Context", variant: int) -> None:
    _check(lib().hs_set_row_pass(ctx.handle, variant), "hs_set_row_pass")


def hs_selftest_wait_timeout(ctx: "Context", limit_ns: int) -> None:
    _check(lib().hs_selftest_wait_timeout(ctx.handle, limit_ns, _stream()), "hs_selftest_wait_timeout")


def hs_workspace_bytes(max_batch: int, max_rows: int, vocab: int, hq: int, hkv: int) -> int:
    return int(lib().hs_workspace_bytes(max_batch, max_rows, vocab, hq, hkv))


class Context:
    """hs_create / hs_destroy."""

    def __init__(self, device: int = 0, workspace_bytes: int = 256 << 20):
        self.handle = C.c_void_p()
        self.device = device
        _check(lib().hs_create(C.byref(self.handle), device, workspace_bytes), "hs_create")

    def close(self):
        if self.handle:
            lib().hs_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- tensor bundles mirroring the C structs --------------------------------------------------------


@dataclass
class TreeBatch:
    node_off: torch.Tensor   # int32 [B+1]
    parent: torch.Tensor     # int32 [N]
    token: torch.Tensor      # int32 [N]
    batch: int
    n_nodes_total: int

    def c(self) -> _TreeBatch:
        return _TreeBatch(self.batch, self.n_nodes_total, _ptr(self.node_off), _ptr(self.parent), _ptr(self.token))


def make_policy(policy: dict) -> _Policy:
    p = _Policy()
    for i, t in enumerate(policy["thresholds"]):
        p.thresholds[i] = t
    p.d_base, p.alpha, p.n_default, p.top_k = policy["d_base"], policy["alpha"], policy["n_default"], policy["top_k"]
    for i, g in enumerate(policy["gamma_pct"]):
        p.gamma_pct[i] = g
    p.phi_mode, p.pstar_mode, p.entropy_mode = policy["phi_mode"], policy["pstar_mode"], policy["entropy_mode"]
    return p


class _Bundle:
    _i32: tuple = ()
    _f32: tuple = ()
    _cstruct = None

    def c(self):
        s = self._cstruct()
        for name, _ in self._cstruct._fields_:
            v = getattr(self, name)
            setattr(s, name, v if isinstance(v, int) else _ptr(v).value)
        return s


class QuantOut(_Bundle):
    _cstruct = _QuantOut

    def __init__(self, n: int, batch: int, k: int, device):
        f = lambda *s: torch.empty(*s, dtype=torch.float32, device=device)
        i = lambda *s: torch.empty(*s, dtype=torch.int32, device=device)
        self.row_max, self.row_lse, self.h_full, self.i_topk, self.i_trunc = f(n), f(n), f(n), f(n), f(n)
        self.topk_val, self.topk_idx = f(n, k), i(n, k)
        self.logc, self.score, self.phi, self.depth = f(n), f(n), f(n), i(n)
        self.pstar_node, self.phi_star, self.status = i(batch), f(batch), i(batch)


class PrunedTree(_Bundle):
    _cstruct = _PrunedTree

    def __init__(self, n: int, batch: int, device):
        i = lambda *s: torch.zeros(*s, dtype=torch.int32, device=device)
        self.bin, self.d_prime, self.n_prime, self.n_keep = i(batch), i(batch), i(batch), i(batch)
        self.keep_off = i(batch + 1)
        self.keep_idx, self.new_parent, self.new_depth, self.keep_rank = i(n), i(n), i(n), i(n)
        self.anc_mask = torch.zeros(n, 2, dtype=torch.int64, device=device)
        self.status = i(batch)


class AcceptOut(_Bundle):
    _cstruct = _AcceptOut

    def __init__(self, batch: int, path_cap: int, device):
        i = lambda *s: torch.empty(*s, dtype=torch.int32, device=device)
        self.accept_len, self.bonus_token, self.terminal_rank, self.status = i(batch), i(batch), i(batch), i(batch)
        self.path_nodes, self.path_compact, self.path_tokens = i(batch, path_cap), i(batch, path_cap), i(batch, path_cap)
        self.path_cap = path_cap
        self.max_kept_rows = 0


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return HS_BF16
    if t.dtype == torch.float32:
        return HS_F32
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


# ---- the entry points --------------------------------------------------------------------------------


def hs_entropy_quantify(ctx: Context, tree: TreeBatch, draft_logits: torch.Tensor, policy: dict,
                        out: Optional[QuantOut] = None) -> QuantOut:
    if out is None:
        out = QuantOut(tree.n_nodes_total, tree.batch, policy["top_k"], draft_logits.device)
    t, p, o = tree.c(), make_policy(policy), out.c()
    _check(lib().hs_entropy_quantify(ctx.handle, C.byref(t), _ptr(draft_logits), _dtype_code(draft_logits),
                                     draft_logits.stride(0), draft_logits.shape[1], C.byref(p), C.byref(o), _stream()),
           "hs_entropy_quantify")
    return out


HS_STATIC_MAX_ROWS, HS_STATIC_MAX_BATCH, HS_ERR_STATIC_LIMIT = 256, 64, 8


def hs_entropy_quantify_static(tree: TreeBatch, draft_logits: torch.Tensor, policy: dict,
                               out: Optional[QuantOut] = None) -> QuantOut:
    """hs_entropy_quantify without a context: for callers that may not allocate device memory.  The scratch
    is an array built into the library (limits HS_STATIC_MAX_ROWS / HS_STATIC_MAX_BATCH); the outputs are
    still the caller's.  Runs on the current device; calls must not overlap on the GPU."""
    if out is None:
        out = QuantOut(tree.n_nodes_total, tree.batch, policy["top_k"], draft_logits.device)
    t, p, o = tree.c(), make_policy(policy), out.c()
    _check(lib().hs_entropy_quantify_static(C.byref(t), _ptr(draft_logits), _dtype_code(draft_logits),
                                            draft_logits.stride(0), draft_logits.shape[1], C.byref(p), C.byref(o),
                                            _stream()), "hs_entropy_quantify_static")
    return out


def hs_entropy_quantify_prune(ctx: Context, tree: TreeBatch, draft_logits: torch.Tensor, policy: dict,
                              out: Optional[QuantOut] = None, pruned_out: Optional["PrunedTree"] = None):
    """hs_entropy_quantify followed by hs_stratify_prune, as one call of two launches."""
    if out is None:
        out = QuantOut(tree.n_nodes_total, tree.batch, policy["top_k"], draft_logits.device)
    if pruned_out is None:
        pruned_out = PrunedTree(tree.n_nodes_total, tree.batch, tree.parent.device)
    t, p, o, q = tree.c(), make_policy(policy), out.c(), pruned_out.c()
    _check(lib().hs_entropy_quantify_prune(ctx.handle, C.byref(t), _ptr(draft_logits), _dtype_code(draft_logits),
                                           draft_logits.stride(0), draft_logits.shape[1], C.byref(p), C.byref(o),
                                           C.byref(q), _stream()), "hs_entropy_quantify_prune")
    return out, pruned_out


def hs_stratify_prune(ctx: Context, tree: TreeBatch, quant: QuantOut, policy: dict,
                      out: Optional[PrunedTree] = None) -> PrunedTree:
    if out is None:
        out = PrunedTree(tree.n_nodes_total, tree.batch, tree.parent.device)
    t, q, p, o = tree.c(), quant.c(), make_policy(policy), out.c()
    _check(lib().hs_stratify_prune(ctx.handle, C.byref(t), C.byref(q), C.byref(p), C.byref(o), _stream()),
           "hs_stratify_prune")
    return out


def hs_stratify_prune_budget(ctx: Context, tree: TreeBatch, quant: QuantOut, policy: dict, slo_class: torch.Tensor,
                             budget: int, out: Optional[PrunedTree] = None) -> PrunedTree:
    if out is None:
        out = PrunedTree(tree.n_nodes_total, tree.batch, tree.parent.device)
    t, q, p, o = tree.c(), quant.c(), make_policy(policy), out.c()
    _check(lib().hs_stratify_prune_budget(ctx.handle, C.byref(t), C.byref(q), C.byref(p), _ptr(slo_class), budget,
                                          C.byref(o), _stream()), "hs_stratify_prune_budget")
    return out


def hs_tree_verify_attention(ctx: Context, pruned: PrunedTree, q: torch.Tensor, k_tree: torch.Tensor,
                             v_tree: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                             kv_off: torch.Tensor, *, batch: int, max_nodes: int, max_kv_len: int,
                             layout: int = HS_ROWS_COMPACT, node_off: Optional[torch.Tensor] = None,
                             sm_scale: Optional[float] = None, out: Optional[torch.Tensor] = None,
                             lse_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q/out [rows, hq, 128] bf16; k_tree/v_tree [rows, hkv, 128]; k_cache/v_cache [tokens, hkv, 128] (any
    token/head strides that are multiples of 8 elements, innermost dimension contiguous)."""
    rows, hq, hd = q.shape
    hkv = k_tree.shape[1]
    if out is None:
        out = torch.empty_like(q)
    d = _AttnDesc(batch, rows, max_nodes, k_cache.shape[0], max_kv_len, hq, hkv, hd, layout, _ptr(node_off),
                  _ptr(kv_off), k_cache.stride(0) if k_cache.shape[0] else hkv * hd,
                  k_cache.stride(1) if k_cache.shape[0] else hd,
                  float(sm_scale if sm_scale is not None else hd ** -0.5))
    p = pruned.c()
    _check(lib().hs_tree_verify_attention(ctx.handle, C.byref(p), C.byref(d), _ptr(q), _ptr(k_tree), _ptr(v_tree),
                                          _ptr(k_cache), _ptr(v_cache), _ptr(out), _ptr(lse_out), _stream()),
           "hs_tree_verify_attention")
    return out


def hs_accept_path(ctx: Context, tree: TreeBatch, pruned: PrunedTree, target_logits: torch.Tensor,
                   draft_logits: Optional[torch.Tensor], mode: torch.Tensor, temperature: torch.Tensor, *,
                   target_layout: int = HS_ROWS_COMPACT, seed: int = 0, offset: int = 0,
                   uniforms: Optional[torch.Tensor] = None, path_cap: int = 32,
                   out: Optional[AcceptOut] = None) -> AcceptOut:
    if out is None:
        out = AcceptOut(tree.batch, path_cap, target_logits.device)
    t, p, o = tree.c(), pruned.c(), out.c()
    _check(lib().hs_accept_path(ctx.handle, C.byref(t), C.byref(p), _ptr(target_logits), target_layout,
                                _ptr(draft_logits), _dtype_code(target_logits), target_logits.stride(0),
                                target_logits.shape[1], _ptr(mode), _ptr(temperature), seed, offset, _ptr(uniforms),
                                C.byref(o), _stream()),
           "hs_accept_path")
    return out


def hs_philox_uniforms(ctx: Context, seed: int, offset: int, b: torch.Tensor, node: torch.Tensor,
                       stream_id: torch.Tensor) -> torch.Tensor:
    out = torch.empty(b.numel(), dtype=torch.float32, device=b.device)
    _check(lib().hs_philox_uniforms(ctx.handle, seed, offset, _ptr(b), _ptr(node), _ptr(stream_id), b.numel(),
                                    _ptr(out), _stream()), "hs_philox_uniforms")
    return out


class ExpandState(_Bundle):
    """Device arrays of the candidate tree (hs_expand_state)."""
    _cstruct = _ExpandState

    def __init__(self, batch: int, cap: int, top_k: int, device):
        i = lambda *s: torch.zeros(*s, dtype=torch.int32, device=device)
        f = lambda *s: torch.zeros(*s, dtype=torch.float32, device=device)
        self.batch, self.cap, self.top_k = batch, cap, top_k
        self.n_cand, self.n_frontier, self.status = i(batch), i(batch), i(batch)
        self.parent, self.token, self.depth = i(batch, cap), i(batch, cap), i(batch, cap)
        self.logc, self.score = f(batch, cap), f(batch, cap)
        self.frontier = i(batch, top_k)


def hs_expand_init(ctx: Context, st: ExpandState) -> None:
    c = st.c()
    _check(lib().hs_expand_init(ctx.handle, C.byref(c), _stream()), "hs_expand_init")


def hs_expand_level(ctx: Context, st: ExpandState, quant: QuantOut) -> None:
    """One expansion level from the row statistics of the frontier rows (row b * top_k + j = frontier j of b)."""
    c = st.c()
    _check(lib().hs_expand_level(ctx.handle, C.byref(c), _ptr(quant.topk_val), _ptr(quant.topk_idx),
                                 _ptr(quant.row_lse), quant.topk_val.shape[1], _stream()), "hs_expand_level")


def hs_rerank(ctx: Context, st: ExpandState, n_top: Optional[torch.Tensor], n_default: int):
    """Returns (node_off, parent, token, cand_id, depth): the reranked trees as one CSR batch."""
    dev = st.parent.device
    rows = st.batch * min(st.cap, max(n_default, int(n_top.max()) if n_top is not None else 0))
    i = lambda *s: torch.zeros(*s, dtype=torch.int32, device=dev)
    node_off, parent, token, cand_id, depth = i(st.batch + 1), i(rows), i(rows), i(rows), i(rows)
    c = st.c()
    _check(lib().hs_rerank(ctx.handle, C.byref(c), _ptr(n_top), n_default, _ptr(node_off), _ptr(parent), _ptr(token),
                           _ptr(cand_id), _ptr(depth), _stream()), "hs_rerank")
    return node_off, parent, token, cand_id, depth


def hs_cart_workspace_bytes(n: int) -> int:
    return int(lib().hs_cart_workspace_bytes(n))


def hs_cart_fit(ctx: Context, x: torch.Tensor, y: torch.Tensor, depth: int = 3):
    """Trains the stratifier on (Phi(P*), Terminal Confidence Rank) pairs.  Returns (thresholds [2^depth - 1], status [1])."""
    th = torch.empty((1 << depth) - 1, dtype=torch.float32, device=x.device)
    status = torch.zeros(1, dtype=torch.int32, device=x.device)
    _check(lib().hs_cart_fit(ctx.handle, _ptr(x), _ptr(y), x.numel(), depth, _ptr(th), _ptr(status), _stream()),
           "hs_cart_fit")
    return th, status
