"""One verification step on the GPU: uploads a synthetic batch and chains the four C-ABI calls.

Only plumbing lives here (device buffers, the order of the calls); every step of the path runs
inside the CUDA library.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as hb


def _bf16(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def _logits(x: np.ndarray, device) -> torch.Tensor:
    return _bf16(x, device) if x.dtype == np.uint16 else torch.from_numpy(np.ascontiguousarray(x)).to(device)


@dataclass
class DeviceBatch:
    """A batch as the input generators emit it, resident on the device.  Rows of the logits and of
    q / k_tree / v_tree are indexed by drafted node id (HS_ROWS_ORIGINAL)."""
    tree: hb.TreeBatch
    draft: Optional[torch.Tensor]
    target: Optional[torch.Tensor]
    q: Optional[torch.Tensor]
    k_tree: Optional[torch.Tensor]
    v_tree: Optional[torch.Tensor]
    k_cache: Optional[torch.Tensor]
    v_cache: Optional[torch.Tensor]
    kv_off: torch.Tensor
    mode: torch.Tensor
    temperature: torch.Tensor
    seed: int
    offset: int
    max_nodes: int
    max_kv_len: int
    any_sampling: bool = True

    def nbytes(self) -> int:
        ts = [self.tree.node_off, self.tree.parent, self.tree.token, self.draft, self.target, self.q, self.k_tree,
              self.v_tree, self.k_cache, self.v_cache, self.kv_off, self.mode, self.temperature]
        return sum(t.numel() * t.element_size() for t in ts if t is not None)


def upload(batch: dict, device="cuda:0") -> DeviceBatch:
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
    node_off = np.asarray(batch["node_off"])
    kv_off = np.asarray(batch["kv_off"])
    tree = hb.TreeBatch(i32(node_off), i32(batch["parent"]), i32(batch["token"]), len(node_off) - 1, int(node_off[-1]))
    get = lambda k, f: f(batch[k], device) if k in batch else None
    return DeviceBatch(tree, get("draft", _logits), get("target", _logits), get("q", _bf16), get("k_tree", _bf16),
                       get("v_tree", _bf16), get("k_cache", _bf16), get("v_cache", _bf16), i32(kv_off),
                       i32(batch["mode"]),
                       torch.from_numpy(np.asarray(batch["temperature"], dtype=np.float32)).to(device),
                       int(batch["philox_seed"]), int(batch["philox_offset"]),
                       int(np.diff(node_off).max()), int(np.diff(kv_off).max()),
                       bool(np.any(np.asarray(batch["mode"]) == hb.HS_ACCEPT_REJECTION)))


class VerifyStep:
    """Pre-allocated outputs + the four calls in the order of the decode loop."""

    def __init__(self, ctx: hb.Context, db: DeviceBatch, policy: dict, path_cap: int = 32):
        dev = db.tree.parent.device
        self.ctx, self.policy = ctx, policy
        n, b = db.tree.n_nodes_total, db.tree.batch
        self.quant = hb.QuantOut(n, b, policy["top_k"], dev)
        self.pruned = hb.PrunedTree(n, b, dev)
        self.accept = hb.AcceptOut(b, path_cap, dev)
        self.attn_out = torch.zeros_like(db.q) if db.q is not None else None
        self.attn_lse = (torch.zeros(db.q.shape[0], db.q.shape[1], dtype=torch.float32, device=dev)
                         if db.q is not None else None)

    def quantify(self, db: DeviceBatch):
        return hb.hs_entropy_quantify(self.ctx, db.tree, db.draft, self.policy, out=self.quant)

    def prune(self, db: DeviceBatch):
        return hb.hs_stratify_prune(self.ctx, db.tree, self.quant, self.policy, out=self.pruned)

    def attention(self, db: DeviceBatch, max_nodes: Optional[int] = None):
        # The launch is sized by an upper bound of the kept nodes per sequence: what the policy keeps at most of one
        # tree (hs_stratify_prune; a budgeted pruning may keep more: pass the drafted tree size then).
        if max_nodes is None:
            max_nodes = keep_bound(self.policy, db.max_nodes)
        return hb.hs_tree_verify_attention(self.ctx, self.pruned, db.q, db.k_tree, db.v_tree, db.k_cache, db.v_cache,
                                           db.kv_off, batch=db.tree.batch, max_nodes=max_nodes,
                                           max_kv_len=db.max_kv_len, layout=hb.HS_ROWS_ORIGINAL,
                                           node_off=db.tree.node_off, out=self.attn_out, lse_out=self.attn_lse)

    def accept_path(self, db: DeviceBatch):
        draft = db.draft if db.any_sampling else None        # only rejection-sampling sequences read draft rows
        return hb.hs_accept_path(self.ctx, db.tree, self.pruned, db.target, draft, db.mode, db.temperature,
                                 target_layout=hb.HS_ROWS_ORIGINAL, seed=db.seed, offset=db.offset,
                                 path_cap=self.accept.path_cap, out=self.accept)

    def quantify_prune(self, db: DeviceBatch):
        return hb.hs_entropy_quantify_prune(self.ctx, db.tree, db.draft, self.policy, out=self.quant,
                                            pruned_out=self.pruned)

    def run(self, db: DeviceBatch, fused: bool = True):
        """One verification step.  `fused`: entropy pass, tree scores and pruning as one call of two launches
        (hs_entropy_quantify_prune) instead of two calls of three."""
        if fused:
            self.quantify_prune(db)
        else:
            self.quantify(db)
            self.prune(db)
        if db.q is not None:
            self.attention(db)
        self.accept_path(db)
        return self


def refill(db: DeviceBatch, batch: dict) -> None:
    """Copies another batch of the same shapes (nodes, KV lengths, dtypes) into the device buffers of `db`."""
    src = upload(batch, db.tree.parent.device)
    if (src.tree.n_nodes_total, src.tree.batch, src.seed, src.offset) != \
            (db.tree.n_nodes_total, db.tree.batch, db.seed, db.offset):
        raise ValueError("refill needs a batch of the same shape and Philox seed / offset")
    for a, b in ((db.tree.node_off, src.tree.node_off), (db.tree.parent, src.tree.parent), (db.tree.token, src.tree.token),
                 (db.draft, src.draft), (db.target, src.target), (db.q, src.q), (db.k_tree, src.k_tree),
                 (db.v_tree, src.v_tree), (db.k_cache, src.k_cache), (db.v_cache, src.v_cache), (db.kv_off, src.kv_off),
                 (db.mode, src.mode), (db.temperature, src.temperature)):
        if a is not None:
            if a.shape != b.shape:
                raise ValueError("refill needs a batch of the same shape")
            a.copy_(b)


class GraphedStep:
    """The four calls over fixed input buffers, captured once into a CUDA graph and replayed (Sec. 4.3, the
    computation graph kept ready per regime).  One graph serves every entropy bin: the kernels read d', N' and the
    kept nodes from device memory, so nothing in the launch shapes depends on the regime.  Scalars of the calls
    (Philox seed and offset, strides) are part of the graph; the inputs are refreshed in place (`refill`)."""

    def __init__(self, step: VerifyStep, db: DeviceBatch, warmup: int = 2):
        self.step, self.db = step, db
        for _ in range(warmup):                       # first calls resolve attributes and tensor maps outside the capture
            step.run(db)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            step.run(db)

    def replay(self) -> VerifyStep:
        self.graph.replay()
        return self.step


def keep_bound(policy: dict, max_nodes: int) -> int:
    """Most nodes hs_stratify_prune keeps of one tree: the largest N' of the policy's regimes (Sec. 4.3), capped by
    the drafted tree size."""
    n = policy["n_default"]
    for i in range(3):
        n = max(n, (policy["gamma_pct"][i] * policy["n_default"] + 50) // 100 + policy["alpha"] - i)
    return max(1, min(max_nodes, n))


def regime_bounds(policy: dict, max_nodes: int):
    """The kept-node bounds of the regimes of Sec. 4.3: N' of the three low-entropy bins and of the others, ascending,
    capped by the drafted tree size."""
    b = set()
    for i in range(3):
        delta = policy["alpha"] - i
        b.add(min(max_nodes, (policy["gamma_pct"][i] * policy["n_default"] + 50) // 100 + delta))
    b.add(min(max_nodes, policy["n_default"]))
    b.add(max_nodes)
    return sorted(b)


class RegimeStep:
    """Sec. 4.3, Dynamic Computational Adaptation: a computation graph kept ready per regime.  The step runs in two
    phases: graph 1 = quantify + stratify/prune, after which the host reads the largest kept-node count of the
    batch (four bytes: the host has to know it anyway, it is the token count of the target model's forward pass);
    graph 2 = tree attention + acceptance, one graph per regime, captured with grids sized to that regime's N'
    instead of the drafted tree.  A regime is keyed by its bound on the kept nodes per sequence."""

    def __init__(self, step: VerifyStep, db: DeviceBatch, warmup: int = 2):
        self.step, self.db = step, db
        self.n_keep_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        self.n_keep_max = torch.zeros(1, dtype=torch.int32, device=db.tree.parent.device)
        for _ in range(warmup):
            step.run(db)
        torch.cuda.synchronize()
        self.phase1 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.phase1):
            step.quantify(db)
            step.prune(db)
            torch.amax(step.pruned.n_keep, dim=0, keepdim=True, out=self.n_keep_max)
            self.n_keep_host.copy_(self.n_keep_max, non_blocking=True)
        self.bounds = regime_bounds(step.policy, db.max_nodes)
        self.phase2 = {}
        for bound in self.bounds:
            step.accept.max_kept_rows = min(db.tree.n_nodes_total, bound * db.tree.batch)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                if db.q is not None:
                    step.attention(db, max_nodes=bound)
                step.accept_path(db)
            self.phase2[bound] = g
        step.accept.max_kept_rows = 0
        self.last_bound = None
        self.replay()                                        # (sets last_bound; results of the warm-up batch)

    def replay(self) -> VerifyStep:
        self.phase1.replay()
        torch.cuda.current_stream().synchronize()            # the host learns the regime
        n = int(self.n_keep_host[0])
        self.last_bound = next(b for b in self.bounds if b >= n)
        self.phase2[self.last_bound].replay()
        return self.step
