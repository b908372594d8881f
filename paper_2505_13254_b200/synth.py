"""Seeded synthetic inputs for one draft-tree verification step.

These generators stand in for the draft model, the target model and the KV cache
of a speculative-decoding step: they produce a draft tree (parent pointers and
tokens), one row of draft logits and one row of target logits per tree node,
query/key/value vectors for the tree nodes and a key/value prefix.  Nothing of
the verification method itself (Top-K entropy, stratification, pruning,
attention, acceptance) lives here; the module is shared by the CPU oracle's
tests and by the CUDA path's tests and benchmark, and imports neither.

The draft tree follows the expansion/reranking recipe of Sec. 2.2 of the paper
(top-k children per expanded node, frontier and final node set chosen by the
cumulative log-confidence) because the verification path takes such a tree as
its input.  All randomness comes from counter-based Philox streams keyed by
``(seed, stream id)``, so any row can be regenerated independently.

bfloat16 data is carried as ``uint16`` bit patterns (numpy has no bf16 type).
"""

from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# dtype helpers
# ----------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, kind: int, b: int = 0, uid: int = 0) -> np.random.Generator:
    stream = (int(kind) << 56) | (int(b) << 36) | int(uid)
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), stream]))


_K_ROW, _K_TARGET, _K_TREE, _K_ATTN, _K_SEQ, _K_TEMP, _K_BOOST = range(1, 8)

# ----------------------------------------------------------------------------
# configurations (the five workloads of the verification benchmark)
# ----------------------------------------------------------------------------


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    batch: int
    vocab: int
    n_nodes: Tuple[int, int]          # inclusive range of drafted tree sizes (root included)
    draft_depth: int                  # depth the tree was drafted to
    d_base: int                       # base speculative depth of the policy
    top_k: int                        # expansion width = K of the Top-K entropy
    n_default: int                    # default Top-N of the reranking
    tree_kind: str                    # "random" | "eagle"
    logits_dtype: str                 # "f32" | "bf16"
    scale_kind: str                   # "uniform" (c1: s~U[0.2,4]) | "mix" (peaked/flat)
    hq: int
    hkv: int
    head_dim: int
    kv_len: Tuple[int, int]           # inclusive range of prefix lengths
    accept: str                       # "greedy" | "rejection" | "mixed" | "deterministic" | "mixed3"
    temperature: float
    peaked_frac: Tuple[float, float] = (0.6, 0.6)   # per-sequence fraction of peaked rows
    boost_prob: float = 0.9
    stick_prob: float = 0.95

    @property
    def alpha(self) -> int:
        return (self.d_base + 1) // 2

    def scaled(self, **kw) -> "VerifyConfig":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, VerifyConfig] = {
    "c1_tiny": VerifyConfig("c1_tiny", 1, 32000, (60, 60), 6, 6, 10, 60, "random", "f32", "uniform",
                            32, 32, 128, (512, 512), "greedy", 0.0),
    "c2_8b": VerifyConfig("c2_8b", 1, 128256, (60, 60), 8, 8, 10, 60, "eagle", "bf16", "mix",
                          32, 8, 128, (2048, 2048), "greedy", 0.0),
    "c3_70b": VerifyConfig("c3_70b", 1, 128256, (60, 60), 8, 8, 10, 60, "eagle", "bf16", "mix",
                           64, 8, 128, (4096, 4096), "rejection", 1.0),
    "c4_ragged": VerifyConfig("c4_ragged", 16, 128256, (8, 60), 8, 8, 10, 60, "eagle", "bf16", "mix",
                              32, 8, 128, (1024, 8192), "mixed", 1.0, peaked_frac=(0.0, 1.0)),
    "c5_long": VerifyConfig("c5_long", 4, 128256, (96, 96), 12, 8, 10, 60, "eagle", "bf16", "mix",
                            64, 8, 128, (32768, 32768), "rejection", 0.7),
}

# ----------------------------------------------------------------------------
# rows of logits
# ----------------------------------------------------------------------------


def _row_kind(cfg: VerifyConfig, seed: int, b: int, uid: int, peaked_frac: float, lead: bool = False):
    """(scale, peaked) of the row after node ``uid``.  ``lead`` marks the most likely child of a
    peaked node: it stays peaked with probability ``cfg.stick_prob`` (predictable stretches of
    text persist over several tokens), every other node is peaked with probability
    ``peaked_frac``."""
    r = _rng(seed, _K_TEMP, b, uid)
    if cfg.scale_kind == "uniform":
        return float(r.uniform(0.2, 4.0)), False
    u0, u1 = r.random(), r.random()
    peaked = bool(u0 < cfg.stick_prob) if lead else bool(u1 < peaked_frac)
    return ((1.0 / 0.3) if peaked else (1.0 / 3.0)), peaked


def _store(cfg: VerifyConfig, x: np.ndarray) -> np.ndarray:
    """Round to the storage dtype; returns the float32 value actually stored."""
    x = x.astype(np.float32)
    if cfg.logits_dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x))
    return x


def draft_row(cfg: VerifyConfig, seed: int, b: int, uid: int, peaked_frac: float,
              lead: bool = False) -> np.ndarray:
    """Draft logits after node ``uid``: scale * N(0,1), rounded to the storage dtype.

    In the peaked/flat mix a peaked row (temperature 0.3) also gets a head of three tokens, as
    language-model rows have: the first is placed U[0, 3.5] above the log-sum-exp of the
    Gaussian body (top-1 probability 0.5 .. 0.97), the next two 1-3 and a further 0.5-2 below.
    Without a head the Gaussian body gives top-1 probabilities of a few percent and the
    expansion of Sec. 2.2 never grows deeper than two levels."""
    s, peaked = _row_kind(cfg, seed, b, uid, peaked_frac, lead)
    r = _rng(seed, _K_ROW, b, uid)
    x = r.standard_normal(cfg.vocab, dtype=np.float32) * np.float32(s)
    if peaked:
        x64 = x.astype(np.float64)
        m = x64.max()
        lse = m + np.log(np.exp(x64 - m).sum())
        head = r.choice(cfg.vocab, size=3, replace=False)
        v0 = lse + r.uniform(0.0, 3.5)
        v1 = v0 - r.uniform(1.0, 3.0)
        v2 = v1 - r.uniform(0.5, 2.0)
        x[head] = np.array([v0, v1, v2], dtype=np.float32)
    return _store(cfg, x)


def target_row(cfg: VerifyConfig, seed: int, b: int, uid: int, peaked_frac: float,
               draft: np.ndarray, boost_token: int, lead: bool = False) -> np.ndarray:
    """Target logits after node ``uid``: the draft row plus noise of half its scale; with
    probability ``boost_prob`` the logit of ``boost_token`` (token of the most confident
    child) is raised two units above the row maximum so that accepted paths have a
    realistic length."""
    s, _ = _row_kind(cfg, seed, b, uid, peaked_frac, lead)
    z = _rng(seed, _K_TARGET, b, uid).standard_normal(cfg.vocab, dtype=np.float32)
    t = draft + np.float32(0.5 * s) * z
    if boost_token >= 0 and _rng(seed, _K_BOOST, b, uid).random() < cfg.boost_prob:
        t[boost_token] = t.max() + np.float32(2.0)
    return _store(cfg, t)


def _log_softmax64(row: np.ndarray) -> np.ndarray:
    x = row.astype(np.float64)
    m = x.max()
    return x - (m + np.log(np.exp(x - m).sum()))


def _topk_tokens(row: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries, ordered by (value descending, index ascending)."""
    k = min(k, row.shape[0])
    kth = np.partition(row, row.shape[0] - k)[row.shape[0] - k]
    cand = np.nonzero(row >= kth)[0]
    order = np.lexsort((cand, -row[cand].astype(np.float64)))
    return cand[order][:k].astype(np.int64)


# ----------------------------------------------------------------------------
# draft trees
# ----------------------------------------------------------------------------


class _RowCache:
    def __init__(self, cfg, seed, b, peaked_frac):
        self.cfg, self.seed, self.b, self.pf = cfg, seed, b, peaked_frac
        self.rows: Dict[int, np.ndarray] = {}
        self.lead: Dict[int, bool] = {}

    def peaked(self, uid: int) -> bool:
        return _row_kind(self.cfg, self.seed, self.b, uid, self.pf, self.lead.get(uid, False))[1]

    def __call__(self, uid: int) -> np.ndarray:
        if uid not in self.rows:
            self.rows[uid] = draft_row(self.cfg, self.seed, self.b, uid, self.pf,
                                       self.lead.get(uid, False))
        return self.rows[uid]


def _eagle_tree(cfg: VerifyConfig, n: int, rows: _RowCache):
    """Expansion to ``draft_depth`` with top-k children of the k most confident frontier
    nodes per level, then reranking to the n most confident nodes (root included)."""
    k = cfg.top_k
    par, tok, dep, S = [-1], [-1], [0], [0.0]
    frontier = [0]
    for level in range(1, cfg.draft_depth + 1):
        new: List[int] = []
        for p in frontier:
            row = rows(p)
            lp = _log_softmax64(row)
            for j, t in enumerate(_topk_tokens(row, k)):
                par.append(p); tok.append(int(t)); dep.append(level); S.append(S[p] + float(lp[t]))
                new.append(len(par) - 1)
                rows.lead[len(par) - 1] = (j == 0) and rows.peaked(p)
        frontier = sorted(new, key=lambda u: (-S[u], u))[:k]
    order = sorted(range(1, len(par)), key=lambda u: (-S[u], u))[: n - 1]
    keep = set(order) | {0}
    for u in list(keep):                      # ancestor closure (holds already: S is non-increasing)
        while u != -1 and u not in keep:
            keep.add(u); u = par[u]
    uids = sorted(keep)[:n] if len(keep) > n else sorted(keep)
    return uids, par, tok, dep


def _random_tree(cfg: VerifyConfig, seed: int, b: int, n: int, rows: _RowCache):
    """Random parent pointers: each new node hangs under a uniformly drawn earlier node whose
    depth is below ``draft_depth`` and which has fewer than ``top_k`` children; the j-th child
    of a node carries the j-th most likely token of the node's draft row."""
    r = _rng(seed, _K_TREE, b)
    par, dep, nchild = [-1], [0], [0]
    for i in range(1, n):
        ok = [u for u in range(i) if dep[u] < cfg.draft_depth and nchild[u] < cfg.top_k]
        p = ok[int(r.integers(len(ok)))]
        par.append(p); dep.append(dep[p] + 1); nchild.append(0); nchild[p] += 1
    tok = [-1] * n
    seen = [0] * n
    tops: Dict[int, np.ndarray] = {}
    for i in range(1, n):
        p = par[i]
        if p not in tops:
            tops[p] = _topk_tokens(rows(p), cfg.top_k)
        tok[i] = int(tops[p][seen[p]]); seen[p] += 1
    return list(range(n)), par, tok, dep


# ----------------------------------------------------------------------------
# one sequence, one batch
# ----------------------------------------------------------------------------


def make_sequence(cfg: VerifyConfig, seed: int, b: int, with_logits: bool = True,
                  with_attention: bool = True) -> dict:
    rs = _rng(seed, _K_SEQ, b)
    n = int(rs.integers(cfg.n_nodes[0], cfg.n_nodes[1] + 1))
    L = int(rs.integers(cfg.kv_len[0], cfg.kv_len[1] + 1))
    pf = float(rs.uniform(cfg.peaked_frac[0], cfg.peaked_frac[1]))
    rows = _RowCache(cfg, seed, b, pf)
    if cfg.tree_kind == "eagle":
        uids, par, tok, dep = _eagle_tree(cfg, n, rows)
    else:
        uids, par, tok, dep = _random_tree(cfg, seed, b, n, rows)
    n = len(uids)
    local = {u: i for i, u in enumerate(uids)}
    parent = np.array([-1 if par[u] < 0 else local[par[u]] for u in uids], dtype=np.int32)
    token = np.array([max(tok[u], 0) for u in uids], dtype=np.int32)
    depth = np.array([dep[u] for u in uids], dtype=np.int32)
    out = dict(n=n, kv_len=L, parent=parent, token=token, depth=depth, peaked_frac=pf)
    if with_logits:
        draft = np.stack([rows(u) for u in uids])
        # the most confident child of every internal node (first child in creation order has
        # the largest draft probability, because children are emitted in top-k order)
        first_child = np.full(n, -1, dtype=np.int64)
        for i in range(n - 1, 0, -1):
            first_child[parent[i]] = i
        target = np.empty_like(draft)
        for i, u in enumerate(uids):
            bt = int(token[first_child[i]]) if first_child[i] >= 0 else -1
            target[i] = target_row(cfg, seed, b, u, pf, draft[i], bt, rows.lead.get(u, False))
        out["draft"], out["target"] = draft, target
    if with_attention:
        ra = _rng(seed, _K_ATTN, b)
        D = cfg.head_dim
        g = lambda *shape: f32_to_bf16_bits(ra.standard_normal(shape, dtype=np.float32))
        out["q"] = g(n, cfg.hq, D)
        out["k_tree"] = g(n, cfg.hkv, D)
        out["v_tree"] = g(n, cfg.hkv, D)
        out["k_cache"] = g(L, cfg.hkv, D)
        out["v_cache"] = g(L, cfg.hkv, D)
    return out


SALT_STRIDE = 1_000_003


def make_batch(cfg: VerifyConfig, seed: int, with_logits: bool = True,
               with_attention: bool = True, salts=None) -> dict:
    """A ragged batch in CSR form.  Logits and Q/K/V of tree nodes are laid out by original
    node index (row ``node_off[b] + i`` belongs to node i of sequence b).  Logits are float32
    values for ``logits_dtype == "f32"`` and uint16 bfloat16 bit patterns otherwise.
    ``salts[b]`` (default 0) re-draws sequence b alone: it is generated from
    ``seed + salts[b] * SALT_STRIDE``."""
    salts = list(salts) if salts is not None else [0] * cfg.batch
    seqs = [make_sequence(cfg, seed + salts[b] * SALT_STRIDE, b, with_logits, with_attention)
            for b in range(cfg.batch)]
    cat = lambda key: np.concatenate([s[key] for s in seqs], axis=0)
    node_off = np.zeros(cfg.batch + 1, dtype=np.int32)
    node_off[1:] = np.cumsum([s["n"] for s in seqs])
    kv_off = np.zeros(cfg.batch + 1, dtype=np.int32)
    kv_off[1:] = np.cumsum([s["kv_len"] for s in seqs])
    batch = dict(cfg=cfg, seed=seed, salts=salts, node_off=node_off, kv_off=kv_off,
                 parent=cat("parent"), token=cat("token"), depth=cat("depth"))
    if with_logits:
        draft, target = cat("draft"), cat("target")
        if cfg.logits_dtype == "bf16":
            draft, target = f32_to_bf16_bits(draft), f32_to_bf16_bits(target)
        batch["draft"], batch["target"] = draft, target
    if with_attention:
        for key in ("q", "k_tree", "v_tree", "k_cache", "v_cache"):
            batch[key] = cat(key)
    if cfg.accept == "greedy":
        mode = np.zeros(cfg.batch, dtype=np.int32)
    elif cfg.accept == "rejection":
        mode = np.ones(cfg.batch, dtype=np.int32)
    elif cfg.accept == "deterministic":
        mode = np.full(cfg.batch, 2, dtype=np.int32)
    elif cfg.accept == "mixed3":
        mode = (np.arange(cfg.batch) % 3).astype(np.int32)
    else:
        mode = (np.arange(cfg.batch) % 2).astype(np.int32)
    batch["mode"] = mode
    batch["temperature"] = np.where(mode != 0, cfg.temperature, 0.0).astype(np.float32)
    batch["philox_seed"] = (int(seed) * 0x9E3779B97F4A7C15 + 0x1234567) & (2**64 - 1)
    batch["philox_offset"] = 0
    return batch


def default_policy(cfg: VerifyConfig, thresholds) -> dict:
    """Policy table of Sec. 4.2-4.3: seven ascending entropy thresholds (an input: the paper's
    own trained values are not published), base depth, alpha = ceil(depth / 2), default Top-N,
    K, and the gamma factors 0.3 / 0.6 / 1.0 in percent."""
    return dict(thresholds=[float(t) for t in thresholds], d_base=cfg.d_base, alpha=cfg.alpha,
                n_default=cfg.n_default, top_k=cfg.top_k, gamma_pct=[30, 60, 100],
                phi_mode=0, pstar_mode=0, entropy_mode=0)
