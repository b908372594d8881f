"""Writes tests/golden/thresholds.json: the seven entropy thresholds used by the tests and the
benchmark for each synthetic workload.

The paper trains its thresholds with a CART regression on (Phi(P*), Terminal Confidence Rank)
pairs collected from real decoding runs (Sec. 4.2) and does not print them.  They are therefore
an input of the verification path; the values stored here are the octiles (12.5 % ... 87.5 %) of
Phi(P*) over a calibration set of seeded synthetic trees, so that all eight bins occur.

Calls only the input generators and the CPU oracle.  Usage:  python tests/golden/make_thresholds.py
"""
import json
import multiprocessing as mp
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from oracle import row_stats, tree  # noqa: E402
from paper_2505_13254_b200 import synth  # noqa: E402

CAL_SEED0 = 1_000_000          # calibration seeds are disjoint from the seeds tests use
N_SEQ = 256


def phi_star(args):
    name, seed, b = args
    cfg = synth.CONFIGS[name]
    s = synth.make_sequence(cfg, seed, b, with_logits=True, with_attention=False)
    logits = s["draft"].astype(np.float64)
    pol = synth.default_policy(cfg, [0.0] * 7)
    internal = set(int(p) for p in s["parent"] if p >= 0)
    blank = dict(I_topk=0.0, I_trunc=0.0, lse=0.0)
    stats = [row_stats.row_stats(logits[i], cfg.top_k) if i in internal else blank for i in range(s["n"])]
    return tree.tree_scores(s["parent"], s["token"], logits, pol, stats=stats)["phi_star"]


def main():
    out = {}
    with mp.Pool(min(8, os.cpu_count() or 1)) as pool:
        for name, alias in (("c1_tiny", ()), ("c2_8b", ("c3_70b",)), ("c4_ragged", ()), ("c5_long", ())):
            cfg = synth.CONFIGS[name]
            jobs = [(name, CAL_SEED0 + i // cfg.batch, i % cfg.batch) for i in range(N_SEQ)]
            phis = np.array(pool.map(phi_star, jobs))
            th = np.quantile(phis, np.arange(1, 8) / 8.0)
            entry = dict(thresholds=[round(float(t), 4) for t in th], calibration_sequences=N_SEQ,
                         phi_star_min=float(phis.min()), phi_star_max=float(phis.max()))
            out[name] = entry
            for a in alias:                      # same trees and logits, other attention shape
                out[a] = entry
            print(name, entry, flush=True)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "thresholds.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    main()
