#!/usr/bin/env python
"""Benchmark of one HeteroSpec verification step (quantify -> stratify/prune -> tree attention ->
accept) on synthetic inputs shaped like the Llama-3.1-8B workload.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload c2_8b]

Prints ONE JSON line.  A "step" is one pass of the whole path over one batch; inputs rotate through
several distinct device copies whose total size exceeds the L2 cache, so every step reads HBM.
With N > 1 (torchrun) every rank verifies its own batch (independent trees: no collective on the
data path) and the slowest rank's time is used.  `--impl reference` times the CPU oracle instead.
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "verified_draft_trees_per_second"
UNIT = "trees/s"
L2_BYTES = 126 << 20
NOMINAL_HBM_GBS = 8000.0          # the part's nominal HBM3e bandwidth
NOMINAL_BF16_TFLOPS = 2250.0      # nominal dense bf16


def workload_config(cfg):
    """The workload's description, identical in both arms of the benchmark."""
    return {"workload": cfg.name, "batch_per_gpu": cfg.batch, "tree_nodes": list(cfg.n_nodes), "vocab": cfg.vocab,
            "logits_dtype": cfg.logits_dtype, "kv_len": list(cfg.kv_len), "hq": cfg.hq, "hkv": cfg.hkv,
            "head_dim": cfg.head_dim, "attention_layers_per_step": 1, "accept": cfg.accept}


def oracle_threads():
    """Threads the numpy oracle can use: its loops are single-threaded python; only BLAS calls (the
    matrix-vector products of the attention) may use the BLAS pool."""
    try:
        from threadpoolctl import threadpool_info
        n = max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        n = 1
    return n


def load_policy(cfg, synth):
    th = json.load(open(os.path.join(ROOT, "tests", "golden", "thresholds.json")))
    return synth.default_policy(cfg, th[cfg.name]["thresholds"])


def ncu_traffic(kernel, workload):
    """DRAM bytes per launch of `kernel` from the committed ncu capture, or None if there is none or the
    kernel's source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None
    ent = json.load(open(path)).get(kernel, {}).get(workload)
    if not ent:
        return None
    src = os.path.join(ROOT, "paper_2505_13254_b200", "csrc", ent["source"])
    if hashlib.sha1(open(src, "rb").read()).hexdigest() != ent["source_sha1"]:
        return None
    return ent["dram_bytes_per_launch"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak():
    """Dense bf16 TFLOP/s of this machine's B200s (burst figure: the kernel is timed alone)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["bf16_tflops"])
    return 1590.0


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


def rank_seed(rank):
    """Seed of the batch a rank verifies: every rank gets its own independent trees."""
    return int(rank)


def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank defines the time)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(world, batch_per_rank, steps, ms):
    """Trees verified per second by all ranks together: units all ranks processed / slowest rank's time."""
    return world * batch_per_rank * steps / (ms * 1e-3)


def oracle_sample(batch, policy, ostep):
    """One tree through the whole oracle path (all rows, all attention pairs of the kept nodes)."""
    t = time.perf_counter()
    ostep.verify_step(batch, policy, with_attention=True)
    return time.perf_counter() - t


def run_reference(args, cfg, synth):
    from oracle import step as ostep
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    policy = load_policy(cfg, synth)
    batch = synth.make_batch(cfg, 0)
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_sample(batch, policy, ostep)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = cfg.batch * len(times) / total
    cores = oracle_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "each step = the whole batch through the numpy fp64 oracle (all logits rows, "
                                       "all kept-node attention pairs of one layer); python loops on one core, BLAS "
                                       "calls on `cores` threads (host has %d cores)" % (os.cpu_count() or 0)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_8b")
    ap.add_argument("--rotate", type=int, default=0, help="distinct input copies (0 = enough to exceed 2x L2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prefetch", default="all", choices=["none", "kv", "all"],
                    help="inputs the kernels may fetch before their dependency wait (hs_set_prefetch): the benchmark's "
                         "logits and KV cache are resident and never written by the kernel ahead of a call")
    ap.add_argument("--accept", default=None, choices=["greedy", "rejection", "mixed", "deterministic", "mixed3"],
                    help="acceptance mode(s) of the sequences instead of the workload's own")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2505_13254_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    if args.accept:
        cfg = cfg.scaled(accept=args.accept, temperature=cfg.temperature or 1.0)
    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 5                 # bounded: a step is seconds of CPU work
            args.warmup = min(args.warmup, 1)
        return run_reference(args, cfg, synth)

    import torch
    import torch.distributed as dist
    from paper_2505_13254_b200 import binding as hb
    from paper_2505_13254_b200 import step as gstep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    policy = load_policy(cfg, synth)
    batch = synth.make_batch(cfg, rank_seed(rank))           # each rank verifies its own trees
    db0 = gstep.upload(batch, dev)
    per_set = db0.nbytes()
    R = args.rotate or max(2, -(-2 * L2_BYTES // per_set) + 1)
    sets = [db0]
    for _ in range(R - 1):
        c = gstep.upload(batch, dev)
        sets.append(c)
    ws = hb.hs_workspace_bytes(cfg.batch, db0.tree.n_nodes_total, cfg.vocab, cfg.hq, cfg.hkv)
    ctx = hb.Context(local, ws)
    hb.hs_set_prefetch(ctx, {"none": 0, "kv": hb.HS_PREFETCH_KV, "all": hb.HS_PREFETCH_KV | hb.HS_PREFETCH_LOGITS}[args.prefetch])
    st = gstep.VerifyStep(ctx, db0, policy)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----------------------------------------------------------------------
    # The four calls of a step are captured once per input copy into a CUDA graph (R steps per graph), so the
    # timed region replays launches without any Python or ctypes work in between.
    for i in range(max(args.warmup, R)):
        st.run(sets[i % R])
    barrier()

    def capture(fn, count):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(count):
                fn(sets[i % R])
        return g

    def timed_replays(fn, steps):
        """Times exactly `steps` invocations of fn (rotating over the input copies) as graph replays."""
        full, rest = divmod(steps, R)
        g_full = capture(fn, R) if full else None
        g_rest = capture(fn, rest) if rest else None
        for _ in range(2):
            (g_full or g_rest).replay()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(full):
            g_full.replay()
        if g_rest:
            g_rest.replay()
        b.record()
        barrier()
        return a.elapsed_time(b)

    sampler = ClockSampler(local) if rank == 0 else None
    ms = timed_replays(lambda db: st.run(db), args.steps)
    # ---- per-call durations: each call alone, back to back over the rotating inputs ------------------------
    calls = ("quantify", "prune", "quantify_prune", "attention", "accept_path")
    call_us = {c: 1e3 * timed_replays(getattr(st, c), args.steps) / args.steps for c in calls}
    st.run(sets[0])
    barrier()
    clocks = sampler.stop() if sampler else None
    nk = int(st.pruned.n_keep.sum().item())
    n_rows = db0.tree.n_nodes_total

    # ---- end to end: pinned host inputs -> device, the four calls, results -> host, every step -----------
    host = {}
    names = ("draft", "target", "q", "k_tree", "v_tree", "k_cache", "v_cache")
    for n in names:
        host[n] = getattr(db0, n).cpu().pin_memory()
    for n in ("node_off", "parent", "token"):
        host[n] = getattr(db0.tree, n).cpu().pin_memory()
    res_host = {n: getattr(st.accept, n).cpu().pin_memory() for n in ("accept_len", "path_tokens", "bonus_token")}
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in res_host.values())
    # Two staging copies of the inputs on the device and two result buffers on the host: the copies of step n + 1
    # run on a second stream while the kernels of step n run; every step still copies all of its inputs from pinned
    # memory and its results are read back (and waited for) on the host before step n + 2 may reuse the buffers.
    stages = [sets[-1], sets[-2]]
    res_hosts = [res_host, {n: t.clone().pin_memory() for n, t in res_host.items()}]
    copy_stream = torch.cuda.Stream(device=dev)
    main_stream = torch.cuda.current_stream(dev)
    copied = [torch.cuda.Event() for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]

    def e2e_issue(i):
        k = i & 1
        stage = stages[k]
        with torch.cuda.stream(copy_stream):
            if i >= 2:
                copy_stream.wait_event(done[k])              # the kernels of step i - 2 are done with this copy
            for n in names:
                getattr(stage, n).copy_(host[n], non_blocking=True)
            for n in ("node_off", "parent", "token"):
                getattr(stage.tree, n).copy_(host[n], non_blocking=True)
            copied[k].record(copy_stream)
        main_stream.wait_event(copied[k])
        st.run(stage)
        for n, t in res_hosts[k].items():
            t.copy_(getattr(st.accept, n), non_blocking=True)
        done[k].record(main_stream)

    def e2e_loop(count):
        for i in range(count):
            if i >= 2:
                done[i & 1].synchronize()                    # the host has the results of step i - 2
            e2e_issue(i)
        torch.cuda.synchronize()

    e2e_steps = min(args.steps, 100)
    e2e_loop(4)
    barrier()
    t0 = time.perf_counter()
    e2e_loop(e2e_steps)
    e2e_s = time.perf_counter() - t0
    barrier()

    ms, e2e_s = max_over_ranks([ms, e2e_s], dev, world)
    dev_err = hb.hs_device_error(ctx)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    esz = 2 if cfg.logits_dtype == "bf16" else 4
    quant_bytes = n_rows * cfg.vocab * esz
    L = int(np.diff(batch["kv_off"]).sum())
    attn_bytes = 2 * (L + nk) * cfg.hkv * cfg.head_dim * 2 + 2 * nk * cfg.hq * cfg.head_dim * 2
    # rows the acceptance reads: the target row of every kept node and, in rejection mode, the draft row of every kept
    # node that has a kept child
    koff, npar, modes = st.pruned.keep_off.cpu().numpy(), st.pruned.new_parent.cpu().numpy(), db0.mode.cpu().numpy()
    draft_rows = sum(len(set(int(x) for x in npar[koff[b]:koff[b + 1]] if x >= 0))
                     for b in range(cfg.batch) if modes[b] == hb.HS_ACCEPT_REJECTION and db0.any_sampling)
    accept_bytes = (nk + draft_rows) * cfg.vocab * esz
    kern = {
        "quantify": {"bytes": quant_bytes, "us": call_us["quantify"], "launches_per_step": 2},
        "attention": {"bytes": attn_bytes, "us": call_us["attention"], "launches_per_step": 1},
        "accept_path": {"bytes": accept_bytes, "us": call_us["accept_path"],
                        "launches_per_step": 2 if db0.any_sampling else 1},
        "prune": {"bytes": 0, "us": call_us["prune"], "launches_per_step": 1},
        # what a step runs in place of the two calls above: the entropy pass, then tree scores + pruning in one kernel
        "quantify_prune": {"bytes": quant_bytes, "us": call_us["quantify_prune"], "launches_per_step": 2},
    }
    for name in ("quantify", "prune"):
        kern[name]["in_step"] = False          # timed alone for comparison; the step makes the fused call
    for k in kern.values():
        k["gbs"] = k["bytes"] / (k["us"] * 1e-6) / 1e9 if k["us"] > 0 else None
        k["frac_of_%s_hbm" % peak_kind] = k["gbs"] / peak if k["gbs"] else None
        k["frac_of_nominal_hbm"] = k["gbs"] / NOMINAL_HBM_GBS if k["gbs"] else None
    traffic = ncu_traffic("quantify_stream_kernel", cfg.name)
    achieved = kern["quantify"]["gbs"]
    line = {
        "metric": METRIC, "value": whole_job_value(world, cfg.batch, args.steps, ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(cfg),
        "run": {"tree_nodes_total": n_rows, "kept_nodes_total": nk, "parallelism": "replicas" if world > 1 else "single",
                "prefetch": args.prefetch,
                "l2": "inputs rotate through %d distinct device copies, %.0f MB in total (L2 = 126 MB)"
                      % (R, R * per_set / 1e6)},
        "clocks": clocks,
        "e2e": {"value": world * cfg.batch * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * e2e_s / e2e_steps,
                "how": "every step copies all inputs from pinned host memory and reads its results back; the copies of "
                       "step n + 1 overlap the kernels of step n (two staging buffers, two streams)"},
        "gpu_launches": (5 if db0.any_sampling else 4) * args.steps,
        "roofline": {"kernel": "quantify_stream_kernel (hs_entropy_quantify: this kernel + the tree stage)", "bound": "hbm",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                     "peak_kind": peak_kind + " (burst copy figure)", "traffic": traffic,
                     "algorithmic_bytes_per_launch": quant_bytes,
                     "how": "CUDA events around K back-to-back graph-replayed calls of hs_entropy_quantify alone (both of its "
                            "launches in the duration), inputs rotating; with programmatic dependent launch and prefetch "
                            "allowed, the row pass of one call overlaps the tree stage of the call before it"},
        "calls": kern,
        "device_error_word": dev_err,
    }
    a_gbs = kern["attention"]["gbs"]
    # Q K^T and P V of every kept row against its sequence's prefix and tree: 4 * 128 flops per (row, key) pair
    kv_len = np.diff(batch["kv_off"]).astype(np.int64)
    nk_b = st.pruned.n_keep.cpu().numpy().astype(np.int64)[: len(kv_len)]
    attn_flops = float(4 * cfg.head_dim * cfg.hq * (nk_b * (kv_len + nk_b)).sum())
    a_tflops = attn_flops / (kern["attention"]["us"] * 1e-6) / 1e12
    tf_peak = tensor_peak()
    if attn_flops / (tf_peak * 1e12) > attn_bytes / (peak * 1e9):      # the tensor pipe is the longer leg
        line["roofline_attention"] = {"kernel": "tree_attn_umma_kernel (hs_tree_verify_attention, one launch per step)",
                                      "bound": "tensor", "achieved": a_tflops, "peak": tf_peak, "unit": "TFLOP/s",
                                      "frac": a_tflops / tf_peak, "frac_of_nominal": a_tflops / NOMINAL_BF16_TFLOPS,
                                      "peak_kind": peak_kind + " (dense bf16 burst figure)",
                                      "traffic": ncu_traffic("tree_attn_umma_kernel", cfg.name),
                                      "algorithmic_flops_per_launch": attn_flops,
                                      "algorithmic_bytes_per_launch": attn_bytes}
    else:
        line["roofline_attention"] = {"kernel": "tree_attn_umma_kernel (hs_tree_verify_attention, one launch per step)",
                                      "bound": "hbm", "achieved": a_gbs, "peak": peak, "unit": "GB/s",
                                      "frac": a_gbs / peak if a_gbs else None,
                                      "frac_of_nominal": a_gbs / NOMINAL_HBM_GBS if a_gbs else None,
                                      "peak_kind": peak_kind + " (burst copy figure)",
                                      "traffic": ncu_traffic("tree_attn_umma_kernel", cfg.name),
                                      "algorithmic_bytes_per_launch": attn_bytes,
                                      "algorithmic_flops_per_launch": attn_flops}
    # ---- a graph per regime (Sec. 4.3): the same tree forced into the lowest and into the highest entropy bin ---------
    if world == 1:
        regimes = {}
        for name, th in (("bin0", 1e9), ("bin7", -1e9)):
            pol = dict(policy, thresholds=[th] * 7)
            st_r = gstep.VerifyStep(ctx, db0, pol)
            rs = gstep.RegimeStep(st_r, db0)
            one = gstep.GraphedStep(st_r, db0)
            n_rep = min(args.steps, 300)

            def wall(fn):
                for _ in range(5):
                    fn()
                torch.cuda.synchronize()
                t = time.perf_counter()
                for _ in range(n_rep):
                    fn()
                torch.cuda.synchronize()
                return 1e6 * (time.perf_counter() - t) / n_rep
            regimes[name] = {"kept_nodes": int(st_r.pruned.n_keep.sum().item()), "graph_bound": rs.last_bound,
                             "two_phase_us": wall(rs.replay), "one_graph_us": wall(one.replay)}
        line["regime_graphs"] = dict(regimes, how="wall clock per step over back-to-back replays on one input copy (L2-warm); "
                                     "two_phase = quantify + prune, the host reads the kept-node count, then the regime's own "
                                     "graph of attention + acceptance; one_graph = all calls in one graph sized by the drafted tree (the attention: by the most the policy keeps)")
    if not args.no_cpu_baseline:
        from oracle import step as ostep
        nrep = 5
        t = sum(oracle_sample(synth.make_batch(cfg, rank_seed(rank) + 1000 * i) if i else batch, policy, ostep)
                for i in range(nrep))
        line["cpu_baseline"] = {"value": nrep * cfg.batch / t, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": "%d batches of this workload (seeds differ) once each through the numpy fp64 "
                                          "oracle: all logits rows, all kept-node attention pairs of one layer (%.1f s)"
                                          % (nrep, t)}
    print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
