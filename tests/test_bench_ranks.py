"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own trees, no collective on the
data path, the slowest rank's time defines the whole-job throughput."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2505_13254_b200 import synth

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = synth.CONFIGS["c1_tiny"].scaled(vocab=512, n_nodes=(12, 12))
    batch = synth.make_batch(cfg, bench.rank_seed(rank), with_attention=False)
    ms_local = 10.0 * (rank + 1)                       # rank 1 is the slow one
    ms, e2e = bench.max_over_ranks([ms_local, 2.0 * ms_local], torch.device("cpu"), world)
    out[rank] = (ms, e2e, batch["token"].tolist(), bench.whole_job_value(world, cfg.batch, 100, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_trees_and_take_the_slowest_time():
    world, port = 2, 29000 + os.getpid() % 1000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] == 20.0 and r0[1] == r1[1] == 40.0        # max over ranks, on every rank
    assert r0[2] != r1[2]                                          # different trees per rank
    assert np.isclose(r0[3], 2 * 1 * 100 / 20e-3)                   # all ranks' trees / slowest time
