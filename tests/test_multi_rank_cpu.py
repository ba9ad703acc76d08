"""The multi-GPU path of bench.py without GPUs: two gloo ranks on the CPU run the pieces that
differ from the single-rank run -- per-rank workloads (different seeds, hence different data),
the max-over-ranks timing reduction and the whole-job throughput."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from workloads.synthetic import CONFIGS, BatchStream
    w = bench.rank_workload(CONFIGS["tiny"], rank)
    q, k, v = BatchStream(w, 0).next(4)
    # each rank pretends to have measured its own times: rank r is (1 + r) times slower
    ms = [10.0 * (1 + rank), 5.0 * (1 + rank), 20.0 * (1 + rank)]
    mx = bench.max_over_ranks(ms, world, torch.device("cpu"))
    out[rank] = {"seed": w.seed, "q0": float(q[0, 0, 0, 0]), "max": mx,
                 "value": bench.job_tokens_per_s(w.batch, 100, world, mx[0])}
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_batch_and_reduce_by_max():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["seed"] != res[1]["seed"] and res[0]["q0"] != res[1]["q0"]      # independent batches
    for r in (0, 1):
        assert res[r]["max"] == [20.0, 10.0, 40.0]                                  # the slowest rank's times
        np.testing.assert_allclose(res[r]["value"], 2 * 1 * 100 / 20e-3)            # all ranks' tokens / max time
