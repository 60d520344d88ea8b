"""The multi-rank bookkeeping of bench.py, on CPU with two gloo ranks: ranks
draw different images, the job time is the maximum over ranks, and the value is
the work of all ranks over that time."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    import bench
    from paper_2206_10620_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = wl.config_single_layer()[0]
    d = wl.make_layer(spec, seed=bench.rank_seed(rank))
    local_ms = 1.0 + rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
    val = bench.whole_job_gflops(spec.useful_macs(), world, ms)
    out.put((rank, ms, val, float(d.x.sum()), float(d.w.sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks():
    import torch.multiprocessing as mp
    from paper_2206_10620_b200 import workloads as wl
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, v0, x0, w0), (r1, ms1, v1, x1, w1) = res
    assert ms0 == ms1 == 2.0                   # the slowest rank's time, on both ranks
    spec = wl.config_single_layer()[0]
    assert v0 == v1 == pytest.approx(2.0 * spec.useful_macs() * 2 / 2e-3 / 1e9)
    assert x0 != x1                            # different images per rank


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.rank_seed(0) != bench.rank_seed(1)
