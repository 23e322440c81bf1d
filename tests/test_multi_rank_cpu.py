"""Host-side logic of the N > 1 benchmark path on CPU ranks (gloo, world size 2): the path is
"replicas only" -- every rank runs the same independent workload, the time is the maximum over
ranks and the value the sum of the ranks' bytes over that time."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        ms = bench.max_over_ranks(ms_local, world, device="cpu")
        value = bench.replica_value(bytes_per_step=1_000_000, world=world, ms_per_step=ms)
        out.put((rank, ms, value))
    finally:
        dist.barrier()
        dist.destroy_process_group()


def test_two_rank_replica_timing_and_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29731, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == pytest.approx(15.0)                  # the maximum over ranks, on every rank
        assert value == pytest.approx(2 * 1_000_000 / 15.0e-3 / 1e9)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.replica_value(2_000_000_000, 1, 1.0) == pytest.approx(2000.0)
