"""Row-tile sharding: the split every rank agrees on, and the gather path on two gloo ranks (CPU).
The local product is the CPU oracle here, so the collective plumbing runs without a GPU; the gathered
result must equal the unsharded oracle result bit for bit (a row's sum does not depend on the split)."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_row_shard_covers_every_row_once_in_whole_tiles():
    from paper_2607_21985_b200 import build, spdp
    build.build()
    for M, world in [(28672, 8), (28672, 3), (300, 2), (256, 4), (1, 1), (1000, 7), (4096, 16), (11008, 8)]:
        parts = [spdp.spdp_row_shard(M, world, r) for r in range(world)]
        nxt = 0
        for first, rows in parts:
            assert first == nxt or rows == 0
            assert first % 256 == 0 or rows == 0
            nxt += rows
        assert nxt == M
        tiles = [-(-rows // 256) for _, rows in parts]
        assert max(tiles) - min(tiles) <= 1                       # balanced to within one row tile
    with pytest.raises(spdp.SpdpError):
        spdp.spdp_row_shard(100, 2, 2)


WORKER = textwrap.dedent("""
    import os, sys
    import numpy as np, torch, torch.distributed as dist
    sys.path.insert(0, {root!r})
    from oracle import spdp_oracle as O
    from paper_2607_21985_b200 import workloads as WL
    from paper_2607_21985_b200.sharded import RowShardedMatrix
    dist.init_process_group("gloo")
    w = WL.config4({M}, 1024, seed=9)
    a = O.active_ref(w.x, w.rule, w.thr)
    def local(handle, x, y_slice):                                  # the oracle stands in for the GPU product
        y, _ = O.spmspv_ref(handle, x.numpy(), a)
        y_slice.copy_(torch.from_numpy(y))
    sh = RowShardedMatrix(w.M, w.K, lambda r0, n: w.W[r0:r0 + n], lambda rows: rows, local,
                          device="cpu", dtype=torch.float64)
    y = sh.spmspv(torch.from_numpy(w.x))
    y_ref, _ = O.spmspv_ref(w.W, w.x, a)
    assert y.shape[0] == w.M and np.array_equal(y.numpy(), y_ref), "gathered result differs from the unsharded one"
    y2 = sh.spmspv(torch.from_numpy(w.x))                           # buffers are reused from call to call
    assert np.array_equal(y2.numpy(), y_ref)
    sys.stdout.write("rank %d rows %d SHARD_OK\\n" % (dist.get_rank(), sh.rows))          # one write per rank: lines do not interleave
    sys.stdout.flush()
    dist.destroy_process_group()
""")


@pytest.mark.parametrize("M", [2048, 1800])           # equal shards; ragged shards (4 + 4 tiles, the last one partial)
def test_two_gloo_ranks_gather_the_unsharded_result(tmp_path, M):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, M=M))
    import socket
    with socket.socket() as sock:                      # a port that is free right now
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-2000:]
    assert out.stdout.count("SHARD_OK") == 2
