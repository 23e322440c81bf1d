"""The benchmark's own byte model and its host-side N>1 plumbing (no GPU)."""
import json
import os
import subprocess
import sys

import numpy as np

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_active_bytes_equals_oracle_model():
    import bench
    for w in (WL.config1(512, 512), WL.config3(512, 1024), WL.config4(1024, 512), WL.config5(3, 0, 300, 100)):
        p = O.pack_fast(w.W)
        a = O.active_ref(w.x, w.rule, w.thr)
        for yb in (2, 4):
            assert bench.active_bytes(p["colinfo"], O.active_to_words(a), w.M, w.K, yb) == O.active_bytes(p, a, yb)


def test_reference_arm_prints_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--workload", "c1"], capture_output=True, text=True, check=True,
                         timeout=600).stdout
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]


def test_reference_arm_under_two_ranks_only_rank0_prints():
    """Launched the way the driver launches N > 1 (torch.distributed.run): rank 0 alone works."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29611", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1", "--workload", "c1"]
    out = subprocess.run(cmd, capture_output=True, text=True, check=True, timeout=900).stdout
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
