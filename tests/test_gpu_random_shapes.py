"""Seeded random shapes, sparsities, skip fractions and CTA counts: both kernels against the oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    from paper_2607_21985_b200 import spdp
    spdp.lib()
    return spdp


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("seed", range(24))
def test_random_case(S, seed):
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    M = int(rng.integers(1, 2600))
    K = int(rng.integers(1, 9000)) if seed % 3 else int(rng.integers(1, 300))
    sp = float(rng.choice([0.0, 0.3, 0.5, 0.7, 0.9, 0.99]))
    skip = float(rng.choice([0.0, 0.25, 0.5, 0.9]))
    B = int(rng.integers(3, 9))
    W = (rng.standard_normal((M, K), dtype=np.float32) * 0.05)
    W[rng.random((M, K)) < sp] = 0
    if seed % 4 == 0:                                                  # whole columns / row tiles without a nonzero
        W[:, rng.random(K) < 0.3] = 0
        W[: min(M, 256)] = 0
    W = W.astype(np.float16)
    X = rng.standard_normal((B, K), dtype=np.float32).astype(np.float16)
    rule, thr = WL.skip_threshold(X[0], skip)
    acts = np.stack([O.active_ref(X[b], rule, thr) for b in range(B)])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    tol = O.tolerance(S_ref)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        want = O.pack_fast(W)
        got = S.spdp_export(h)
        for key in ("tileoffset", "colinfo", "bitmap", "values"):
            assert np.array_equal(got[key], want[key]), key
        for ctas in (0, int(rng.integers(1, 1025))):
            if ctas:
                S.spdp_set_num_ctas(h, ctas)
            y = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, dev(X[0]), rule, thr, y)
            Y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv_batch(h, dev(X), rule, thr, Y)
            torch.cuda.synchronize()
            assert S.spdp_last_device_status(h) == 0
            assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - Y_ref[0]) <= tol[0]), (M, K, sp, skip, ctas)
            assert np.all(np.abs(Y.cpu().numpy().astype(np.float64) - Y_ref) <= tol), (M, K, sp, skip, B, ctas)
    finally:
        S.spdp_free(h)
