"""Prefill product on the packed handle (spdp_spmm, Sec. 4.3) against the oracle's dense fp64 definition."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2607_21985_b200 import spdp
    spdp.lib()
    return spdp


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run(S, h, X, M, ydtype=torch.float32):
    Y = torch.full((X.shape[0], M), float("nan"), dtype=ydtype, device="cuda")      # poison: every entry must be written
    S.spdp_spmm(h, dev(X), Y)
    torch.cuda.synchronize()
    assert S.spdp_last_device_status(h) == 0
    return Y.float().cpu().numpy().astype(np.float64)


def check(Y, Y_ref, S_ref):
    err = np.abs(Y - Y_ref)
    tol = O.tolerance(S_ref)                       # |y - y_ref| <= 1e-3 * S + 1e-5
    assert np.all(err <= tol), f"worst error/tolerance {np.nanmax(err / tol):.3g}"


@pytest.mark.parametrize("M,K,sp,seed", [(256, 16, 0.5, 1), (300, 40, 0.3, 2), (1, 8, 0.0, 3), (257, 24, 0.5, 4),
                                         (1024, 1024, 0.5, 5), (768, 4400, 0.7, 6), (2304, 528, 0.9, 7),
                                         (512, 72, 0.0, 8)])
@pytest.mark.parametrize("N", [1, 16, 128, 300])
def test_spmm_matches_oracle(S, M, K, sp, seed, N):
    rw, rx = WL._rngs(seed)
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), sp).astype(np.float16)
    X = rx.standard_normal((N, K), dtype=np.float32).astype(np.float16)
    Y_ref, S_ref = O.spmm_ref(W, X)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        for dt in (torch.float32, torch.float16):
            check(run(S, h, X, M, dt), Y_ref, S_ref)
        assert np.array_equal(run(S, h, X, M), run(S, h, X, M))          # the same bits from call to call
    finally:
        S.spdp_free(h)


def test_spmm_exact_on_integers_and_strided_tensors(S):
    rng = np.random.Generator(np.random.PCG64(61))
    M, K, N = 700, 904, 37
    W = rng.integers(-8, 9, (M, K)).astype(np.float16)
    W[rng.random((M, K)) < 0.6] = 0
    X = rng.integers(-4, 5, (N, K)).astype(np.float16)
    Y_ref, _ = O.spmm_ref(W, X)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        assert np.array_equal(run(S, h, X, M), Y_ref)                     # every partial sum is an exact integer
        Xd = torch.zeros((N, K + 24), dtype=torch.float16, device="cuda")  # padded row strides (a multiple of 8 elements)
        Xd[:, :K] = dev(X)
        Yd = torch.full((N, M + 5), float("nan"), dtype=torch.float32, device="cuda")
        S.spdp_spmm(h, Xd[:, :K], Yd[:, :M])
        torch.cuda.synchronize()
        out = Yd.cpu().numpy()
        assert np.array_equal(out[:, :M].astype(np.float64), Y_ref) and np.all(np.isnan(out[:, M:]))
        # one token agrees with the decode call without dynamic pruning
        y1 = torch.empty(M, dtype=torch.float32, device="cuda")
        S.spdp_spmspv(h, dev(X[3]), O.DP_NONE, 0.0, y1)
        torch.cuda.synchronize()
        assert np.array_equal(y1.cpu().numpy().astype(np.float64), Y_ref[3])
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("R,K,N", [(80, 200, 1), (80, 200, 256), (80, 72, 300), (40, 136, 600), (30, 264, 700), (3, 520, 1100),
                                   (76, 264, 100), (150, 520, 300), (75, 2048, 700)])
def test_spmm_both_kernels(S, R, K, N):
    """The launch chooses between a CTA per row tile (256 tokens) and a CTA pair per row tile (512 tokens) by the
    rounds of CTAs each needs: many row tiles with few tokens take the first, the rest the second.  These shapes
    reach both, with one and with several token blocks, ragged in M, K and N.  The last three leave a last round of
    two CTA pairs on a 148-SM GPU: those tiles are cut along K and their slices added by a second kernel."""
    rw, rx = WL._rngs(100 + R)
    M = 256 * R - 37
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), 0.5).astype(np.float16)
    X = rx.standard_normal((N, K), dtype=np.float32).astype(np.float16)
    Y_ref, S_ref = O.spmm_ref(W, X)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        y = run(S, h, X, M)
        check(y, Y_ref, S_ref)
        check(run(S, h, X, M, torch.float16), Y_ref, S_ref)
        assert np.array_equal(y, run(S, h, X, M))                       # the same bits from call to call
    finally:
        S.spdp_free(h)


def test_spmm_rejects_bad_arguments(S):
    h = S.spdp_pack_tiled_cbc(torch.zeros((256, 32), dtype=torch.float16, device="cuda"))
    try:
        X = torch.zeros((4, 40), dtype=torch.float16, device="cuda")
        Y = torch.zeros((4, 256), dtype=torch.float32, device="cuda")
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmm(h, X[:, 1:33], Y)                                  # X not 16-byte aligned
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmm(h, X[:, :32], Y[:, :100].contiguous())             # fewer than M outputs per token
        Xo = torch.zeros((4, 35), dtype=torch.float16, device="cuda")
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmm(h, Xo[:, :32], Y)                                  # row stride not a multiple of 8 elements
    finally:
        S.spdp_free(h)
