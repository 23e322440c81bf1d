"""Parity at the benchmark's full sizes, in the launch configuration the benchmark times
(default CTA count, fp16 y), against the C oracle: packed arrays and active set bit-exact, every
output inside the tolerance."""
import numpy as np
import pytest

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def S():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2607_21985_b200 import spdp
    spdp.lib()
    return spdp


CASES = {
    "c1": lambda: WL.config1(),
    "c2": lambda: WL.config2(),
    "c3": lambda: WL.config3(),
    "c4": lambda: WL.config4(),
    "c5_sp30_dp0": lambda: WL.config5(0, 0),
    "c5_sp50_dp50": lambda: WL.config5(1, 2),
    "c5_sp70_dp25": lambda: WL.config5(2, 1),
    "c5_sp90_dp75": lambda: WL.config5(3, 3),
}


@pytest.mark.parametrize("name", list(CASES))
def test_full_size_layer(S, c_oracle, name):
    w = CASES[name]()
    a = c_oracle.active(w.x, w.rule, w.thr)
    want = c_oracle.pack(w.W)
    y_ref, S_ref, _ = c_oracle.spmspv(w.W, w.x, a)
    Wd = torch.from_numpy(w.W).cuda()
    h = S.spdp_pack_tiled_cbc(Wd)
    del Wd
    try:
        got = S.spdp_export(h)
        for key in ("tileoffset", "colinfo", "bitmap", "values"):
            assert np.array_equal(got[key], want[key]), key
        xd = torch.from_numpy(w.x).cuda()
        bits = torch.zeros((w.K + 31) // 32, dtype=torch.int32, device="cuda")
        S.spdp_active_columns(h, xd, w.rule, w.thr, bits)
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), O.active_to_words(a))
        for dt in (torch.float16, torch.float32):
            y = torch.full((w.M,), float("nan"), dtype=dt, device="cuda")
            S.spdp_spmspv(h, xd, w.rule, w.thr, y)
            torch.cuda.synchronize()
            assert S.spdp_last_device_status(h) == 0
            err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
            tol = O.tolerance(S_ref)
            assert np.all(err <= tol), f"{name}: worst error/tolerance {np.nanmax(err / tol):.3g}"
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("name,B", [("c4", 8), ("c1", 5), ("c3", 8)])
def test_full_size_small_batch(S, c_oracle, name, B):
    """The small-batch entry point at full size, default CTA count, fp16 outputs: every token against
    the C oracle's single-vector result for that token."""
    w = CASES[name]()
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(500 + B)))
    X = np.concatenate([w.x[None, :], rng.standard_normal((B - 1, w.K), dtype=np.float32).astype(np.float16)])
    h = S.spdp_pack_tiled_cbc(torch.from_numpy(w.W).cuda())
    try:
        Y = torch.full((B, w.M), float("nan"), dtype=torch.float16, device="cuda")
        S.spdp_spmspv_batch(h, torch.from_numpy(X).cuda(), w.rule, w.thr, Y)
        torch.cuda.synchronize()
        out = Y.cpu().numpy().astype(np.float64)
        for b in range(B):
            a = c_oracle.active(X[b], w.rule, w.thr)
            y_ref, S_ref, _ = c_oracle.spmspv(w.W, X[b], a)
            err = np.abs(out[b] - y_ref)
            tol = O.tolerance(S_ref)
            assert np.all(err <= tol), f"{name} token {b}: worst error/tolerance {np.nanmax(err / tol):.3g}"
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("name,N", [("c1", 16), ("c1", 128), ("c1", 1024), ("c4_rows3584", 128), ("c4_rows3584", 1024)])
def test_full_size_prefill(S, c_oracle, name, N):
    """The prefill entry point on benchmark-shaped layers (c1 whole; c4's K = 8192 with 14 of its 112 row
    tiles, so that the fp64 oracle product stays within seconds): every token of a sample against the C
    oracle's single-vector result without DP, fp16 outputs as the benchmark uses them."""
    w = CASES["c1"]() if name == "c1" else WL.config4(M=3584)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(600 + N)))
    X = rng.standard_normal((N, w.K), dtype=np.float32).astype(np.float16)
    h = S.spdp_pack_tiled_cbc(torch.from_numpy(w.W).cuda())
    try:
        Y = torch.full((N, w.M), float("nan"), dtype=torch.float16, device="cuda")
        S.spdp_spmm(h, torch.from_numpy(X).cuda(), Y)
        torch.cuda.synchronize()
        assert S.spdp_last_device_status(h) == 0
        out = Y.cpu().numpy().astype(np.float64)
        assert not np.isnan(out).any()
        every = np.ones(w.K, dtype=bool)
        for n in sorted(set([0, 1, N // 3, N // 2, N - 2, N - 1]) & set(range(N))):
            y_ref, S_ref, _ = c_oracle.spmspv(w.W, X[n], every)
            err = np.abs(out[n] - y_ref)
            tol = O.tolerance(S_ref)
            assert np.all(err <= tol), f"{name} token {n}: worst error/tolerance {np.nanmax(err / tol):.3g}"
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("name", ["c1", "c3"])
def test_full_size_q4(S, name):
    """The 4-bit variant at full size, default CTA count, fp16 y: packed arrays bit for bit against the
    oracle's, y on the rows of three row tiles against the product on the dequantised weights."""
    w = CASES[name]()
    a = O.active_ref(w.x, w.rule, w.thr)
    want = O.pack_q4_fast(w.W)
    h = S.spdp_pack_tiled_cbc_q4(torch.from_numpy(w.W).cuda())
    try:
        got = S.spdp_export_q4(h)
        for key in ("tileoffset", "colinfo", "bitmap", "codes", "scales"):
            assert np.array_equal(got[key], want[key]), key
        y = torch.full((w.M,), float("nan"), dtype=torch.float16, device="cuda")
        S.spdp_spmspv(h, torch.from_numpy(w.x).cuda(), w.rule, w.thr, y)
        torch.cuda.synchronize()
        assert S.spdp_last_device_status(h) == 0
        out = y.cpu().numpy().astype(np.float64)
        R = w.M // 256
        for r in (0, R // 2, R - 1):
            sub = O.pack_q4_fast(w.W[256 * r:256 * (r + 1)])
            y_ref, S_ref = O.spmspv_dense64_ref(O.dequant_q4_ref(sub), w.x, a)
            assert np.all(np.abs(out[256 * r:256 * (r + 1)] - y_ref) <= O.tolerance(S_ref)), (name, r)
    finally:
        S.spdp_free(h)
