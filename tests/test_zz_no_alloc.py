"""The allocation-free entry point (spdp_spmspv_noalloc) against the oracle and the handle-based call.

Collected last on purpose: the entry point keeps its scratch in one fixed device array that
every call shares, so it runs after everything else and must also pass alone in a fresh process.
It serves callers that may not allocate device memory through the library (a process whose
device memory is owned by its own arena, or one that forbids driver allocations after start-up);
they pass the packed arrays themselves.  Here the arrays simply come from a packed handle.
"""
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


def _noalloc(S, h, w, dt):
    info = S.spdp_get_info(h)
    got = torch.full((w.M,), float("nan"), dtype=dt, device="cuda")
    S.spdp_spmspv_noalloc(info.tileoffset_dev, info.colinfo_dev, info.bitmap_dev, info.values_dev, w.M, w.K,
                          torch.from_numpy(w.x).cuda(), w.rule, w.thr, got)
    torch.cuda.synchronize()
    return got.cpu().numpy()


@pytest.mark.parametrize("make", [lambda: WL.config1(1024, 1024, seed=3), lambda: WL.config4(3584, 1040, seed=5),
                                  lambda: WL.config3(300, 4400, seed=7)])
def test_noalloc_matches_oracle_and_handle_entry_point_twice(S, make):
    w = make()
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    tol = O.tolerance(S_ref)                               # |y - y_ref| <= 1e-3 * S + 1e-5, S from the oracle
    h = S.spdp_pack_tiled_cbc(torch.from_numpy(w.W).cuda())
    try:
        x = torch.from_numpy(w.x).cuda()
        for dt in (torch.float32, torch.float16):
            want = torch.full((w.M,), float("nan"), dtype=dt, device="cuda")
            S.spdp_spmspv(h, x, w.rule, w.thr, want)      # the handle's default CTA count is the one noalloc uses
            torch.cuda.synchronize()
            want = want.cpu().numpy()
            for call in range(2):                          # two calls in a row share the scratch array
                got = _noalloc(S, h, w, dt)
                err = np.abs(got.astype(np.float64) - y_ref)
                assert np.all(err <= tol), f"call {call}: worst error/tolerance {np.nanmax(err / tol):.3g}"
                assert np.array_equal(got, want), f"call {call}: differs from spdp_spmspv at the same CTA count"
    finally:
        S.spdp_free(h)


def test_noalloc_after_a_call_of_another_shape(S):
    """A launch with many CTAs, then one with few, then many again: each call must empty the part of the
    shared array it uses, whatever the call before left there."""
    big = WL.config1(2048, 1024, seed=11)                   # 512 GTiles: one CTA per SM
    small = WL.config2(256, 160, seed=12)                   # 10 GTiles: 10 CTAs
    hs = {}
    try:
        for name, w in (("big", big), ("small", small)):
            hs[name] = S.spdp_pack_tiled_cbc(torch.from_numpy(w.W).cuda())
        for name, w in (("big", big), ("small", small), ("big", big), ("small", small)):
            a = O.active_ref(w.x, w.rule, w.thr)
            y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
            want = torch.full((w.M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(hs[name], torch.from_numpy(w.x).cuda(), w.rule, w.thr, want)
            got = _noalloc(S, hs[name], w, torch.float32)
            assert np.all(np.abs(got.astype(np.float64) - y_ref) <= O.tolerance(S_ref)), name
            assert np.array_equal(got, want.cpu().numpy()), name
    finally:
        for h in hs.values():
            S.spdp_free(h)


def test_noalloc_rejects_oversize_and_bad_arguments(S):
    x = torch.zeros(16, dtype=torch.float16, device="cuda")
    y = torch.zeros(16, dtype=torch.float32, device="cuda")
    buf = torch.zeros(64, dtype=torch.int64, device="cuda")
    with pytest.raises(S.SpdpError, match="UNSUPPORTED_SHAPE"):       # 2^26 column tiles: beyond the library's limit
        S.spdp_spmspv_noalloc(buf, buf, buf, buf, (1 << 22) * 256, 16, x, 0, 0.0, y)
    with pytest.raises(S.SpdpError, match="INVALID_ARG"):
        S.spdp_spmspv_noalloc(buf, buf, buf, buf, 16, 16, x, 2, 0.0, y)      # mask rule without a mask
    with pytest.raises(S.SpdpError, match="INVALID_ARG"):
        S.spdp_spmspv_noalloc(0, buf, buf, buf, 16, 16, x, 0, 0.0, y)        # null array
