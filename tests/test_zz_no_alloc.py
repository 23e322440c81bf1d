"""The allocation-free entry point (spdp_spmspv_noalloc) against the handle-based one.

Collected last on purpose: the entry point keeps its scratch in one fixed device array that
every call shares, so it runs after everything else and must also pass alone in a fresh process.
It serves callers that may not allocate device memory through the library (a process whose
device memory is owned by its own arena, or one that forbids driver allocations after start-up);
they pass the packed arrays themselves.  Here the arrays simply come from a packed handle.
"""
import numpy as np
import pytest

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


@pytest.mark.parametrize("make", [lambda: WL.config1(1024, 1024, seed=3), lambda: WL.config4(3584, 1040, seed=5),
                                  lambda: WL.config3(300, 4400, seed=7)])
def test_noalloc_matches_handle_entry_point_twice(S, make):
    w = make()
    h = S.spdp_pack_tiled_cbc(torch.from_numpy(w.W).cuda())
    try:
        info = S.spdp_get_info(h)
        x = torch.from_numpy(w.x).cuda()
        arrays = (info.tileoffset_dev, info.colinfo_dev, info.bitmap_dev, info.values_dev)
        for dt in (torch.float32, torch.float16):
            want = torch.full((w.M,), float("nan"), dtype=dt, device="cuda")
            S.spdp_spmspv(h, x, w.rule, w.thr, want)
            torch.cuda.synchronize()
            want64 = want.cpu().numpy().astype(np.float64)
            # the error scale of the parity gate, rebuilt from the handle path's own |W||x| product
            scale = torch.full((w.M,), float("nan"), dtype=torch.float32, device="cuda")
            habs = S.spdp_pack_tiled_cbc(torch.from_numpy(np.abs(w.W)).cuda())
            try:
                S.spdp_spmspv(habs, torch.from_numpy(np.abs(w.x)).cuda(), w.rule, w.thr, scale)
                torch.cuda.synchronize()
            finally:
                S.spdp_free(habs)
            tol = 1e-3 * scale.cpu().numpy().astype(np.float64) + 1e-5
            for call in range(2):                      # two calls in a row share the scratch array
                got = torch.full((w.M,), float("nan"), dtype=dt, device="cuda")
                S.spdp_spmspv_noalloc(*arrays, w.M, w.K, x, w.rule, w.thr, got)
                torch.cuda.synchronize()
                err = np.abs(got.cpu().numpy().astype(np.float64) - want64)
                assert np.all(err <= tol), f"call {call}: worst error/tolerance {np.nanmax(err / tol):.3g}"
    finally:
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
