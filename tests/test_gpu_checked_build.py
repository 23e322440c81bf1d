"""The checked build of the library (libspdp_checked.so, -DSPDP_CHECKED) on the small and ragged parity
cases: every index the kernels derive from the packed arrays is range-checked on the device and a
violation would land in the handle's status word.  Expected here: results within the parity bound and
a status of 0.  (The firing path of the check itself is exercised on the host, on made-up indices, in
tests/test_hostdev_helpers.py; no test feeds bad data to a GPU.)"""
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
    from paper_2607_21985_b200 import build, spdp
    saved = (spdp.LIB_PATH, spdp._lib)
    spdp.LIB_PATH, spdp._lib = build.build_checked(), None
    spdp.lib()
    yield spdp
    spdp.LIB_PATH, spdp._lib = saved


def dev(a):
    a = np.ascontiguousarray(a)
    return torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a).cuda()


CASES = [(256, 16, 0.5, 0.5, 1), (300, 40, 0.3, 0.25, 3), (1, 1, 0.0, 0.0, 4), (257, 17, 0.5, 0.5, 5),
         (1024, 1024, 0.5, 0.5, 6), (768, 4400, 0.7, 0.9, 7), (2304, 528, 0.9, 0.4, 8), (512, 20000, 0.5, 0.3, 11),
         (1000, 8200, 0.2, 0.6, 13)]


@pytest.mark.parametrize("M,K,sp,skip,seed", CASES)
def test_checked_build_parity_and_clean_status(S, M, K, sp, skip, seed):
    rw, rx = WL._rngs(seed)
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), sp).astype(np.float16)
    X = rx.standard_normal((5, K), dtype=np.float32).astype(np.float16)
    rule, thr = WL.skip_threshold(X[0], skip)
    acts = np.stack([O.active_ref(X[b], rule, thr) for b in range(5)])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        for ctas in (0, 3, 37):
            S.spdp_set_num_ctas(h, ctas)
            y = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, dev(X[0]), rule, thr, y)
            Y = torch.full((5, M), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv_batch(h, dev(X), rule, thr, Y)
            ym = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, dev(X[0]), O.DP_MASK, 0.0, ym, mask=dev(O.active_to_words(acts[0])))
            torch.cuda.synchronize()
            assert S.spdp_last_device_status(h) == 0
            tol = O.tolerance(S_ref)
            assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - Y_ref[0]) <= tol[0])
            assert np.all(np.abs(ym.cpu().numpy().astype(np.float64) - Y_ref[0]) <= tol[0])
            assert np.all(np.abs(Y.cpu().numpy().astype(np.float64) - Y_ref) <= tol)
    finally:
        S.spdp_free(h)
