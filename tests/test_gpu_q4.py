"""The 4-bit Values variant on the GPU (Sec. 5.1 / Sec. 6): packed arrays bit-exact against the oracle's
quantiser and layout, y within the parity bound of the product on the DEQUANTISED weights."""
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
    a = np.ascontiguousarray(a)
    return torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a).cuda()


def assert_same_q4(got, want):
    for key in ("tileoffset", "colinfo", "bitmap", "codes", "scales"):
        assert got[key].dtype == want[key].dtype and got[key].shape == want[key].shape, key
        assert np.array_equal(got[key], want[key]), key
    assert got["nnz"] == want["nnz"] and got["pad_elems"] == 32


@pytest.mark.parametrize("M,K,sp,skip,seed", [(256, 16, 0.5, 0.5, 1), (300, 40, 0.3, 0.25, 2), (1, 1, 0.0, 0.0, 3),
                                              (257, 17, 0.5, 0.5, 4), (1024, 1024, 0.5, 0.5, 5), (768, 4400, 0.7, 0.9, 6),
                                              (2304, 528, 0.9, 0.4, 7), (512, 20000, 0.5, 0.3, 8), (4096, 272, 0.0, 0.1, 9)])
def test_q4_pack_bit_exact_and_product_on_dequantised_weights(S, M, K, sp, skip, seed):
    rw, rx = WL._rngs(seed)
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), sp).astype(np.float16)
    x = rx.standard_normal(K, dtype=np.float32).astype(np.float16)
    rule, thr = WL.skip_threshold(x, skip)
    a = O.active_ref(x, rule, thr)
    want = O.pack_q4_fast(W)
    h = S.spdp_pack_tiled_cbc_q4(dev(W))
    try:
        assert_same_q4(S.spdp_export_q4(h), want)
        info = S.spdp_get_info(h)
        assert info.values_len == int(want["tileoffset"][-1]) and info.pad_elems == 32
        small = M * K <= 1 << 21
        Wd = O.dequant_q4_ref(want) if small else None
        if small:
            y_ref, S_ref = O.spmspv_dense64_ref(Wd, x, a)
        for ctas in (0, 3, 37):
            S.spdp_set_num_ctas(h, ctas)
            for dt in (torch.float32, torch.float16):
                y = torch.full((M,), float("nan"), dtype=dt, device="cuda")
                S.spdp_spmspv(h, dev(x), rule, thr, y)
                torch.cuda.synchronize()
                assert S.spdp_last_device_status(h) == 0
                if small:
                    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
                    assert np.all(err <= O.tolerance(S_ref)), f"worst {np.nanmax(err / O.tolerance(S_ref)):.3g}"
            y2 = torch.full((M,), float("nan"), dtype=torch.float16, device="cuda")
            S.spdp_spmspv(h, dev(x), rule, thr, y2)
            torch.cuda.synchronize()
            assert np.array_equal(y.cpu().numpy(), y2.cpu().numpy())      # fixed summation order
        if small:
            ym = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, dev(x), O.DP_MASK, 0.0, ym, mask=dev(O.active_to_words(a)))
            torch.cuda.synchronize()
            assert np.all(np.abs(ym.cpu().numpy().astype(np.float64) - y_ref) <= O.tolerance(S_ref))
    finally:
        S.spdp_free(h)


def test_q4_large_matrix_rows_sampled_against_the_oracle(S):
    """A layer-shaped case: packed arrays bit-exact, y checked on the rows of a few row tiles."""
    w = WL.config4(3584, 2048, seed=5)
    a = O.active_ref(w.x, w.rule, w.thr)
    want = O.pack_q4_fast(w.W)
    h = S.spdp_pack_tiled_cbc_q4(dev(w.W))
    try:
        assert_same_q4(S.spdp_export_q4(h), want)
        y = torch.full((w.M,), float("nan"), dtype=torch.float32, device="cuda")
        S.spdp_spmspv(h, dev(w.x), w.rule, w.thr, y)
        torch.cuda.synchronize()
        yh = y.cpu().numpy().astype(np.float64)
        for r in (0, 5, 13):
            sub = O.pack_q4_fast(w.W[256 * r:256 * (r + 1)])
            y_ref, S_ref = O.spmspv_dense64_ref(O.dequant_q4_ref(sub), w.x, a)
            assert np.all(np.abs(yh[256 * r:256 * (r + 1)] - y_ref) <= O.tolerance(S_ref))
    finally:
        S.spdp_free(h)


def test_q4_exact_when_weights_lie_on_the_grid_and_other_calls_are_refused(S):
    rng = np.random.Generator(np.random.PCG64(71))
    M, K = 600, 200
    W = (rng.integers(-7, 8, (M, K)) * 0.5).astype(np.float16)
    W[rng.random((M, K)) < 0.5] = 0
    W[0, :] = 3.5
    W[256, :] = 3.5
    W[512, :] = -3.5
    x = rng.integers(-4, 5, K).astype(np.float16)
    a = O.active_ref(x, O.DP_ABS_GT, 1.0)
    y_ref, _ = O.spmspv_ref(W, x, a)                     # the quantisation is lossless here: the fp16 definition applies
    h = S.spdp_pack_tiled_cbc_q4(dev(W))
    try:
        y = torch.empty(M, dtype=torch.float32, device="cuda")
        S.spdp_spmspv(h, dev(x), O.DP_ABS_GT, 1.0, y)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy().astype(np.float64), y_ref)
        yh = np.full(M, np.nan, np.float32)
        S.spdp_spmspv_host(h, x, O.DP_ABS_GT, 1.0, yh)
        assert np.array_equal(yh.astype(np.float64), y_ref)
        with pytest.raises(S.SpdpError, match="UNSUPPORTED_SHAPE"):
            S.spdp_export(h)
        with pytest.raises(S.SpdpError, match="UNSUPPORTED_SHAPE"):
            S.spdp_spmm(h, torch.zeros((2, K), dtype=torch.float16, device="cuda"), torch.zeros((2, M), device="cuda"))
        with pytest.raises(S.SpdpError, match="UNSUPPORTED_SHAPE"):
            S.spdp_unpack(h, torch.zeros((M, K), dtype=torch.float16, device="cuda"))
    finally:
        S.spdp_free(h)
