"""The C oracle (full-size / timed CPU baseline) against the NumPy oracle and NumPy itself.

Nothing here calls the CUDA library.
"""
import numpy as np
import pytest

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL


def test_half_widening_all_bit_patterns(c_oracle):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([c_oracle.half_to_double(int(b)) for b in bits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


@pytest.mark.parametrize("M,K,pad,seed", [(256, 16, 8, 1), (300, 40, 8, 2), (512, 64, 1, 3), (1, 1, 8, 4),
                                          (1024, 48, 8, 5)])
def test_pack_unpack_match_numpy_oracle(c_oracle, M, K, pad, seed):
    W = WL.special_values_matrix(M, K, seed)
    p = O.pack_ref(W, pad_elems=pad)
    q = c_oracle.pack(W, pad_elems=pad)
    for key in ("tileoffset", "colinfo", "bitmap", "values"):
        assert p[key].dtype == q[key].dtype and np.array_equal(p[key], q[key]), key
    assert q["nnz"] == p["nnz"]
    assert np.array_equal(c_oracle.unpack(q), O.canon(W))


def test_active_and_spmspv_match_numpy_oracle(c_oracle):
    w = WL.config1(M=512, K=768, seed=5)
    x = w.x.copy()
    x[:6] = np.asarray([np.nan, np.inf, -0.0, w.thr, -w.thr, 0.0], np.float16)
    a_py = O.active_ref(x, w.rule, w.thr)
    a_c = c_oracle.active(x, w.rule, w.thr)
    assert np.array_equal(a_py, a_c)
    x = w.x
    a = O.active_ref(x, w.rule, w.thr)
    y_py, S_py = O.spmspv_ref(w.W, x, a)
    for threads in (1, 3):
        y_c, S_c, used = c_oracle.spmspv(w.W, x, a, threads=threads)
        assert used == threads
        # same products, different summation order: a few ulps of the running sums
        assert np.all(np.abs(y_c - y_py) <= 1e-13 * S_py + 1e-300)
        assert np.allclose(S_c, S_py, rtol=1e-13)
    m = O.active_to_words(a)
    assert np.array_equal(c_oracle.active(x, O.DP_MASK, 0.0, m), a)
    p = c_oracle.pack(w.W)
    assert c_oracle.active_bytes(p, a, 2) == O.active_bytes(p, a, 2)
    assert c_oracle.active_bytes(p, a, 4) == O.active_bytes(p, a, 4)


def test_mid_size_config_shapes(c_oracle):
    """A scaled-down copy of each benchmark layer: packers agree, realised sparsities are on target."""
    for w, sp, skip in ((WL.config1(512, 512), 0.5, 0.5), (WL.config2(768, 512), 0.6, 0.5),
                        (WL.config3(512, 1024), 0.7, 0.9), (WL.config4(1024, 512), 0.5, 0.4),
                        (WL.config5(3, 1, 512, 512), 0.9, 0.25)):
        assert abs(w.weight_sparsity - sp) < 0.02, w.name
        a = c_oracle.active(w.x, w.rule, w.thr)
        assert abs((~a).mean() - skip) < 0.01, w.name
        p, q = c_oracle.pack(w.W), O.pack_fast(w.W)
        for key in ("tileoffset", "colinfo", "bitmap", "values"):
            assert np.array_equal(p[key], q[key]), (w.name, key)
    # per-column sparsity of the 70B-shaped layer spreads over 0.3 .. 0.7
    w = WL.config4(2048, 512)
    col_sp = (w.W == 0).mean(axis=0)
    assert col_sp.min() < 0.36 and col_sp.max() > 0.64 and abs(col_sp.mean() - 0.5) < 0.02
