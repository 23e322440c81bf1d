"""Pins for the oracle's 4-bit Values variant (Sec. 5.1: 4-bit round-to-nearest; Sec. 6: low-bit Values
next to unchanged sparsity metadata).  Nothing here calls the CUDA library."""
import numpy as np

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL


def _f16(a):
    return np.asarray(a, dtype=np.float16)


def test_quantiser_on_a_hand_computed_column():
    # fp16(0.7) = 0.7001953125; / 7 = 0.100027901... -> nearest fp16 is 0x2E67 = 0.10003662109375
    # 0.7001953125 / s = 6.9994 -> 7;  fp16(-0.35) / s = -3.4997 -> -3;  fp16(0.1) / s = 0.9994 -> 1;
    # fp16(0.0499) / s = 0.4988 -> 0
    s16, codes = O.quantise_q4_ref(_f16([0.7, -0.35, 0.1, 0.0499]))
    assert int(s16) == 0x2E67
    assert codes.tolist() == [15, 5, 9, 8]
    # exactly representable: max 0.875 -> scale 0.125 (0x3000); -0.4375 / s = -3.5 -> -4 and 0.0625 / s = 0.5 -> 0 (ties to even)
    s16, codes = O.quantise_q4_ref(_f16([0.875, -0.4375, 0.125, 0.0625]))
    assert int(s16) == 0x3000 and codes.tolist() == [15, 4, 9, 8]
    # ties go to even: with scale 0.5, 0.25 -> 0.5 -> 0 and 0.75 -> 1.5 -> 2
    s16, codes = O.quantise_q4_ref(_f16([3.5, 0.25, 0.75, -1.25]))
    assert float(s16.view(np.float16)) == 0.5
    assert codes.tolist() == [15, 8, 10, 8 - 2]             # -1.25 / 0.5 = -2.5 -> -2
    # an all-tiny column whose scale underflows to zero keeps code 8 (weight 0)
    s16, codes = O.quantise_q4_ref(np.array([0x0001, 0x8001], np.uint16))
    assert int(s16) == 0 and codes.tolist() == [8, 8]


def test_values_on_the_grid_survive_exactly_and_others_within_half_a_step():
    rng = np.random.Generator(np.random.PCG64(3))
    M, K = 512, 48
    W = (rng.integers(-7, 8, (M, K)) * 0.5).astype(np.float16)          # multiples of 0.5 up to 3.5
    W[rng.random((M, K)) < 0.5] = 0
    W[0, :] = 3.5                                                       # every column tile of row tile 0 reaches the maximum
    W[256, :] = -3.5
    p = O.pack_q4_ref(W)
    assert np.array_equal(O.dequant_q4_ref(p), W.astype(np.float64))    # scale 0.5, every value on the grid
    w = WL.config1(512, 64, seed=2)
    p = O.pack_q4_fast(w.W)
    err = np.abs(O.dequant_q4_ref(p) - w.W.astype(np.float64))
    R, C, _ = O.grid(w.M, w.K)
    s = p["scales"].view(np.float16).astype(np.float64).reshape(R, C * 16)[:, :w.K]
    bound = np.repeat(s, 256, axis=0)[:w.M] * 0.5 * (1 + 2.0 ** -9)
    assert np.all(err <= bound + (w.W == 0) * 0)                        # round to nearest: at most half a step
    assert np.all(O.dequant_q4_ref(p)[w.W == 0] == 0)                   # pruned weights stay pruned


def test_q4_layout_invariants_and_fast_equals_reference():
    W = WL.special_values_matrix(600, 40, 4)
    Wb = W.view(np.uint16).copy()
    Wb[(Wb & 0x7C00) == 0x7C00] = 0x3C00                                # the variant is defined for finite weights
    W = Wb.view(np.float16)
    a, b = O.pack_q4_ref(W), O.pack_q4_fast(W)
    for k in ("tileoffset", "colinfo", "bitmap", "codes", "scales"):
        assert a[k].dtype == b[k].dtype and np.array_equal(a[k], b[k]), k
    base = O.pack_fast(W)
    assert np.array_equal(a["bitmap"], base["bitmap"])                  # the sparsity metadata does not change
    assert np.array_equal(a["colinfo"] & 0xFFFF, base["colinfo"] & 0xFFFF)
    assert np.all(a["tileoffset"] % 32 == 0) and np.all((a["colinfo"] >> 16) % 32 == 0)
    assert a["codes"].shape[0] * 2 == int(a["tileoffset"][-1])
    nib = np.stack([a["codes"] & 15, a["codes"] >> 4], axis=1).reshape(-1)
    n = (a["colinfo"] & 0xFFFF).astype(np.int64)
    start = np.repeat(a["tileoffset"][:-1].astype(np.int64), 16) + (a["colinfo"] >> 16)
    stored = np.zeros(nib.shape[0], bool)
    for s0, k in zip(start, n):
        stored[s0:s0 + k] = True
    assert np.all(nib[stored] >= 1) and np.all(nib[~stored] == 0)       # code 0 is padding only


def test_q4_byte_model_and_product_on_dequantised_weights():
    w = WL.config1(512, 96, seed=6)
    p = O.pack_q4_fast(w.W)
    a = O.active_ref(w.x, w.rule, w.thr)
    Wd = O.dequant_q4_ref(p)
    y, S = O.spmspv_dense64_ref(Wd, w.x, a)
    yb, Sb = np.zeros(w.M), np.zeros(w.M)
    xd = w.x.astype(np.float64)
    for j in np.flatnonzero(a):                                         # explicit loop over the active columns
        yb += Wd[:, j] * xd[j]
        Sb += np.abs(Wd[:, j] * xd[j])
    assert np.allclose(y, yb, rtol=1e-12, atol=1e-15) and np.allclose(S, Sb, rtol=1e-12, atol=1e-15)
    n = (p["colinfo"] & 0xFFFF).astype(np.int64).reshape(2, 96)
    tiles = int(((32 + (n + 31) // 32 * 16 + 6) * a[None, :]).sum())
    want = tiles + 4 * (2 * int(a.reshape(6, 16).any(axis=1).sum()) + 1) + 2 * 96 + 2 * 512
    assert O.active_bytes_q4(p, a) == want
