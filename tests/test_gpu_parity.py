"""Parity of the CUDA library (through the C ABI) with the CPU oracle on the same seeded inputs.

Bars: packed arrays and the active-column set bit-exact; every output within
|y - y_ref| <= 1e-3 * sum_j |W_ij x_j| + 1e-5 (y widened to fp64, no re-rounding); exact
equality where every partial sum is exactly representable.
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


def dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    return torch.from_numpy(a).cuda()


def assert_same_packed(got, want):
    for key in ("tileoffset", "colinfo", "bitmap", "values"):
        assert got[key].dtype == want[key].dtype, key
        assert got[key].shape == want[key].shape, key
        assert np.array_equal(got[key], want[key]), key
    assert got["nnz"] == want["nnz"]


def gpu_spmspv(S, h, x, rule, thr, M, ydtype=torch.float32, mask_words=None):
    xd = dev(x)
    y = torch.full((M,), float("nan"), dtype=ydtype, device="cuda")        # poison: every entry must be written
    md = dev(mask_words) if mask_words is not None else None
    S.spdp_spmspv(h, xd, rule, thr, y, mask=md)
    torch.cuda.synchronize()
    assert S.spdp_last_device_status(h) == 0
    return y.cpu().numpy().astype(np.float64)


def gpu_active(S, h, x, rule, thr, K, mask_words=None):
    bits = torch.full(((K + 31) // 32,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    S.spdp_active_columns(h, dev(x), rule, thr, bits, cnt, mask=dev(mask_words) if mask_words is not None else None)
    torch.cuda.synchronize()
    return bits.cpu().numpy().view(np.uint32), int(cnt.item())


def check_y(y, y_ref, S_ref):
    err = np.abs(y - y_ref)
    tol = O.tolerance(S_ref)
    bad = np.flatnonzero(~(err <= tol))
    assert bad.size == 0, f"{bad.size} outputs out of tolerance, worst ratio {np.nanmax(err / tol):.3g} at {bad[:5]}"
    return float(np.max(err / tol))


# ------------------------------------------------------------------------------------------
# packer / unpacker: bit-exact
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,K,seed", [(256, 16, 1), (512, 48, 2), (1, 1, 3), (257, 17, 4), (300, 40, 5),
                                      (1000, 200, 6), (2048, 272, 7)])
def test_pack_bit_exact_and_unpack(S, M, K, seed):
    W = WL.special_values_matrix(M, K, seed)
    want = O.pack_fast(W)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        got = S.spdp_export(h)
        assert_same_packed(got, want)
        info = S.spdp_get_info(h)
        assert (info.M, info.K, info.nnz, info.values_len) == (M, K, want["nnz"], len(want["values"]))
        assert info.packed_bytes == O.packed_bytes(want)
        out = torch.full((M, K + 3), -1.0, dtype=torch.float16, device="cuda")[:, :K]   # ldw != K
        S.spdp_unpack(h, out)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().view(np.uint16), O.canon(W))
    finally:
        S.spdp_free(h)


def test_pack_strided_input_and_storage_formula(S):
    M, K = 512, 96
    W = WL.special_values_matrix(M, K, 9)
    big = torch.zeros((M, K + 24), dtype=torch.float16, device="cuda")
    big[:, :K] = dev(W)
    h8 = S.spdp_pack_tiled_cbc(big[:, :K])
    h1 = S.spdp_pack_tiled_cbc(big[:, :K], pad_elems=1)
    try:
        assert_same_packed(S.spdp_export(h8), O.pack_fast(W))
        got1 = S.spdp_export(h1)
        assert_same_packed(got1, O.pack_fast(W, pad_elems=1))
        nnz = int(np.count_nonzero(W.view(np.uint16) & 0x7FFF))
        # Sec. 4.1 storage formula, exact when nothing is padded
        assert S.spdp_get_info(h1).packed_bytes == O.storage_formula_bytes(M, K, nnz)
        with pytest.raises(S.SpdpError, match="UNSUPPORTED_SHAPE"):
            S.spdp_spmspv(h1, torch.zeros(K, dtype=torch.float16, device="cuda"), 0, 0.0,
                          torch.zeros(M, dtype=torch.float32, device="cuda"))
    finally:
        S.spdp_free(h8)
        S.spdp_free(h1)


def test_pack_empty_and_full(S):
    for fill in (0.0, 1.0):
        W = np.full((512, 32), fill, np.float16)
        h = S.spdp_pack_tiled_cbc(dev(W))
        try:
            assert_same_packed(S.spdp_export(h), O.pack_ref(W))
        finally:
            S.spdp_free(h)


# ------------------------------------------------------------------------------------------
# active-column set: bit-exact
# ------------------------------------------------------------------------------------------
def test_active_set_bit_exact(S):
    K = 1000
    rng = np.random.Generator(np.random.PCG64(11))
    x = rng.standard_normal(K, dtype=np.float32).astype(np.float16)
    thr = float(np.float16(0.5))
    up, dn = np.nextafter(np.float16(0.5), np.float16(9)), np.nextafter(np.float16(0.5), np.float16(0))
    x[:14] = np.asarray([0.0, -0.0, 0.5, -0.5, up, -up, dn, -dn, np.nan, np.inf, -np.inf, 6e-8, -6e-8, 65504], np.float16)
    h = S.spdp_pack_tiled_cbc(dev(np.ones((256, K), np.float16)))
    try:
        for rule, t in ((O.DP_ABS_GT, thr), (O.DP_ABS_GT, 0.0), (O.DP_ABS_GT, -1.0), (O.DP_NONE, 0.0),
                        (O.DP_ABS_GT, 1e30), (O.DP_ABS_GT, float("inf"))):
            want = O.active_ref(x, rule, t)
            bits, cnt = gpu_active(S, h, x, rule, t, K)
            assert np.array_equal(bits, O.active_to_words(want)) and cnt == int(want.sum())
        m = rng.random(K) < 0.3
        bits, cnt = gpu_active(S, h, x, O.DP_MASK, 0.0, K, O.active_to_words(m))
        assert np.array_equal(bits, O.active_to_words(m)) and cnt == int(m.sum())
    finally:
        S.spdp_free(h)


# ------------------------------------------------------------------------------------------
# spMspV against the oracle
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,K,sp,skip,seed", [
    (256, 16, 0.5, 0.5, 1), (512, 64, 0.5, 0.0, 2), (300, 40, 0.3, 0.25, 3), (1, 1, 0.0, 0.0, 4),
    (257, 17, 0.5, 0.5, 5), (1024, 1024, 0.5, 0.5, 6), (768, 4400, 0.7, 0.9, 7), (2304, 528, 0.9, 0.4, 8),
    (4096, 272, 0.0, 0.1, 9), (256, 8192, 0.6, 0.5, 10),
    # rows longer than one batch of the kernel (pieces carry their sums over) and ragged long rows
    (512, 20000, 0.5, 0.3, 11), (300, 16400, 0.9, 0.0, 12), (1000, 8200, 0.2, 0.6, 13)])
@pytest.mark.parametrize("ydtype", ["f32", "f16"])
def test_spmspv_matches_oracle(S, M, K, sp, skip, seed, ydtype):
    rw, rx = WL._rngs(seed)
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), sp).astype(np.float16)
    x = rx.standard_normal(K, dtype=np.float32).astype(np.float16)
    rule, thr = WL.skip_threshold(x, skip)
    a = O.active_ref(x, rule, thr)
    y_ref, S_ref = O.spmspv_ref(W, x, a)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        bits, cnt = gpu_active(S, h, x, rule, thr, K)
        assert np.array_equal(bits, O.active_to_words(a)) and cnt == int(a.sum())
        yd = torch.float32 if ydtype == "f32" else torch.float16
        y = gpu_spmspv(S, h, x, rule, thr, M, yd)
        check_y(y, y_ref, S_ref)
        y2 = gpu_spmspv(S, h, x, rule, thr, M, yd)
        assert np.array_equal(y, y2)                                   # fixed summation order
        for ctas in (1, 3, 37, 1000):                                  # other split-K layouts
            S.spdp_set_num_ctas(h, ctas)
            check_y(gpu_spmspv(S, h, x, rule, thr, M, yd), y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_spmspv_exact_on_integers_and_powers_of_two(S):
    """Every product and partial sum is exactly representable: the GPU must match exactly."""
    rng = np.random.Generator(np.random.PCG64(21))
    M, K = 700, 900
    W = rng.integers(-8, 9, (M, K)).astype(np.float16)
    W[rng.random((M, K)) < 0.6] = 0
    x = rng.integers(-4, 5, K).astype(np.float16)
    a = O.active_ref(x, O.DP_ABS_GT, 1.0)
    y_ref, _ = O.spmspv_ref(W, x, a)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        assert np.array_equal(gpu_spmspv(S, h, x, O.DP_ABS_GT, 1.0, M), y_ref)
        Wp = (2.0 ** rng.integers(-6, 3, (M, K))).astype(np.float16) * rng.choice([-1, 1], (M, K)).astype(np.float16)
        Wp[rng.random((M, K)) < 0.5] = 0
        xp = (2.0 ** rng.integers(-3, 3, K)).astype(np.float16)
        hp = S.spdp_pack_tiled_cbc(dev(Wp))
        try:
            yp_ref, _ = O.spmspv_ref(Wp, xp, np.ones(K, bool))
            assert np.array_equal(gpu_spmspv(S, hp, xp, O.DP_NONE, 0.0, M), yp_ref)
        finally:
            S.spdp_free(hp)
    finally:
        S.spdp_free(h)


def test_spmspv_degenerate_cases(S):
    M, K = 600, 100
    rng = np.random.Generator(np.random.PCG64(23))
    W = (rng.standard_normal((M, K), dtype=np.float32) * 0.02).astype(np.float16)
    W[:, 10:20] = 0                                  # empty columns
    W[256:512, :] = 0                                # an empty row tile
    x = rng.standard_normal(K, dtype=np.float32).astype(np.float16)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        # nothing active: y is written as zeros
        y = gpu_spmspv(S, h, x, O.DP_ABS_GT, 1e9, M)
        assert not y.any()
        y = gpu_spmspv(S, h, x, O.DP_MASK, 0.0, M, mask_words=np.zeros(4, np.uint32))
        assert not y.any()
        # a single active column; explicit mask rule
        m = np.zeros(K, bool)
        m[37] = True
        y = gpu_spmspv(S, h, x, O.DP_MASK, 0.0, M, mask_words=O.active_to_words(m))
        y_ref, S_ref = O.spmspv_ref(W, x, m)
        check_y(y, y_ref, S_ref)
        # NaN activation is active and propagates; Inf weight in a skipped column does not
        W2 = W.copy()
        W2[5, 50] = np.inf
        x2 = x.copy()
        x2[50] = 0.0
        x2[60] = np.nan
        h2 = S.spdp_pack_tiled_cbc(dev(W2))
        try:
            y = gpu_spmspv(S, h2, x2, O.DP_ABS_GT, 0.0, M)
            nz60 = O.is_nonzero(W2[:, 60])
            assert np.all(np.isnan(y[nz60])) and not np.isnan(y[~nz60]).any()
        finally:
            S.spdp_free(h2)
    finally:
        S.spdp_free(h)


def test_unaligned_x_and_mask_rule_on_a_long_row(S):
    """x that is only 2-byte aligned takes the kernel's plain-load path; the explicit mask rule on two batches."""
    w = WL.config2(768, 9000, seed=8)
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    h = S.spdp_pack_tiled_cbc(dev(w.W))
    try:
        buf = torch.zeros(w.K + 8, dtype=torch.float16, device="cuda")
        for shift in (1, 3, 8):
            xs = buf[shift: shift + w.K]
            xs.copy_(dev(w.x))
            assert xs.data_ptr() % 16 == (2 * shift) % 16
            y = torch.full((w.M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, xs, w.rule, w.thr, y)
            torch.cuda.synchronize()
            check_y(y.cpu().numpy().astype(np.float64), y_ref, S_ref)
        y = gpu_spmspv(S, h, w.x, O.DP_MASK, 0.0, w.M, mask_words=O.active_to_words(a))
        check_y(y, y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_spmspv_in_a_cuda_graph(S):
    """spdp_spmspv only launches (no allocation, no synchronisation): it can be captured and replayed."""
    w = WL.config1(1024, 2048, seed=9)
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    h = S.spdp_pack_tiled_cbc(dev(w.W))
    try:
        x = dev(w.x)
        y = torch.zeros(w.M, dtype=torch.float32, device="cuda")
        S.spdp_spmspv(h, x, w.rule, w.thr, y)                      # warm-up outside the capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                S.spdp_spmspv(h, x, w.rule, w.thr, y, stream=side)
        for _ in range(3):
            y.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            check_y(y.cpu().numpy().astype(np.float64), y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_imported_oracle_arrays_give_same_result(S):
    w = WL.config1(768, 640, seed=4)
    p = O.pack_fast(w.W)
    h_imp = S.spdp_import_tiled_cbc(w.M, w.K, p["tileoffset"], p["colinfo"], p["bitmap"], p["values"])
    h_gpu = S.spdp_pack_tiled_cbc(dev(w.W))
    try:
        assert_same_packed(S.spdp_export(h_imp), p)
        y1 = gpu_spmspv(S, h_imp, w.x, w.rule, w.thr, w.M)
        y2 = gpu_spmspv(S, h_gpu, w.x, w.rule, w.thr, w.M)
        assert np.array_equal(y1, y2)
        bad = p["colinfo"].copy()
        bad[3] += 1
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_import_tiled_cbc(w.M, w.K, p["tileoffset"], bad, p["bitmap"], p["values"])
    finally:
        S.spdp_free(h_imp)
        S.spdp_free(h_gpu)


def test_host_vector_entry_point(S):
    w = WL.config2(1024, 512, seed=6)
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    h = S.spdp_pack_tiled_cbc(dev(w.W))
    try:
        xh = torch.from_numpy(w.x.copy()).pin_memory()
        for dt in (torch.float16, torch.float32):
            yh = torch.full((w.M,), float("nan"), dtype=dt).pin_memory()
            S.spdp_spmspv_host(h, xh, w.rule, w.thr, yh)
            check_y(yh.numpy().astype(np.float64), y_ref, S_ref)
        yn = np.full(w.M, np.nan, np.float32)
        S.spdp_spmspv_host(h, w.x, O.DP_MASK, 0.0, yn, mask_host=O.active_to_words(a))
        check_y(yn.astype(np.float64), y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_host_vector_entry_point_repeated_calls(S):
    """The same pinned buffers call after call (the library may replay a recorded graph): new contents
    of x must give new results, and a different CTA count, other buffers or pageable memory still work."""
    rng = np.random.Generator(np.random.PCG64(91))
    M, K = 1300, 2100
    W = (rng.standard_normal((M, K)) * (rng.random((M, K)) < 0.5) * 0.05).astype(np.float16)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        xh = torch.zeros(K, dtype=torch.float16).pin_memory()
        yh = torch.zeros(M, dtype=torch.float32).pin_memory()
        for step in range(6):
            x = rng.standard_normal(K).astype(np.float16)
            xh.copy_(torch.from_numpy(x))
            yh.fill_(float("nan"))
            if step == 4:
                S.spdp_set_num_ctas(h, 37)
            S.spdp_spmspv_host(h, xh, O.DP_ABS_GT, 0.4, yh)
            a = O.active_ref(x, O.DP_ABS_GT, 0.4)
            y_ref, S_ref = O.spmspv_ref(W, x, a)
            check_y(yh.numpy().astype(np.float64), y_ref, S_ref)
        y2 = torch.zeros(M, dtype=torch.float16).pin_memory()          # another output buffer and dtype
        S.spdp_spmspv_host(h, xh, O.DP_ABS_GT, 0.4, y2)
        check_y(y2.numpy().astype(np.float64), y_ref, S_ref)
        yn = np.full(M, np.nan, np.float32)                            # pageable memory
        for _ in range(3):
            S.spdp_spmspv_host(h, x, O.DP_ABS_GT, 0.4, yn)
            check_y(yn.astype(np.float64), y_ref, S_ref)
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("make", [lambda: WL.config1(1024, 1024), lambda: WL.config2(1536, 1024),
                                  lambda: WL.config3(1024, 2752), lambda: WL.config4(3584, 1024),
                                  lambda: WL.config5(0, 0, 1024, 1024), lambda: WL.config5(3, 3, 1024, 1024)])
def test_scaled_down_benchmark_layers(S, make):
    w = make()
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    h = S.spdp_pack_tiled_cbc(dev(w.W))
    try:
        assert_same_packed(S.spdp_export(h), O.pack_fast(w.W))
        bits, _ = gpu_active(S, h, w.x, w.rule, w.thr, w.K)
        assert np.array_equal(bits, O.active_to_words(a))
        check_y(gpu_spmspv(S, h, w.x, w.rule, w.thr, w.M, torch.float16), y_ref, S_ref)
        check_y(gpu_spmspv(S, h, w.x, w.rule, w.thr, w.M, torch.float32), y_ref, S_ref)
    finally:
        S.spdp_free(h)


# ------------------------------------------------------------------------------------------
# the single-vector kernel's own DP test (it lists the active columns itself, 8 per thread)
# ------------------------------------------------------------------------------------------
def _striped_identity(M, K):
    """One stored 1.0 per column, at row j % M: y then shows every column's decision by itself."""
    W = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    j = torch.arange(K, device="cuda")
    W[j % M, j] = 1.0
    return W


@pytest.mark.parametrize("thr", [0.5, 0.50006103515625, 0.3, 0.0, -0.0, -1.0, 1e-10, 70000.0, float("inf"),
                                 float("-inf"), float("nan"), 6.1e-5, 5.96e-8])
def test_spmspv_active_set_on_threshold_edges(S, thr):
    """Values at, just below and just above the threshold (in fp16 steps), zeros of both signs, subnormals,
    the largest finite values, NaN and both infinities, under finite, infinite and NaN thresholds: the
    kernel's in-line DP test must take the oracle's decision for every one.  Also with x only 2-byte
    aligned (the plain-load path) and with the probes astride column 8192, where a CTA that owns a long
    stretch of one row tile ends one list of columns and begins the next."""
    base = np.float16(thr) if np.isfinite(thr) and abs(thr) < 65504 else np.float16(1.0)
    around = np.array([base, np.nextafter(base, np.float16(np.inf)), np.nextafter(base, np.float16(-np.inf)),
                       -base, 0.0, -0.0, 6e-8, -6e-8, 6.1e-5, 65504, -65504, 0.25, 0.5, 0.75,
                       np.nan, np.inf, -np.inf], dtype=np.float16)
    rng = np.random.Generator(np.random.PCG64(78))
    for K, ctas, shift in ((64, 0, 0), (16400, 1, 0), (16400, 3, 1), (16400, 0, 3)):
        M = min(K, 256)
        first = 0 if K == 64 else 8192 - 7                     # probes astride the end of the first list
        x = np.zeros(K, dtype=np.float16)
        x[first:first + len(around)] = rng.permutation(around)
        a = O.active_ref(x, O.DP_ABS_GT, thr)
        want = np.zeros(M, dtype=np.float32)
        for p in range(first, first + len(around)):
            if a[p]:
                want[p % M] = np.float32(x[p])
        h = S.spdp_pack_tiled_cbc(_striped_identity(M, K))
        try:
            if ctas:
                S.spdp_set_num_ctas(h, ctas)
            buf = torch.zeros(K + 8, dtype=torch.float16, device="cuda")
            xs = buf[shift:shift + K]
            xs.copy_(dev(x))
            y = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, xs, O.DP_ABS_GT, thr, y)
            torch.cuda.synchronize()
            assert np.array_equal(y.cpu().numpy(), want, equal_nan=True), (thr, K, ctas, shift)
            bits, cnt = gpu_active(S, h, x, O.DP_ABS_GT, thr, K)
            assert np.array_equal(bits, O.active_to_words(a)) and cnt == int(a.sum())
        finally:
            S.spdp_free(h)


def test_mask_rule_with_the_mask_at_the_end_of_its_allocation(S):
    """Explicit mask whose last word is the last word of its buffer, on shapes where a CTA's range starts at
    an odd GTile column (the list then has padding units between its two pieces, which must not read the
    mask), and a first call issued on a side stream right after packing."""
    for M, K, ctas in ((512, 4096, 3), (768, 4128, 7), (1024, 2080, 5)):
        rw, rx = WL._rngs(40 + ctas)
        W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), 0.5).astype(np.float16)
        x = rx.standard_normal(K, dtype=np.float32).astype(np.float16)
        m = rx.random(K) < 0.5
        y_ref, S_ref = O.spmspv_ref(W, x, m)
        words = O.active_to_words(m)
        arena = torch.zeros(4096 + len(words), dtype=torch.int32, device="cuda")
        md = arena[4096:]
        md.copy_(dev(words))
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            h = S.spdp_pack_tiled_cbc(dev(W), stream=side)
            try:
                S.spdp_set_num_ctas(h, ctas)
                y = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
                S.spdp_spmspv(h, dev(x), O.DP_MASK, 0.0, y, mask=md, stream=side)
                side.synchronize()
                check_y(y.cpu().numpy().astype(np.float64), y_ref, S_ref)
            finally:
                S.spdp_free(h)


def test_row_sharded_handles_reproduce_the_product(S):
    """Row-tile sharding on one GPU: every rank's slice packed as its own matrix, the slices of y side by
    side against the oracle (the collective that joins them is exercised by the two-rank CPU test)."""
    w = WL.config4(2304, 1040, seed=12)
    a = O.active_ref(w.x, w.rule, w.thr)
    y_ref, S_ref = O.spmspv_ref(w.W, w.x, a)
    x = dev(w.x)
    for world in (2, 3, 16):
        y = torch.full((w.M,), float("nan"), dtype=torch.float32, device="cuda")
        for rank in range(world):
            first, rows = S.spdp_row_shard(w.M, world, rank)
            if rows == 0:
                continue
            h = S.spdp_pack_tiled_cbc(dev(w.W[first:first + rows]))
            try:
                S.spdp_spmspv(h, x, w.rule, w.thr, y[first:first + rows])
            finally:
                torch.cuda.synchronize()
                S.spdp_free(h)
        check_y(y.cpu().numpy().astype(np.float64), y_ref, S_ref)


def test_producer_fused_activation_and_mask(S):
    """x = silu(gate) * up with the keep-mask written in the same pass: x within one fp16 step of the fp64
    definition, the mask exactly the set the magnitude rule chooses on the stored x, and the decode call
    with that mask bit-identical to the decode call that tests x itself."""
    rng = np.random.Generator(np.random.PCG64(83))
    M, K = 1536, 3000
    gate = rng.standard_normal(K).astype(np.float16) * np.float16(2.0)
    up = rng.standard_normal(K).astype(np.float16)
    gate[:4] = np.asarray([0.0, -0.0, 30.0, -30.0], np.float16)
    W = (rng.standard_normal((M, K)) * (rng.random((M, K)) < 0.5) * 0.05).astype(np.float16)
    thr = 0.3
    x_out = torch.full((K,), float("nan"), dtype=torch.float16, device="cuda")
    mask = torch.full(((K + 31) // 32,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    S.spdp_swiglu_dp(dev(gate), dev(up), thr, x_out, mask, cnt)
    torch.cuda.synchronize()
    xg = x_out.cpu().numpy()
    ref = O.swiglu_ref(gate, up)
    step = np.maximum(np.abs(ref), 2.0 ** -14) * 2.0 ** -10                  # one fp16 step at that magnitude
    assert np.all(np.abs(xg.astype(np.float64) - ref) <= step)
    a = O.active_ref(xg, O.DP_ABS_GT, thr)                                   # decided on the kernel's own fp16 x
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), O.active_to_words(a)) and int(cnt.item()) == int(a.sum())
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        y_mask = torch.empty(M, dtype=torch.float32, device="cuda")
        y_test = torch.empty(M, dtype=torch.float32, device="cuda")
        S.spdp_spmspv(h, x_out, O.DP_MASK, 0.0, y_mask, mask=mask)
        S.spdp_spmspv(h, x_out, O.DP_ABS_GT, thr, y_test)
        torch.cuda.synchronize()
        assert np.array_equal(y_mask.cpu().numpy(), y_test.cpu().numpy())
        y_ref, S_ref = O.spmspv_ref(W, xg, a)
        check_y(y_mask.cpu().numpy().astype(np.float64), y_ref, S_ref)
    finally:
        S.spdp_free(h)
