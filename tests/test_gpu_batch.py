"""Small-batch decode (spdp_spmspv_batch) against the oracle's token-by-token definition."""
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


def check(Y, Y_ref, S_ref):
    err = np.abs(Y.astype(np.float64) - Y_ref)
    tol = O.tolerance(S_ref)
    assert np.all(err <= tol), f"worst error/tolerance {np.max(err / tol):.3g}"


def run_batch(S, h, X, rule, thr, M, ydtype=torch.float32, mask=None):
    B = X.shape[0]
    Y = torch.full((B, M), float("nan"), dtype=ydtype, device="cuda")
    S.spdp_spmspv_batch(h, dev(X), rule, thr, Y, mask=None if mask is None else dev(mask))
    torch.cuda.synchronize()
    assert S.spdp_last_device_status(h) == 0
    return Y.float().cpu().numpy()


@pytest.mark.parametrize("M,K,sp,skip,seed", [
    (256, 16, 0.5, 0.5, 1), (300, 40, 0.3, 0.25, 2), (1, 1, 0.0, 0.0, 3), (257, 17, 0.5, 0.5, 4),
    (1024, 1024, 0.5, 0.4, 5), (768, 4400, 0.7, 0.9, 6), (2304, 528, 0.9, 0.4, 7), (256, 8192, 0.6, 0.5, 8),
    (512, 20000, 0.5, 0.3, 9), (1000, 8200, 0.2, 0.6, 10)])
@pytest.mark.parametrize("B", [1, 2, 3, 5, 8])
def test_batch_matches_oracle(S, M, K, sp, skip, seed, B):
    rw, rx = WL._rngs(seed)
    W = WL.prune_global_magnitude(WL.normal_weights(rw, M, K), sp).astype(np.float16)
    X = rx.standard_normal((B, K), dtype=np.float32).astype(np.float16)
    # one threshold for the whole batch (the library takes a scalar): the first token's quantile
    rule, thr = WL.skip_threshold(X[0], skip)
    acts = np.stack([O.active_ref(X[b], rule, thr) for b in range(B)])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        for ydtype in (torch.float32, torch.float16):
            Y = run_batch(S, h, X, rule, thr, M, ydtype)
            check(Y, Y_ref, S_ref)
        Y2 = run_batch(S, h, X, rule, thr, M, torch.float16)
        assert np.array_equal(Y, Y2)                                   # fixed summation order
        for ctas in (1, 3, 37, 1000):                                  # other split-K layouts
            S.spdp_set_num_ctas(h, ctas)
            check(run_batch(S, h, X, rule, thr, M), Y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_batch_with_masks_strides_and_idle_tokens(S):
    """Per-token explicit masks, padded row strides, a token that keeps nothing and one that keeps all."""
    rng = np.random.Generator(np.random.PCG64(31))
    M, K, B = 700, 3000, 4
    W = (rng.standard_normal((M, K)) * (rng.random((M, K)) < 0.4) * 0.05).astype(np.float16)
    X = rng.standard_normal((B, K)).astype(np.float16)
    acts = rng.random((B, K)) < 0.35
    acts[1] = False
    acts[2] = True
    words = np.stack([O.active_to_words(a) for a in acts])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        Xd = torch.zeros((B, K + 24), dtype=torch.float16, device="cuda")
        Xd[:, :K] = dev(X)
        Yd = torch.full((B, M + 5), float("nan"), dtype=torch.float32, device="cuda")
        md = torch.zeros((B, words.shape[1] + 3), dtype=torch.int32, device="cuda")
        md[:, :words.shape[1]] = dev(words.view(np.int32))
        S.spdp_spmspv_batch(h, Xd[:, :K], O.DP_MASK, 0.0, Yd[:, :M], mask=md[:, :words.shape[1]])
        torch.cuda.synchronize()
        out = Yd.cpu().numpy()
        check(out[:, :M], Y_ref, S_ref)
        assert np.all(out[1, :M] == 0.0)                               # nothing kept: zeros, still written
        assert np.all(np.isnan(out[:, M:]))                            # nothing written beyond M
        # odd row stride: the slices of x are no longer 16-byte aligned
        Xo = torch.zeros((B, K + 3), dtype=torch.float16, device="cuda")
        Xo[:, :K] = dev(X)
        Yo = torch.empty((B, M), dtype=torch.float32, device="cuda")
        S.spdp_spmspv_batch(h, Xo[:, :K], O.DP_MASK, 0.0, Yo, mask=md[:, :words.shape[1]])
        torch.cuda.synchronize()
        check(Yo.cpu().numpy(), Y_ref, S_ref)
    finally:
        S.spdp_free(h)


def test_batch_exact_on_integers_and_agrees_with_single_vector_calls(S):
    rng = np.random.Generator(np.random.PCG64(32))
    M, K, B = 900, 1200, 8
    W = rng.integers(-8, 9, (M, K)).astype(np.float16)
    W[rng.random((M, K)) < 0.6] = 0
    X = rng.integers(-4, 5, (B, K)).astype(np.float16)
    acts = np.stack([O.active_ref(X[b], O.DP_ABS_GT, 1.0) for b in range(B)])
    Y_ref, _ = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        Y = run_batch(S, h, X, O.DP_ABS_GT, 1.0, M)
        assert np.array_equal(Y, Y_ref)                                # every partial sum is exact
        for b in range(B):
            y1 = torch.empty(M, dtype=torch.float32, device="cuda")
            S.spdp_spmspv(h, dev(X[b]), O.DP_ABS_GT, 1.0, y1)
            torch.cuda.synchronize()
            assert np.array_equal(y1.cpu().numpy(), Y[b])
    finally:
        S.spdp_free(h)


def test_batch_rejects_bad_arguments(S):
    W = torch.zeros((256, 32), dtype=torch.float16, device="cuda")
    h = S.spdp_pack_tiled_cbc(W)
    try:
        Y9 = torch.zeros((9, 256), dtype=torch.float32, device="cuda")
        X9 = torch.zeros((9, 32), dtype=torch.float16, device="cuda")
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmspv_batch(h, X9, 0, 0.0, Y9)                     # more than 8 tokens
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmspv_batch(h, X9[:2], 2, 0.0, Y9[:2])             # mask rule without masks
        with pytest.raises(S.SpdpError, match="INVALID_ARG"):
            S.spdp_spmspv_batch(h, X9[:1], 0, 0.0, Y9[:1, :100].contiguous())   # fewer than M outputs per token
    finally:
        S.spdp_free(h)


@pytest.mark.parametrize("thr", [0.5, 0.50006103515625, 0.3, 0.0, -0.0, -1.0, 1e-10, 70000.0, float("inf"), float("nan"),
                                 6.1e-5, 5.96e-8])
def test_batch_active_sets_on_threshold_edges(S, thr):
    """W = identity, so y shows each token's active set exactly: values at, just below and just above the
    threshold (in fp16 steps), zeros of both signs, subnormals and the largest finite values.  (Activations
    are kept finite: the tensor-core product multiplies the zeros of a fetched tile with x, so a NaN or Inf
    activation would mark every row of its K-block, which is the dense reading of the definition.)"""
    K = 64
    W = np.eye(K, dtype=np.float16)
    base = np.float16(thr) if np.isfinite(thr) and abs(thr) < 65504 else np.float16(1.0)
    around = [base, np.nextafter(base, np.float16(np.inf)), np.nextafter(base, np.float16(-np.inf)),
              -base, np.float16(0.0), np.float16(-0.0), np.float16(6e-8), np.float16(-6e-8), np.float16(6.1e-5),
              np.float16(65504), np.float16(-65504),
              np.float16(0.25), np.float16(0.5), np.float16(0.75)]
    rng = np.random.Generator(np.random.PCG64(77))
    X = np.zeros((3, K), dtype=np.float16)
    for b in range(3):
        vals = np.array(around, dtype=np.float16)
        X[b, :len(vals)] = rng.permutation(vals)
        X[b, len(vals):] = rng.standard_normal(K - len(vals)).astype(np.float16)
    acts = np.stack([O.active_ref(X[b], O.DP_ABS_GT, thr) for b in range(3)])
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        Y = run_batch(S, h, X, O.DP_ABS_GT, thr, K)
        for b in range(3):
            want = np.where(acts[b], X[b].astype(np.float32), np.float32(0.0))
            assert np.array_equal(Y[b], want), (thr, b)
    finally:
        S.spdp_free(h)


def test_batch_in_a_cuda_graph_next_to_single_calls(S):
    """The batch call only launches: captured with a single-vector call on the same handle and replayed."""
    rng = np.random.Generator(np.random.PCG64(41))
    M, K, B = 1500, 3000, 6
    W = (rng.standard_normal((M, K)) * (rng.random((M, K)) < 0.45) * 0.05).astype(np.float16)
    X = rng.standard_normal((B, K)).astype(np.float16)
    rule, thr = O.DP_ABS_GT, 0.5
    acts = np.stack([O.active_ref(X[b], rule, thr) for b in range(B)])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        Xd = dev(X)
        Y = torch.zeros((B, M), dtype=torch.float32, device="cuda")
        y0 = torch.zeros(M, dtype=torch.float32, device="cuda")
        S.spdp_spmspv_batch(h, Xd, rule, thr, Y)                       # warm-up outside the capture
        S.spdp_spmspv(h, Xd[0], rule, thr, y0)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                S.spdp_spmspv_batch(h, Xd, rule, thr, Y, stream=side.cuda_stream)
                S.spdp_spmspv(h, Xd[0], rule, thr, y0, stream=side.cuda_stream)
                S.spdp_spmspv_batch(h, Xd, rule, thr, Y, stream=side.cuda_stream)
        for _ in range(3):
            Y.fill_(float("nan"))
            y0.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            check(Y.cpu().numpy(), Y_ref, S_ref)
            check(y0.cpu().numpy()[None, :], Y_ref[:1], S_ref[:1])
    finally:
        S.spdp_free(h)


def test_batch_non_finite_values_follow_the_documented_reading(S):
    """Where the batch call departs from the token-by-token definition, pinned so that it cannot drift:
    a token that skips a column enters it with x = 0, so (a) an Inf weight in a column tile that is fetched
    for ANOTHER token gives NaN (0 * Inf) in that row for the token that skips the column -- and only
    there; (b) a NaN activation of a kept column reaches every row of that token (0 * NaN through the
    zeros of the fetched tiles).  Tokens without such values, and all other rows, follow the definition."""
    rng = np.random.Generator(np.random.PCG64(55))
    M, K, B = 300, 64, 4
    W = (rng.standard_normal((M, K)) * (rng.random((M, K)) < 0.5) * 0.05).astype(np.float16)
    W[5, 50] = np.inf
    X = rng.standard_normal((B, K)).astype(np.float16)
    X[0, 50] = 1.0            # token 0 keeps column 50
    X[1, 50] = 0.0            # token 1 skips it (thr = 0 skips exact zeros), token 0 makes it fetched
    X[2, 50] = 0.0
    X[2, 60] = np.nan         # token 2 keeps a NaN activation
    X[3, 50] = 2.0
    rule, thr = O.DP_ABS_GT, 0.0
    acts = np.stack([O.active_ref(X[b], rule, thr) for b in range(B)])
    Y_ref, S_ref = O.spmspv_batch_ref(W, X, acts)
    h = S.spdp_pack_tiled_cbc(dev(W))
    try:
        Y = run_batch(S, h, X, rule, thr, M)
    finally:
        S.spdp_free(h)
    rows = np.arange(M) != 5
    assert Y[0, 5] == np.inf and Y[3, 5] == np.inf                    # kept: Inf * x, as the definition
    check(Y[[0, 3]][:, rows], Y_ref[[0, 3]][:, rows], S_ref[[0, 3]][:, rows])
    assert np.isnan(Y[1, 5]) and np.isfinite(Y_ref[1, 5])             # (a): 0 * Inf where the definition omits
    check(Y[1:2, rows], Y_ref[1:2, rows], S_ref[1:2, rows])           # ... and nowhere else
    assert np.isnan(Y[2]).all()                                       # (b): every row of the token
