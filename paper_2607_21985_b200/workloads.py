"""Seeded synthetic inputs: pruned fp16 weight matrices, activation vectors, DP thresholds.

Input generation only -- no Tiled-CBC, no DP rule, no products.  The tests, the smoke check
and the benchmark feed the SAME arrays from here to the CUDA library and to the CPU oracle.

The layers stand in for the paper's kernel workloads (real pruned projection matrices of the
LLM shape set of Sec. 5.3, unstructured static sparsity and dynamic sparsity of 30-50 %,
batch 1, fp16): same shapes class, dtype, sparsity regime and batch size, random values.

Recipe (every config): rng_W, rng_x = PCG64 streams spawned from SeedSequence(seed);
W ~ N(0, 0.02^2) drawn in float32 row-major, pruned in float32, cast to fp16
(round-to-nearest-even); x drawn in float32 (float64 for Laplace), cast to fp16.
"Magnitude-pruned to sparsity s": the floor(s*M*K) smallest |w| of the whole matrix become 0.
"Skip p of the columns": thr = midpoint (fp32) between the k-th and (k+1)-th smallest |x_j|
of the fp16 vector, k = round(p*K); if the two are equal thr is that value.  The library only
ever receives the scalar thr.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

DP_NONE, DP_ABS_GT, DP_MASK = 0, 1, 2


@dataclass
class Workload:
    name: str
    M: int
    K: int
    W: np.ndarray            # float16 [M, K], statically pruned (zeros are the pruned weights)
    x: np.ndarray            # float16 [K]
    rule: int
    thr: float
    weight_sparsity: float   # realised fraction of zero weights
    skip_target: float       # requested fraction of skipped columns


def _rngs(seed: int):
    ss = np.random.SeedSequence(seed).spawn(2)
    return np.random.Generator(np.random.PCG64(ss[0])), np.random.Generator(np.random.PCG64(ss[1]))


def normal_weights(rng, M: int, K: int, std: float = 0.02) -> np.ndarray:
    return rng.standard_normal((M, K), dtype=np.float32) * np.float32(std)


def prune_global_magnitude(G: np.ndarray, sparsity: float) -> np.ndarray:
    """Zero the floor(s*size) smallest-magnitude entries of the whole float32 matrix (in place)."""
    k = int(np.floor(sparsity * G.size))
    if k <= 0:
        return G
    a = np.abs(G).reshape(-1)
    tau = np.partition(a, k - 1)[k - 1]
    del a
    G[np.abs(G) <= tau] = 0
    return G


def prune_per_column(G: np.ndarray, col_sparsity: np.ndarray) -> np.ndarray:
    """Column j keeps its round((1-s_j)*M) largest-magnitude entries (in place)."""
    M, K = G.shape
    At = np.ascontiguousarray(np.abs(G).T)                     # [K, M], one column per row
    tau = np.full(K, -1.0, dtype=np.float32)
    for j in range(K):
        drop = M - int(round((1.0 - float(col_sparsity[j])) * M))
        if drop > 0:
            tau[j] = np.partition(At[j], drop - 1)[drop - 1]
    del At
    G[np.abs(G) <= tau[None, :]] = 0
    return G


def skip_threshold(x16: np.ndarray, skip: float):
    """(rule, thr) that skips the round(skip*K) columns of smallest |x_j| (see module docstring)."""
    K = x16.shape[0]
    k = int(round(skip * K))
    if k <= 0:
        return DP_NONE, -1.0
    a = np.sort(np.abs(x16.astype(np.float32)))
    if k >= K:
        return DP_ABS_GT, float(a[-1])
    lo, hi = a[k - 1], a[k]
    thr = np.float32(lo) if lo == hi else np.float32((np.float32(lo) + np.float32(hi)) * np.float32(0.5))
    return DP_ABS_GT, float(thr)


def _finish(name, G, x32, skip) -> Workload:
    W = G.astype(np.float16)
    x = np.asarray(x32).astype(np.float16)
    rule, thr = skip_threshold(x, skip)
    return Workload(name, W.shape[0], W.shape[1], W, x, rule, thr, float((W == 0).mean()), skip)


def config1(M=4096, K=4096, seed=0) -> Workload:
    """Single layer, W 50 % magnitude-pruned, x ~ N(0,1), 50 % of the columns skipped."""
    rw, rx = _rngs(seed)
    G = prune_global_magnitude(normal_weights(rw, M, K), 0.50)
    return _finish(f"c1_{M}x{K}_sp50_dp50", G, rx.standard_normal(K, dtype=np.float32), 0.50)


def config2(M=11008, K=4096, seed=1) -> Workload:
    """Llama-7B-shaped MLP up-projection, W 60 % sparse, x ~ Laplace(0,1), 50 % skipped."""
    rw, rx = _rngs(seed)
    G = prune_global_magnitude(normal_weights(rw, M, K), 0.60)
    return _finish(f"c2_{M}x{K}_sp60_dp50", G, rx.laplace(0.0, 1.0, K).astype(np.float32), 0.50)


def config3(M=4096, K=11008, seed=2) -> Workload:
    """Llama-7B-shaped MLP down-projection, W 70 % sparse, x = ReLU(N(0,1)), ~90 % skipped."""
    rw, rx = _rngs(seed)
    G = prune_global_magnitude(normal_weights(rw, M, K), 0.70)
    x = np.maximum(rx.standard_normal(K, dtype=np.float32), np.float32(0))
    return _finish(f"c3_{M}x{K}_sp70_dp90", G, x, 0.90)


def config4(M=28672, K=8192, seed=3) -> Workload:
    """Llama-70B-shaped MLP, W 50 % sparse with per-column sparsity 0.5 + 0.2*U(-1,1),
    x ~ N(0,1), 40 % skipped."""
    rw, rx = _rngs(seed)
    G = normal_weights(rw, M, K)
    s = 0.5 + 0.2 * rw.uniform(-1.0, 1.0, K)
    G = prune_per_column(G, s)
    return _finish(f"c4_{M}x{K}_sp50pm20_dp40", G, rx.standard_normal(K, dtype=np.float32), 0.40)


SWEEP_SP = (0.30, 0.50, 0.70, 0.90)
SWEEP_DP = (0.0, 0.25, 0.50, 0.75)


def config5(i_s: int, i_d: int, M=8192, K=8192) -> Workload:
    """One point of the 8192 x 8192 sweep: weight sparsity SWEEP_SP[i_s], skip SWEEP_DP[i_d]."""
    rw, rx = _rngs(100 + 4 * i_s + i_d)
    sp, dp = SWEEP_SP[i_s], SWEEP_DP[i_d]
    G = prune_global_magnitude(normal_weights(rw, M, K), sp)
    return _finish(f"c5_{M}x{K}_sp{int(sp * 100)}_dp{int(dp * 100)}", G,
                   rx.standard_normal(K, dtype=np.float32), dp)


def special_values_matrix(M: int, K: int, seed: int) -> np.ndarray:
    """fp16 matrix sprinkled with -0.0, NaN, +-Inf, subnormals, empty and full columns."""
    rng = np.random.Generator(np.random.PCG64(seed))
    W = (rng.standard_normal((M, K), dtype=np.float32) * np.float32(0.02)).astype(np.float16)
    W[rng.random((M, K)) < 0.5] = 0
    b = W.view(np.uint16)
    specials = np.array([0x8000, 0x7E00, 0xFE01, 0x7C00, 0xFC00, 0x0001, 0x8001, 0x03FF, 0x7BFF], np.uint16)
    pick = rng.random((M, K)) < 0.05
    b[pick] = specials[rng.integers(0, len(specials), int(pick.sum()))]
    if K >= 3:
        b[:, 1] = 0                         # an empty column
        b[:, 2] = 0x3C00                    # a full column (all 1.0)
    return W
