"""CPU oracle for the SPDP decode path (Tiled-CBC pack / unpack, DP active set, spMspV).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA
library is checked against.  It may be imported by the test-suite, by the smoke check and by
the benchmark's CPU-baseline leg, and by nothing else.  It shares no code with the CUDA path
and imports nothing from the package; the package imports nothing from here.

Everything is NumPy on the host.  Floating point is fp64 (the paper fixes no accumulator
precision; the fp16 inputs widen to fp64 exactly).  fp16 tensors travel as ``np.uint16`` bit
patterns or ``np.float16`` arrays; the packed format is compared byte for byte, so bit patterns
are never re-rounded.

What follows the paper, and where:

* Static pruning is a fixed 0/1 mask on W (Sec. 2.2, "Static Pruning", W_sp = W (.) M).
* Dynamic pruning is a 0/1 mask chosen by the input x, column-wise (Sec. 2.2, "Dynamic
  Pruning", W_dp(x) = W (.) M(x)); the decode kernel tests a magnitude metric of x_j against a
  threshold (Sec. 4.2 step (3), Sec. 4.2.3).
* Tiled-CBC (Sec. 4.1): column tiles of TILE_M x 1 = 256 x 1, four 64-bit bitmap words per
  column tile, GTiles of TILE_M x TILE_K = 256 x 16 stored in row-major GTile order, arrays
  TileOffset / Values / Bitmap / ColInfo, ColInfo = (column start offset in the tile) << 16 |
  (nonzeros in the column).
* Each column's values are padded to a 16-byte boundary, i.e. to a multiple of 8 fp16
  (Sec. 4.2.3, the "7 values -> 2 bytes of padding" example).
* Storage cost (Sec. 4.1): 4(NGT+1) + 4*NGT*TILE_K + 8*NBM + 2*NNZ bytes.
* Decoding (Sec. 4.2.1): an element whose bit is set is Values[base + rank], rank = number of
  set bits before its position.

Readings taken where the paper is silent (each is listed in the design notes of the repo):
bit b of word w of a column tile is row 64*w + b (least significant bit first); offsets are
counted in fp16 elements, padding included; "nonzero" means (bits & 0x7FFF) != 0, so -0.0 is
dropped and NaN/Inf/subnormals are kept verbatim; a column is active iff NOT(|x_j| <= thr)
evaluated on the exactly widened fp16 value, so ties are skipped and NaN is active; an active
column is multiplied by the unmodified x_j; matrices whose sides are not multiples of the tile
are zero-extended logically.

Parity pins live in tests/test_oracle_*.py.  What stays "parity unpinned": the bit order,
word order and offset units are this file's reading (no file of the authors exists to compare
with); they are pinned only against the decode rule and the round trip.
"""
from __future__ import annotations

import numpy as np

TILE_M = 256          # rows per column tile (Sec. 4.1, Tiling Design)
TILE_K = 16           # column tiles per GTile (Sec. 4.2.3)
WORDS_PER_COL = 4     # 64-bit bitmap words per column tile (Sec. 4.1)
PAD_ELEMS = 8         # 16-byte padding of every column's values (Sec. 4.2.3)

DP_NONE = 0           # every column active
DP_ABS_GT = 1         # active iff not (|x_j| <= thr)
DP_MASK = 2           # explicit K-bit mask (Sec. 6, DP variants that materialise masks)


# --------------------------------------------------------------------------------------
# helpers that are not part of the method: dtype plumbing only
# --------------------------------------------------------------------------------------
def as_bits(a) -> np.ndarray:
    """fp16 array (np.float16 or np.uint16 bit patterns) -> np.uint16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.float16:
        return a.view(np.uint16)
    if a.dtype == np.uint16:
        return a
    raise TypeError(f"expected float16 or uint16 bit patterns, got {a.dtype}")


def as_f64(bits) -> np.ndarray:
    """fp16 bit patterns -> float64, exactly."""
    return as_bits(bits).view(np.float16).astype(np.float64)


def pad_up(n, pad_elems: int = PAD_ELEMS):
    """Padded length of a column with n nonzeros (Sec. 4.2.3: 7 -> 8, 8 -> 8, 9 -> 16, 0 -> 0)."""
    return (np.asarray(n) + pad_elems - 1) // pad_elems * pad_elems


def grid(M: int, K: int):
    """(R, C, NGT): row tiles, GTile columns, number of GTiles (Sec. 4.1, NGT)."""
    R = (M + TILE_M - 1) // TILE_M
    C = (K + TILE_K - 1) // TILE_K
    return R, C, R * C


# --------------------------------------------------------------------------------------
# Tiled-CBC (Sec. 4.1)
# --------------------------------------------------------------------------------------
def is_nonzero(bits) -> np.ndarray:
    """The stored-element predicate: an fp16 is kept iff it is not +0 or -0."""
    return (as_bits(bits) & np.uint16(0x7FFF)) != 0


def canon(W) -> np.ndarray:
    """What a pack -> unpack round trip returns: W with every -0.0 replaced by +0.0 (bits)."""
    b = as_bits(W).copy()
    b[~is_nonzero(b)] = 0
    return b


def pack_ref(W, pad_elems: int = PAD_ELEMS) -> dict:
    """Dense row-major fp16 W[M][K] -> the four Tiled-CBC arrays (Sec. 4.1, Storage Structure).

    Written as the definition: loop over GTiles in row-major order, over the 16 columns of a
    GTile, over the 256 rows of a column tile.  Slow on purpose; use small matrices.
    Returns dict(M, K, pad_elems, tileoffset u32[NGT+1], colinfo u32[NGT*16],
    bitmap u64[NGT*16*4], values u16[TileOffset[NGT]], nnz).
    """
    Wb = as_bits(W)
    M, K = Wb.shape
    R, C, NGT = grid(M, K)
    tileoffset = np.zeros(NGT + 1, dtype=np.uint32)
    colinfo = np.zeros(NGT * TILE_K, dtype=np.uint32)
    bitmap = np.zeros(NGT * TILE_K * WORDS_PER_COL, dtype=np.uint64)
    values = []
    nnz = 0
    for r in range(R):
        for c in range(C):
            g = r * C + c                                  # GTiles in row-major order
            tile_start = len(values)
            if tile_start >= 1 << 32:
                raise OverflowError("TileOffset does not fit 32 bits")
            tileoffset[g] = tile_start
            for cc in range(TILE_K):
                j = c * TILE_K + cc
                off = len(values) - tile_start             # TileOffset_Col, in fp16 elements
                n = 0
                if j < K:
                    for p in range(TILE_M):
                        i = r * TILE_M + p
                        if i < M and (int(Wb[i, j]) & 0x7FFF) != 0:
                            w, b = divmod(p, 64)
                            bitmap[(g * TILE_K + cc) * WORDS_PER_COL + w] |= np.uint64(1) << np.uint64(b)
                            values.append(int(Wb[i, j]))   # nonzeros of the column in row order
                            n += 1
                values.extend([0] * (int(pad_up(n, pad_elems)) - n))   # pad with 0x0000
                assert off < 1 << 16 and n <= TILE_M
                colinfo[g * TILE_K + cc] = (off << 16) | n  # upper 16: offset, lower 16: nnz
                nnz += n
    if len(values) >= 1 << 32:
        raise OverflowError("TileOffset does not fit 32 bits")
    tileoffset[NGT] = len(values)
    return dict(M=M, K=K, pad_elems=pad_elems, tileoffset=tileoffset, colinfo=colinfo,
                bitmap=bitmap, values=np.asarray(values, dtype=np.uint16), nnz=nnz)


def pack_fast(W, pad_elems: int = PAD_ELEMS) -> dict:
    """Same arrays as pack_ref, computed with whole-array NumPy steps so that mid-size matrices
    finish in seconds.  tests/test_oracle_format.py checks it byte for byte against pack_ref."""
    Wb = as_bits(W)
    M, K = Wb.shape
    R, C, NGT = grid(M, K)
    Wp = np.zeros((R * TILE_M, C * TILE_K), dtype=np.uint16)      # logical zero extension
    Wp[:M, :K] = Wb
    # [R, 256, C, 16] -> [R, C, 16, 256]: GTile-major, then column of the tile, then row.
    T = Wp.reshape(R, TILE_M, C, TILE_K).transpose(0, 2, 3, 1).reshape(NGT * TILE_K, TILE_M)
    nzmask = (T & np.uint16(0x7FFF)) != 0
    bitmap = np.ascontiguousarray(np.packbits(nzmask, axis=1, bitorder="little")).reshape(-1).view(np.uint64).copy()
    n = nzmask.sum(axis=1).astype(np.int64)                       # nnz of every column tile
    padded = pad_up(n, pad_elems).astype(np.int64)
    start = np.concatenate([[0], np.cumsum(padded)])              # column start in Values
    if start[-1] >= 1 << 32:
        raise OverflowError("TileOffset does not fit 32 bits")
    tileoffset = start[:: TILE_K].astype(np.uint32)               # every 16th column start
    off_in_tile = start[:-1] - np.repeat(start[:-1:TILE_K], TILE_K)
    colinfo = ((off_in_tile << 16) | n).astype(np.uint32)
    values = np.zeros(int(start[-1]), dtype=np.uint16)
    rank = np.cumsum(nzmask, axis=1) - 1                          # rank of every set bit
    dest = (start[:-1, None] + rank)[nzmask]
    values[dest] = T[nzmask]
    return dict(M=M, K=K, pad_elems=pad_elems, tileoffset=tileoffset, colinfo=colinfo,
                bitmap=bitmap, values=values, nnz=int(n.sum()))


def decode_element_ref(p: dict, i: int, j: int) -> int:
    """One element of the packed matrix from the decode rule alone (Sec. 4.2.1):
    bit clear -> 0, else Values[TileOffset[g] + TileOffset_Col + rank] with rank the number of
    set bits before the element's position in its column tile."""
    _, C, _ = grid(p["M"], p["K"])
    r, pos = divmod(i, TILE_M)
    c, cc = divmod(j, TILE_K)
    slot = (r * C + c) * TILE_K + cc
    w, b = divmod(pos, 64)
    words = [int(x) for x in p["bitmap"][slot * WORDS_PER_COL: slot * WORDS_PER_COL + WORDS_PER_COL]]
    if not (words[w] >> b) & 1:
        return 0
    rank = sum(bin(words[q]).count("1") for q in range(w)) + bin(words[w] & ((1 << b) - 1)).count("1")
    base = int(p["tileoffset"][r * C + c]) + (int(p["colinfo"][slot]) >> 16)
    return int(p["values"][base + rank])


def unpack_ref(p: dict) -> np.ndarray:
    """Packed arrays -> dense fp16 bit patterns [M][K], column tile by column tile: walk the
    set bits of a column in row order and take the column's values in storage order."""
    M, K = p["M"], p["K"]
    R, C, _ = grid(M, K)
    out = np.zeros((M, K), dtype=np.uint16)
    for r in range(R):
        for c in range(C):
            g = r * C + c
            for cc in range(TILE_K):
                j = c * TILE_K + cc
                slot = g * TILE_K + cc
                ci = int(p["colinfo"][slot])
                nxt = int(p["tileoffset"][g]) + (ci >> 16)
                for w in range(WORDS_PER_COL):
                    word = int(p["bitmap"][slot * WORDS_PER_COL + w])
                    for b in range(64):
                        if (word >> b) & 1:
                            out[r * TILE_M + 64 * w + b, j] = p["values"][nxt]
                            nxt += 1
                assert nxt - int(p["tileoffset"][g]) - (ci >> 16) == (ci & 0xFFFF)
    return out


def storage_formula_bytes(M: int, K: int, nnz: int) -> int:
    """Stor_Tiled-CBC of Sec. 4.1 (no padding term): 4(NGT+1) + 4*NGT*TILE_K + 8*NBM + 2*NNZ."""
    _, _, NGT = grid(M, K)
    NBM = NGT * TILE_K * WORDS_PER_COL      # = M*K/64 when the tile sizes divide M and K
    return 4 * (NGT + 1) + 4 * NGT * TILE_K + 8 * NBM + 2 * nnz


def packed_bytes(p: dict) -> int:
    """Bytes the four arrays actually occupy."""
    return int(p["tileoffset"].nbytes + p["colinfo"].nbytes + p["bitmap"].nbytes + p["values"].nbytes)


# --------------------------------------------------------------------------------------
# Dynamic pruning: the active column set (Sec. 2.2; Sec. 4.2 steps (2)-(3))
# --------------------------------------------------------------------------------------
def active_ref(x, rule: int, thr: float = 0.0, mask_words=None) -> np.ndarray:
    """Boolean K-vector: column j is fetched and multiplied iff active[j].

    DP_ABS_GT: active iff not (|x_j| <= thr), compared in fp32 on the exactly widened fp16
    value with thr rounded to fp32 (a tie is skipped; NaN is active; thr < 0 keeps all).
    DP_MASK: bit (j % 32) of 32-bit word j // 32."""
    xb = as_bits(x)
    K = xb.shape[0]
    if rule == DP_NONE:
        return np.ones(K, dtype=bool)
    if rule == DP_ABS_GT:
        xf = xb.view(np.float16).astype(np.float32)
        with np.errstate(invalid="ignore"):
            return ~(np.abs(xf) <= np.float32(thr))
    if rule == DP_MASK:
        mw = np.asarray(mask_words, dtype=np.uint32)
        j = np.arange(K)
        return ((mw[j // 32] >> (j % 32).astype(np.uint32)) & 1).astype(bool)
    raise ValueError("unknown DP rule")


def active_to_words(active) -> np.ndarray:
    """Boolean K-vector -> ceil(K/32) uint32 words, bit j%32 of word j//32."""
    a = np.asarray(active, dtype=bool)
    K = a.shape[0]
    padded = np.zeros((K + 31) // 32 * 32, dtype=bool)
    padded[:K] = a
    return np.packbits(padded, bitorder="little").view(np.uint32).copy()


# --------------------------------------------------------------------------------------
# spMspV: the result and its error scale (plain definition)
# --------------------------------------------------------------------------------------
def spmspv_ref(W, x, active):
    """y[i] = sum_{j active} W[i][j] * x[j] in fp64 over the dense masked matrix, and the error
    scale S[i] = sum_{j active} |W[i][j] * x[j]|.  Inactive columns are left out of the sum
    (not multiplied by zero).  Returns (y, S) as float64 arrays of length M."""
    Wd = as_f64(W)
    xd = as_f64(x)
    idx = np.flatnonzero(np.asarray(active, dtype=bool))
    Wa = Wd[:, idx]
    xa = xd[idx]
    y = Wa @ xa
    S = np.abs(Wa) @ np.abs(xa)
    return y, S


def spmspv_bruteforce(W, x, active):
    """The same sums as spmspv_ref as an explicit double loop (tiny inputs only)."""
    Wd = as_f64(W)
    xd = as_f64(x)
    M, K = Wd.shape
    y = np.zeros(M)
    S = np.zeros(M)
    for i in range(M):
        for j in range(K):
            if active[j]:
                t = float(Wd[i, j]) * float(xd[j])
                y[i] += t
                S[i] += abs(t)
    return y, S


def spmspv_batch_ref(W, X, actives):
    """Small-batch decode (the paper's future work, Sec. 6): B tokens share one pass over W_sp and
    every token keeps its own active set.  The result is the single-vector definition of Sec. 4.2
    applied token by token: Y[b][i] = sum_{j in A_b} W[i][j] * X[b][j], S[b][i] the matching error
    scale.  X is [B][K], actives is [B][K] bool.  Returns (Y, S), float64 [B][M]."""
    X = np.asarray(X)
    actives = np.asarray(actives, dtype=bool)
    ys, ss = [], []
    for b in range(X.shape[0]):
        y, S = spmspv_ref(W, X[b], actives[b])
        ys.append(y)
        ss.append(S)
    return np.stack(ys), np.stack(ss)


def union_active(actives) -> np.ndarray:
    """Columns that at least one token of the batch keeps: what a batched call has to fetch."""
    return np.asarray(actives, dtype=bool).any(axis=0)


def active_bytes_batch(p: dict, actives, y_bytes_per_elem: int = 2) -> int:
    """Bytes a batched call must move: the matrix bytes of the union of the tokens' active columns
    (once), and every token's x and y."""
    actives = np.asarray(actives, dtype=bool)
    B = actives.shape[0]
    one = active_bytes(p, union_active(actives), y_bytes_per_elem)
    return one + (B - 1) * (2 * p["K"] + y_bytes_per_elem * p["M"])


def spmm_ref(W, X):
    """Prefill product on the statically pruned matrix alone (Sec. 4.3, SPDP-SpMM: N tokens, static
    pruning only, no dynamic pruning): Y[n][i] = sum_j W[i][j] * X[n][j] in fp64 over the dense masked
    matrix, and the error scale S[n][i] = sum_j |W[i][j] * X[n][j]|.  X is [N][K] (one token per row),
    Y and S are float64 [N][M]."""
    Wd = as_f64(W)
    Xd = as_f64(X)
    return Xd @ Wd.T, np.abs(Xd) @ np.abs(Wd).T


# --------------------------------------------------------------------------------------
# Low-bit Values payload (Sec. 5.1: 4-bit round-to-nearest weights, applied in the order static
# pruning -> quantisation -> dynamic pruning; Sec. 6: Values are stored apart from the sparsity
# metadata, so they can be low-bit).  The paper fixes no packed layout for it; this one keeps
# TileOffset / ColInfo / Bitmap as they are and replaces Values by 4-bit codes plus one fp16 scale
# per column tile:
#   scale  = fp16( max|w| of the column tile's stored values / 7 )          (computed in fp32)
#   q      = clamp( rint( w / scale ), -7, 7 )   in fp32, ties to even;  q = 0 where scale == 0
#   code   = q + 8   (1..15; 0 never encodes a stored value)
#   Codes  : per column tile its n codes in row order, two per byte (even rank = low nibble),
#            zero-padded to 32 codes (16 bytes); TileOffset and ColInfo offsets count CODES
#   weight = (code - 8) * scale
# Non-finite weights are outside this variant (their codes are unspecified).
# --------------------------------------------------------------------------------------
Q4_PAD = 32


def quantise_q4_ref(vals):
    """One column tile's stored values (fp16) -> (scale as fp16 bits, codes uint8 in 1..15)."""
    v32 = as_bits(np.asarray(vals)).view(np.float16).astype(np.float32)
    if v32.size == 0:
        return np.uint16(0), np.zeros(0, np.uint8)
    s16 = (np.max(np.abs(v32)) / np.float32(7.0)).astype(np.float16)
    s32 = np.float32(s16)
    if s32 == 0:
        q = np.zeros(v32.shape, np.int32)
    else:
        q = np.clip(np.rint(v32 / s32), -7, 7).astype(np.int32)
    return s16.view(np.uint16), (q + 8).astype(np.uint8)


def pack_q4_ref(W) -> dict:
    """Dense pruned fp16 W -> the 4-bit variant of Tiled-CBC, written as the definition (loops over
    GTiles and columns).  Returns dict(M, K, pad_elems=32, tileoffset u32[NGT+1] (in codes),
    colinfo u32[NGT*16] (offset in codes << 16 | nnz), bitmap u64[NGT*64], codes u8[TileOffset[NGT]/2],
    scales u16[NGT*16] (fp16 bits), nnz)."""
    Wb = as_bits(W)
    M, K = Wb.shape
    R, C, NGT = grid(M, K)
    base = pack_ref(Wb, pad_elems=Q4_PAD)                  # same bitmap; offsets with the 32-code padding
    scales = np.zeros(NGT * TILE_K, dtype=np.uint16)
    nibbles = np.zeros(int(base["tileoffset"][NGT]), dtype=np.uint8)
    for g in range(NGT):
        for cc in range(TILE_K):
            slot = g * TILE_K + cc
            ci = int(base["colinfo"][slot])
            start, n = int(base["tileoffset"][g]) + (ci >> 16), ci & 0xFFFF
            s16, codes = quantise_q4_ref(base["values"][start:start + n])
            scales[slot] = s16
            nibbles[start:start + n] = codes
    codes = (nibbles[0::2] | (nibbles[1::2] << 4)).astype(np.uint8)
    return dict(M=M, K=K, pad_elems=Q4_PAD, tileoffset=base["tileoffset"], colinfo=base["colinfo"],
                bitmap=base["bitmap"], codes=codes, scales=scales, nnz=base["nnz"])


def pack_q4_fast(W) -> dict:
    """Same arrays as pack_q4_ref with whole-array NumPy steps (checked byte for byte against it)."""
    Wb = as_bits(W)
    base = pack_fast(Wb, pad_elems=Q4_PAD)
    NGT = base["tileoffset"].shape[0] - 1
    n = (base["colinfo"] & np.uint32(0xFFFF)).astype(np.int64)
    start = np.repeat(base["tileoffset"][:-1].astype(np.int64), TILE_K) + (base["colinfo"] >> 16).astype(np.int64)
    v32 = base["values"].view(np.float16).astype(np.float32)
    owner = np.repeat(np.arange(NGT * TILE_K), pad_up(n, Q4_PAD))       # column tile of every (padded) element
    stored = np.zeros(v32.shape[0], dtype=bool)
    idx = np.concatenate([np.arange(s, s + k) for s, k in zip(start, n)]) if n.sum() else np.zeros(0, np.int64)
    stored[idx] = True
    mx = np.zeros(NGT * TILE_K, dtype=np.float32)
    np.maximum.at(mx, owner[stored], np.abs(v32[stored]))
    s16 = (mx / np.float32(7.0)).astype(np.float16)
    s32 = s16.astype(np.float32)
    per = s32[owner]
    with np.errstate(divide="ignore", invalid="ignore"):
        q = np.where(per == 0, np.float32(0), np.clip(np.rint(v32 / per), -7, 7))
    nibbles = np.where(stored, q.astype(np.int32) + 8, 0).astype(np.uint8)
    codes = (nibbles[0::2] | (nibbles[1::2] << 4)).astype(np.uint8)
    return dict(M=base["M"], K=base["K"], pad_elems=Q4_PAD, tileoffset=base["tileoffset"], colinfo=base["colinfo"],
                bitmap=base["bitmap"], codes=codes, scales=s16.view(np.uint16), nnz=base["nnz"])


def dequant_q4_ref(p: dict) -> np.ndarray:
    """The weights the 4-bit arrays stand for, dense float64 [M][K]: bit clear -> 0, else
    (code - 8) * scale with the code found by the decode rule of Sec. 4.2.1 (rank = set bits before)."""
    M, K = p["M"], p["K"]
    R, C, _ = grid(M, K)
    out = np.zeros((M, K), dtype=np.float64)
    nib = np.empty(p["codes"].shape[0] * 2, dtype=np.uint8)
    nib[0::2] = p["codes"] & 15
    nib[1::2] = p["codes"] >> 4
    for r in range(R):
        for c in range(C):
            g = r * C + c
            for cc in range(TILE_K):
                j = c * TILE_K + cc
                slot = g * TILE_K + cc
                nxt = int(p["tileoffset"][g]) + (int(p["colinfo"][slot]) >> 16)
                s = float(np.uint16(p["scales"][slot]).view(np.float16))
                for w in range(WORDS_PER_COL):
                    word = int(p["bitmap"][slot * WORDS_PER_COL + w])
                    for b in range(64):
                        if (word >> b) & 1:
                            out[r * TILE_M + 64 * w + b, j] = (int(nib[nxt]) - 8) * s
                            nxt += 1
    return out


def spmspv_dense64_ref(Wd, x, active):
    """The spMspV definition on a float64 weight matrix (the dequantised weights): (y, S)."""
    xd = as_f64(x)
    idx = np.flatnonzero(np.asarray(active, dtype=bool))
    Wa = np.asarray(Wd, dtype=np.float64)[:, idx]
    return Wa @ xd[idx], np.abs(Wa) @ np.abs(xd[idx])


def active_bytes_q4(p: dict, active, y_bytes_per_elem: int = 2) -> int:
    """Byte model of one call on the 4-bit variant: per active column tile 32 B of bitmap, its padded
    codes (half a byte each), 4 B of ColInfo and 2 B of scale; TileOffset, x and y as before."""
    M, K = p["M"], p["K"]
    R, C, _ = grid(M, K)
    a = np.zeros(C * TILE_K, dtype=bool)
    a[:K] = np.asarray(active, dtype=bool)
    n = (p["colinfo"] & np.uint32(0xFFFF)).astype(np.int64).reshape(R, C * TILE_K)
    per_tile = 32 + pad_up(n, Q4_PAD) // 2 + 4 + 2
    gt_active = int(a.reshape(C, TILE_K).any(axis=1).sum()) * R
    return int(per_tile[:, a].sum()) + 4 * (gt_active + 1) + 2 * K + y_bytes_per_elem * M


def swiglu_ref(gate, up) -> np.ndarray:
    """The activation in front of a gated MLP's down-projection, x = silu(gate) * up with
    silu(g) = g / (1 + exp(-g)), in fp64 on the exactly widened fp16 inputs.  Returns float64 [K]
    (a producer kernel rounds it to fp16; the DP decision is then taken on the rounded value)."""
    g, u = as_f64(gate), as_f64(up)
    return g / (1.0 + np.exp(-g)) * u


def tolerance(S) -> np.ndarray:
    """Per-output bound of the parity gate: 1e-3 * S[i] + 1e-5."""
    return 1e-3 * np.asarray(S, dtype=np.float64) + 1e-5


# --------------------------------------------------------------------------------------
# Byte model for the roofline (same form as Eq. 3: traffic ~ (M/CR)(1-s) + N)
# --------------------------------------------------------------------------------------
def active_bytes(p: dict, active, y_bytes_per_elem: int = 2) -> int:
    """Bytes the method must move for one call: per active column tile its 32-byte bitmap, its
    padded values and its ColInfo word; one TileOffset word per GTile holding an active column
    (plus one); x and y."""
    M, K = p["M"], p["K"]
    R, C, NGT = grid(M, K)
    a = np.zeros(C * TILE_K, dtype=bool)
    a[:K] = np.asarray(active, dtype=bool)
    n = (p["colinfo"] & np.uint32(0xFFFF)).astype(np.int64).reshape(R, C * TILE_K)
    per_tile = 32 + 2 * pad_up(n, p["pad_elems"]) + 4
    total = int(per_tile[:, a].sum())
    gt_active = int(a.reshape(C, TILE_K).any(axis=1).sum()) * R
    return total + 4 * (gt_active + 1) + 2 * K + y_bytes_per_elem * M
