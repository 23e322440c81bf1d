"""Pins for the oracle's Tiled-CBC packer / unpacker (Sec. 4.1, Sec. 4.2.1, Sec. 4.2.3).

Nothing here calls the CUDA library.  Expected values are the paper's (tests/golden/*.txt),
closed forms, hand-built arrays, or an independent decoder.
"""
import os

import numpy as np
import pytest

from oracle import spdp_oracle as O
from paper_2607_21985_b200 import workloads as WL

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _rand_sparse(M, K, density, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    W = (rng.standard_normal((M, K), dtype=np.float32) * np.float32(0.02)).astype(np.float16)
    W[rng.random((M, K)) >= density] = 0
    return W


def test_format_constants_match_paper():
    gold = {k: int(v) for k, v in _golden_rows("format_constants.txt")}
    assert O.TILE_M == gold["TILE_M"] and O.TILE_K == gold["TILE_K"]
    assert O.WORDS_PER_COL == gold["WORDS_PER_COLUMN"]
    W = np.zeros((256, 16), np.float16)
    W[:3, 5] = 1.0
    W[:2, 4] = 1.0
    p = O.pack_ref(W)
    ci = int(p["colinfo"][5])
    assert ci >> gold["COLINFO_OFFSET_SHIFT"] == 8 and ci & gold["COLINFO_NNZ_MASK"] == 3
    assert p["tileoffset"].dtype.itemsize == 4 and p["colinfo"].dtype.itemsize == 4
    assert p["bitmap"].dtype.itemsize == 8 and p["values"].dtype.itemsize == 2


def test_padding_rule_paper_example():
    for nnz, padded, pad_bytes in _golden_rows("padding_rule.txt"):
        assert int(O.pad_up(int(nnz))) == int(padded)
        assert 2 * (int(padded) - int(nnz)) == int(pad_bytes)
    assert [int(O.pad_up(n)) for n in (0, 1, 8, 9, 16, 255, 256)] == [0, 8, 8, 16, 16, 256, 256]
    # the packer applies it: a column of 7 nonzeros occupies 8 slots, one of 9 occupies 16
    W = np.zeros((256, 16), np.float16)
    W[:7, 0] = 1.0
    W[:9, 1] = 2.0
    p = O.pack_ref(W)
    assert p["colinfo"][1] >> 16 == 8 and p["colinfo"][2] >> 16 == 24
    assert int(p["tileoffset"][1]) == 24 and len(p["values"]) == 24


@pytest.mark.parametrize("M,K,density,seed", [(256, 16, 0.5, 1), (512, 48, 0.3, 2), (768, 32, 0.9, 3),
                                              (256, 64, 0.0, 4), (256, 32, 1.0, 5)])
def test_storage_formula_exact_without_padding(M, K, density, seed):
    """Sec. 4.1: Stor = 4(NGT+1) + 4*NGT*TILE_K + 8*NBM + 2*NNZ, exact when the pad unit is 1."""
    W = _rand_sparse(M, K, density, seed)
    p = O.pack_ref(W, pad_elems=1)
    nnz = int(np.count_nonzero(W.view(np.uint16) & 0x7FFF))
    assert p["nnz"] == nnz
    NGT = (M // 256) * (K // 16)
    NBM = M * K // 64
    expect = 4 * (NGT + 1) + 4 * NGT * 16 + 8 * NBM + 2 * nnz
    assert O.packed_bytes(p) == expect == O.storage_formula_bytes(M, K, nnz)
    # with the 16-byte padding the only extra bytes are the padding halfwords
    p8 = O.pack_ref(W)
    n = (p8["colinfo"] & 0xFFFF).astype(np.int64)
    assert O.packed_bytes(p8) == expect + 2 * int((O.pad_up(n) - n).sum())


def test_compression_ratio_from_formula():
    """Eq. 1 with the storage formula: metadata is 4/4096 + 4/256 + 8/64 bytes per element, so
    CR(s) = 2 / (0.1416 + 2(1-s)) for large matrices; break-even near 7.1 % sparsity."""
    M = K = 8192
    meta = 4 / 4096 + 4 / 256 + 8 / 64
    for s, cr in ((0.0, 0.934), (0.3, 1.297), (0.5, 1.752), (0.7, 2.697), (0.9, 5.855)):
        nnz = int(round(M * K * (1 - s)))
        got = 2 * M * K / O.storage_formula_bytes(M, K, nnz)
        assert abs(got - cr) < 2e-3
        assert abs(got - 2 / (meta + 2 * (1 - s))) < 1e-4
    assert abs(meta / 2 - 0.0708) < 1e-3


def test_hand_built_tile():
    """A GTile whose every field can be written down by hand: column cc has nonzeros exactly at
    rows 0..(cc mod 8), so n = cc mod 8 + 1 <= 8 and every column pads to 8."""
    W = np.zeros((256, 16), np.float16)
    for cc in range(16):
        for i in range(cc % 8 + 1):
            W[i, cc] = np.float16(1 + cc + i / 8)
    p = O.pack_ref(W)
    assert p["tileoffset"].tolist() == [0, 128]
    for cc in range(16):
        n = cc % 8 + 1
        assert int(p["colinfo"][cc]) == ((8 * cc) << 16) | n
        assert [int(w) for w in p["bitmap"][4 * cc: 4 * cc + 4]] == [(1 << n) - 1, 0, 0, 0]
        seg = p["values"][8 * cc: 8 * cc + 8]
        assert seg[:n].tolist() == W.view(np.uint16)[:n, cc].tolist()
        assert not seg[n:].any()
    # second case: one column with 9 nonzeros at rows 60..68 straddles two bitmap words
    W = np.zeros((256, 16), np.float16)
    W[60:69, 3] = np.arange(1, 10, dtype=np.float16)
    W[255, 15] = np.float16(-2.0)
    p = O.pack_ref(W)
    assert [int(w) for w in p["bitmap"][12:16]] == [0xF << 60, 0x1F, 0, 0]
    assert int(p["colinfo"][3]) == 9 and int(p["colinfo"][4]) == 16 << 16
    assert int(p["colinfo"][15]) == (16 << 16) | 1
    assert [int(w) for w in p["bitmap"][60:64]] == [0, 0, 0, 1 << 63]
    assert p["tileoffset"].tolist() == [0, 24]
    assert p["values"][:9].view(np.float16).tolist() == list(range(1, 10))
    assert p["values"][16] == np.float16(-2.0).view(np.uint16)


def test_gtiles_are_row_major_and_adjacent_along_k():
    """Sec. 4.1 + Alg. 1 (ColInfo + TILE_K is the next iteration's segment): GTile (r, c) has
    linear index r*C + c."""
    M, K = 512, 48
    W = np.zeros((M, K), np.float16)
    W[256 + 5, 16 + 2] = 3.0          # row tile 1, GTile column 1, column 2 of the tile, row 5
    p = O.pack_ref(W)
    g = 1 * 3 + 1
    assert int(p["colinfo"][g * 16 + 2]) & 0xFFFF == 1
    assert int(p["bitmap"][(g * 16 + 2) * 4]) == 1 << 5
    assert np.count_nonzero(p["colinfo"] & 0xFFFF) == 1
    assert p["tileoffset"].tolist() == [0, 0, 0, 0, 0, 8, 8]


@pytest.mark.parametrize("M,K,seed", [(256, 16, 11), (512, 32, 12), (300, 20, 13), (1, 1, 14), (257, 17, 15)])
def test_round_trip_and_independent_decoder(M, K, seed):
    W = WL.special_values_matrix(M, K, seed)
    p = O.pack_ref(W)
    back = O.unpack_ref(p)
    assert np.array_equal(back, O.canon(W))              # bit-exact up to -0 -> +0
    # the per-element decoder uses only the decode rule of Sec. 4.2.1 (bit test + masked popcount)
    rng = np.random.Generator(np.random.PCG64(seed))
    for _ in range(300):
        i, j = int(rng.integers(M)), int(rng.integers(K))
        assert O.decode_element_ref(p, i, j) == int(O.canon(W)[i, j])


@pytest.mark.parametrize("M,K,density,pad,seed", [(512, 64, 0.5, 8, 21), (300, 40, 0.2, 8, 22),
                                                  (256, 16, 0.95, 1, 23), (1024, 16, 0.05, 8, 24)])
def test_invariants_and_fast_packer(M, K, density, pad, seed):
    W = _rand_sparse(M, K, density, seed)
    p = O.pack_ref(W, pad_elems=pad)
    q = O.pack_fast(W, pad_elems=pad)
    for key in ("tileoffset", "colinfo", "bitmap", "values"):
        assert p[key].dtype == q[key].dtype and np.array_equal(p[key], q[key]), key
    nnz = int(np.count_nonzero(W.view(np.uint16) & 0x7FFF))
    popc = sum(bin(int(w)).count("1") for w in p["bitmap"])
    assert popc == nnz == p["nnz"]
    n = (p["colinfo"] & 0xFFFF).astype(np.int64).reshape(-1, 16)
    off = (p["colinfo"] >> 16).astype(np.int64).reshape(-1, 16)
    padded = O.pad_up(n, pad)
    assert np.array_equal(off, np.cumsum(padded, axis=1) - padded)          # prefix sums of pad8
    to = p["tileoffset"].astype(np.int64)
    assert to[0] == 0 and np.all(np.diff(to) == padded.sum(axis=1)) and to[-1] == len(p["values"])
    assert np.all(to % pad == 0)
    # every padding halfword is 0x0000, every stored value is nonzero
    start = (to[:-1, None] + off).reshape(-1)
    for s, k, pk in zip(start, n.reshape(-1), padded.reshape(-1)):
        assert np.all(p["values"][s: s + k] & 0x7FFF) and not p["values"][s + k: s + pk].any()


def test_empty_and_full():
    W = np.zeros((256, 32), np.float16)
    p = O.pack_ref(W)
    assert not p["bitmap"].any() and not p["colinfo"].any() and not p["tileoffset"].any()
    assert len(p["values"]) == 0
    W[:] = 1.0
    p = O.pack_ref(W)
    assert np.all(p["bitmap"] == np.uint64(0xFFFFFFFFFFFFFFFF))
    assert (p["colinfo"] & 0xFFFF).tolist() == [256] * 32
    assert (p["colinfo"][:16] >> 16).tolist() == [256 * c for c in range(16)]   # max offset 3840 < 2^16
    assert p["tileoffset"].tolist() == [0, 4096, 8192]


def test_active_bytes_model():
    """Bytes per active column tile: 32 (bitmap) + 2*pad8(n) (values) + 4 (ColInfo)."""
    W = np.zeros((512, 32), np.float16)
    W[:7, 0] = 1.0           # pad8 -> 8 in row tile 0
    W[256:256 + 9, 0] = 1.0  # pad8 -> 16 in row tile 1
    W[:, 20] = 1.0           # 256 + 256
    p = O.pack_ref(W)
    a = np.zeros(32, bool)
    a[0] = True
    base = 2 * 32 + 2 * 512
    assert O.active_bytes(p, a) == (36 + 16) + (36 + 32) + 4 * (2 + 1) + base
    a[20] = True
    assert O.active_bytes(p, a) == (36 + 16) + (36 + 32) + 2 * (36 + 512) + 4 * (4 + 1) + base
    assert O.active_bytes(p, np.zeros(32, bool), 4) == 4 + 2 * 32 + 4 * 512
