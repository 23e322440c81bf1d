"""The helpers the kernels share with the host (csrc/spdp_hostdev.h), compiled for the host and
run without a GPU: the split of the GTiles over the CTAs at the limits of its 32-bit arithmetic,
and the range check of the checked build on made-up indices (its firing path is only ever
exercised here, never by feeding bad data to a GPU)."""
import ctypes
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def H(tmp_path_factory):
    out = tmp_path_factory.mktemp("hostdev") / "libhostdev_shim.so"
    subprocess.run(["g++", "-O1", "-shared", "-fPIC", "-I", os.path.join(ROOT, "paper_2607_21985_b200", "csrc"),
                    "-o", str(out), os.path.join(ROOT, "tests", "hostdev_shim.cpp")], check=True)
    L = ctypes.CDLL(str(out))
    L.shim_range_begin.restype = ctypes.c_uint
    L.shim_range_begin.argtypes = [ctypes.c_uint] * 3
    L.shim_range_owner.argtypes = [ctypes.c_uint] * 3
    L.shim_span_ok.argtypes = [ctypes.c_ulonglong] * 3
    return L


@pytest.mark.parametrize("ngt,P", [(1, 1), (7, 3), (4096, 148), (57344, 148), (11008, 1000), ((1 << 22) - 1, 1024),
                                   ((1 << 22) - 1, 1023), (1 << 21, 1024)])
def test_ranges_partition_the_gtiles_and_owner_inverts_them(H, ngt, P):
    begins = [H.shim_range_begin(ngt, P, c) for c in range(P + 1)]
    assert begins[0] == 0 and begins[-1] == ngt
    assert all(a <= b for a, b in zip(begins, begins[1:]))
    assert begins == [ngt * c // P for c in range(P + 1)]            # no 32-bit wrap at the limits
    probe = sorted({0, ngt - 1, ngt // 2, ngt // 3} | {b for b in begins if b < ngt} | {b - 1 for b in begins if b >= 1})
    for g in probe:
        c = H.shim_range_owner(ngt, P, g)
        assert 0 <= c < P and begins[c] <= g < begins[c + 1], (g, c)


def test_owner_needs_more_than_32_bits_at_the_limits():
    """Why range_owner is 64-bit: its numerator passes 2^32 for the last GTiles at the largest sizes."""
    ngt, P = (1 << 22) - 1, 1024
    assert (ngt * P + ngt - 1) >= 1 << 32 > ngt * P


def test_span_check_fires_only_outside_the_range(H):
    ok = lambda f, c, l: bool(H.shim_span_ok(f, c, l))
    assert ok(0, 0, 0) and ok(0, 16, 16) and ok(15, 1, 16) and ok(16, 0, 16)
    assert not ok(16, 1, 16) and not ok(0, 17, 16) and not ok(17, 0, 16)
    assert not ok((1 << 64) - 1, 2, 1 << 40)                          # first + count would wrap
    assert H.shim_check_code(3) == -1003 and H.shim_check_code(0) == -1000
