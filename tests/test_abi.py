"""The C-ABI library: it loads, exports every symbol include/spdp.h declares, and rejects bad
arguments on the host.  No kernel is launched here (runs without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2607_21985_b200 import build, spdp
    build.build()
    return spdp.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "spdp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"SPDP_API\s+[\w\s\*]+?\b(spdp_\w+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    from paper_2607_21985_b200 import spdp
    names = _declared()
    assert len(names) >= 14
    assert sorted(spdp.EXPORTS) == names
    for n in names:
        assert getattr(L, n) is not None


def test_only_declared_symbols_are_public():
    import subprocess
    from paper_2607_21985_b200 import spdp
    out = subprocess.run(["nm", "-D", "--defined-only", spdp.LIB_PATH], capture_output=True, text=True, check=True).stdout
    public = sorted(l.split()[-1] for l in out.splitlines() if " T " in l and "spdp" in l.split()[-1])
    assert public == _declared()


def test_status_strings(L):
    from paper_2607_21985_b200 import spdp
    assert spdp.spdp_status_string(0) == "SPDP_OK"
    assert spdp.spdp_status_string(-2) == "SPDP_ERR_UNSUPPORTED_SHAPE"
    assert spdp.spdp_status_string(-6) == "SPDP_ERR_TIMEOUT"
    assert spdp.spdp_status_string(99) == "SPDP_ERR_UNKNOWN"


def test_host_side_argument_checks(L):
    h = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x1000)
    # null pointers and unsupported tile shapes are rejected before any CUDA call
    assert L.spdp_pack_tiled_cbc(None, 256, 16, 16, 256, 16, None, ctypes.byref(h)) == -1
    assert L.spdp_pack_tiled_cbc(fake, 256, 16, 16, 256, 16, None, None) == -1
    assert L.spdp_pack_tiled_cbc(fake, 256, 16, 16, 128, 16, None, ctypes.byref(h)) == -2
    assert L.spdp_pack_tiled_cbc(fake, 256, 16, 16, 256, 32, None, ctypes.byref(h)) == -2
    assert L.spdp_pack_tiled_cbc(fake, 0, 16, 16, 256, 16, None, ctypes.byref(h)) == -2
    assert L.spdp_pack_tiled_cbc(fake, 256, 16, 8, 256, 16, None, ctypes.byref(h)) == -2      # ldw < K
    assert L.spdp_pack_tiled_cbc(ctypes.c_void_p(0x1001), 256, 16, 16, 256, 16, None, ctypes.byref(h)) == -1
    assert h.value is None
    assert L.spdp_free(None) == 0
    assert L.spdp_spmspv(None, fake, 0, 0.0, None, fake, 0, None) == -1
    assert L.spdp_get_info(None, None) == -1
    assert L.spdp_export(None, None, None, None, None) == -1
    assert L.spdp_unpack(None, fake, 16, None) == -1
    assert L.spdp_active_columns(None, fake, 0, 0.0, None, fake, None, None) == -1
    assert L.spdp_last_device_status(None, None) == -1
    assert L.spdp_set_num_ctas(None, 4) == -1
    assert L.spdp_import_tiled_cbc(256, 16, 8, None, None, None, None, 0, ctypes.byref(h)) == -1
    # a pointer that is not a handle (wrong magic) is refused
    buf = ctypes.create_string_buffer(512)
    assert L.spdp_free(ctypes.cast(buf, ctypes.c_void_p)) == -1
    assert L.spdp_spmspv(ctypes.cast(buf, ctypes.c_void_p), fake, 0, 0.0, None, fake, 0, None) == -1


def test_binding_fails_loudly_without_library(monkeypatch):
    from paper_2607_21985_b200 import spdp
    monkeypatch.setattr(spdp, "_lib", None)
    monkeypatch.setattr(spdp, "LIB_PATH", "/nonexistent/libspdp.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        spdp.lib()
