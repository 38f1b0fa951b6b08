"""Host-side checks that need no GPU: the C-ABI library builds, loads, exports every symbol that
include/rudder.h declares, and rejects bad arguments before touching a device."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    from paper_2609_39056_b200 import build
    build.build()
    import paper_2609_39056_b200 as rd
    return rd.lib()


def test_exports_every_declared_symbol(L):
    import paper_2609_39056_b200 as rd
    header = (ROOT / "include" / "rudder.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rudder_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in rudder.h but not exported"
    assert declared == set(rd.EXPORTED)


def test_status_strings(L):
    import paper_2609_39056_b200 as rd
    seen = {rd.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_pack_rejects_bad_arguments_on_host(L):
    import paper_2609_39056_b200 as rd
    out = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: the checks below fail first
    f = L.rudder_pack_weights
    assert f(None, None, 128, 128, rd.W4A8_INT, 64, None, ctypes.byref(out)) == rd.ERR_ARG
    assert f(fake, None, 100, 128, rd.W4A8_INT, 64, None, ctypes.byref(out)) == rd.ERR_SHAPE     # N % 64
    assert f(fake, None, 128, 192, rd.W4A8_INT, 64, None, ctypes.byref(out)) == rd.ERR_SHAPE     # K % 128
    assert f(fake, None, 128, 256, rd.W4A8_INT, 32, None, ctypes.byref(out)) == rd.ERR_SHAPE     # group
    assert f(fake, None, 128, 256, 9, 64, None, ctypes.byref(out)) == rd.ERR_UNSUPPORTED
    assert out.value is None


def test_linear_rejects_null_and_workspace_query(L):
    import paper_2609_39056_b200 as rd
    assert L.rudder_linear(None, None, 0, 1, None, 0, None, None, None, 0, None, 0, None) == rd.ERR_ARG
    assert L.rudder_linear_workspace_bytes(None, 16) == 0
    assert L.rudder_block(None, 1, None, 0, None, 0, None) == rd.ERR_ARG
    assert L.rudder_weight_free(None) == rd.OK


def test_import_rejects_bad_arguments_on_host(L):
    import paper_2609_39056_b200 as rd
    out = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: the checks below fail first
    f = L.rudder_weight_import
    assert f(None, fake, fake, None, 128, 128, rd.W4A8_INT, 64, None, ctypes.byref(out)) == rd.ERR_ARG
    assert f(fake, fake, fake, None, 128, 256, rd.W4A4_NVFP4, 16, None, ctypes.byref(out)) == rd.ERR_ARG   # NVFP4 needs its tensor scale
    assert f(fake, fake, fake, None, 100, 128, rd.W4A8_INT, 64, None, ctypes.byref(out)) == rd.ERR_SHAPE
    assert f(fake, fake, fake, None, 128, 256, rd.W4A8_INT, 32, None, ctypes.byref(out)) == rd.ERR_SHAPE
    assert out.value is None
