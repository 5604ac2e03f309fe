"""CPU checks of the boundary: the library loads, exports every declared symbol, and rejects bad
arguments on the host before anything is launched (no GPU needed for any of this)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cq():
    import paper_2511_19705_b200 as m
    from paper_2511_19705_b200 import build
    build.build()
    m.lib()
    return m


def _declared():
    text = open(os.path.join(ROOT, "include", "cafeq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cafeq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(cq):
    names = _declared()
    assert set(names) == set(cq.EXPORTS)
    L = cq.lib()
    for n in names:
        assert getattr(L, n) is not None
    assert cq.version() >= 100
    assert cq.status_string(0) == "ok" and "singular" in cq.status_string(5)


def test_struct_sizes_match_header_layout(cq):
    # uint32 + 2*int32 + (pad) int64 + 7*int32 -> 56 bytes with natural alignment
    assert ctypes.sizeof(cq.MatrixDesc) == 56
    assert ctypes.sizeof(cq.OptCfg) == 52


def test_workspace_size_and_argument_errors(cq):
    d = cq.make_desc(256, 512, 4, 128, 128)
    n = cq.workspace_size(d)
    assert n > 3 * 256 * 512 * 4
    d2 = cq.make_desc(64, 256, 4, 128, 128, cq.AXIS_IN)
    d1 = cq.make_desc(256, 96, 4, 0, 128, cq.AXIS_OUT)
    assert cq.workspace_size(d1, d2) > cq.workspace_size(d1)
    L = cq.lib()
    nb = ctypes.c_size_t(0)
    bad = cq.make_desc(256, 512, 4, 100, 128)            # group does not divide d_in
    assert L.cafeq_workspace_size(ctypes.byref(bad), None, None, ctypes.byref(nb)) == 1
    bad = cq.make_desc(256, 512, 9, 128, 128)            # bits out of range
    assert L.cafeq_workspace_size(ctypes.byref(bad), None, None, ctypes.byref(nb)) == 1
    bad = cq.make_desc(256, 512, 4, 128, 96)             # block does not tile d_in
    assert L.cafeq_workspace_size(ctypes.byref(bad), None, None, ctypes.byref(nb)) == 1
    bad = cq.make_desc(256, 512, 4, 128, 128)
    bad.struct_size = 12
    assert L.cafeq_workspace_size(ctypes.byref(bad), None, None, ctypes.byref(nb)) == 1
    # null pointers are refused before any launch
    z = ctypes.c_void_p(0)
    assert L.cafeq_rtn(ctypes.byref(d), z, z, z, z, z, ctypes.c_size_t(0), z) == 1
    assert L.cafeq_pack(ctypes.byref(d), z, z, z) == 1
    assert L.cafeq_proxy_loss_fwd_bwd(ctypes.byref(d), z, z, z, z, 0, 0, ctypes.c_float(0), 0, z, z, z, z,
                                      ctypes.c_size_t(0), z) == 1


def test_missing_library_fails_loudly(cq, monkeypatch):
    import paper_2511_19705_b200 as m
    monkeypatch.setattr(m, "_lib", None)
    monkeypatch.setattr(m, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError):
        m.lib()
