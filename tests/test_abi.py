"""The C-ABI shared library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import build as mcbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(mc_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = mcbuild.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    decl = declared_functions()
    assert "mc_decode_attn" in decl and "mc_kv_layout_create" in decl and len(decl) >= 13
    for name in decl:
        assert hasattr(lib, name), name
    assert set(decl) == set(mc.EXPORTS), set(decl) ^ set(mc.EXPORTS)


def test_host_only_calls_work_without_a_gpu():
    L = mc.lib()
    assert mc.mc_status_string(mc.MC_OK) == "ok"
    assert "workspace" in mc.mc_status_string(mc.MC_ERR_WORKSPACE_TOO_SMALL)
    assert L.mc_workspace_bytes(None) == 0
    h = ctypes.c_void_p()
    assert L.mc_kv_layout_create(None, ctypes.byref(h)) == mc.MC_ERR_INVALID_ARG
    d = mc.LayoutDesc()                      # all zero: rejected before any CUDA call
    assert L.mc_kv_layout_create(ctypes.byref(d), ctypes.byref(h)) == mc.MC_ERR_INVALID_ARG and not h.value
    assert L.mc_kv_layout_destroy(None) == mc.MC_OK
    assert L.mc_decode_attn(None, None, 1.0, None, None, None, 0, None) == mc.MC_ERR_INVALID_ARG


def test_binding_fails_loudly_when_the_library_is_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(mc, "_lib", None)
    monkeypatch.setattr(mc, "_LIB_PATH", str(tmp_path / "nope.so"))
    try:
        mc.lib()
    except RuntimeError as e:
        assert "no fallback" in str(e)
    else:
        raise AssertionError("expected a RuntimeError")
