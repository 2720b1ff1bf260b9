"""The C-ABI library loads, exports what include/rglru.h declares, and validates arguments on the host.
No kernel is launched here: every call below fails validation before any CUDA work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2402_19427_b200 import build, binding
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rglru.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rglru_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2402_19427_b200 import binding
    names = declared_symbols()
    assert len(names) >= 9
    for n in names:
        assert getattr(lib, n) is not None, n
    assert sorted(binding.EXPORTED) == names
    assert lib.rglru_abi_version() == 102


def test_status_strings(lib):
    from paper_2402_19427_b200 import binding
    seen = set()
    for code in range(9):
        s = binding.status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert binding.status_string(99) == "unknown status"


def test_workspace_bytes_host_only(lib):
    from paper_2402_19427_b200 import binding as b
    S = lambda *a, **k: b.Shape(*a, **k)
    assert b.workspace_bytes(S(1, 256, 256, 2, b.F32, 8.0, 0), b.OP_PREFILL) >= 256
    assert b.workspace_bytes(S(512, 1, 2560, 10, b.BF16, 8.0, 0), b.OP_DECODE) >= 256
    n = b.workspace_bytes(S(2, 64, 64, 2, b.F32, 8.0, 0), b.OP_BACKWARD)
    assert n >= 256 + 4 * 2 * 64 * 64 * 4
    assert b.workspace_bytes(S(0, 256, 256, 2, b.F32, 8.0, 0), b.OP_PREFILL) == 0       # bad B
    assert b.workspace_bytes(S(1, 256, 250, 4, b.F32, 8.0, 0), b.OP_PREFILL) == 0       # D % H
    assert b.workspace_bytes(S(1, 256, 256, 2, 7, 8.0, 0), b.OP_PREFILL) == 0           # dtype
    assert b.workspace_bytes(S(1, 256, 256, 2, b.F32, 8.0, 0), 9) == 0                  # op
    assert b.workspace_bytes(S(1, 0, 256, 2, b.F32, 8.0, 0), b.OP_DECODE) >= 256        # T ignored for decode


def test_argument_errors_are_return_codes(lib):
    from paper_2402_19427_b200 import binding as b
    good = 0x7F0000001000  # aligned, never dereferenced: validation fails first in every call below
    odd = good + 4
    pp = b.ParamPtrs(good, 0, good, good, good, good, good)
    sh = b.Shape(1, 16, 64, 2, b.F32, 8.0, 0)
    vp = ctypes.c_void_p

    def prefill(shape=sh, params=pp, x=good, h0=None, cs=None, y=good + 0x100000, hT=good, cso=good, ws=good, wsb=1 << 20):
        return lib.rglru_prefill(ctypes.byref(shape) if shape else None, ctypes.byref(params) if params else None,
                                 vp(x) if x else None, h0, cs, vp(y) if y else None, vp(hT) if hT else None,
                                 vp(cso) if cso else None, vp(ws) if ws else None, wsb, None)

    assert prefill(shape=None) == b.ERR_NULL
    assert prefill(params=None) == b.ERR_NULL
    assert prefill(x=None) == b.ERR_NULL
    assert prefill(ws=None) == b.ERR_NULL
    assert prefill(shape=b.Shape(1, 0, 64, 2, b.F32, 8.0, 0)) == b.ERR_SHAPE
    assert prefill(shape=b.Shape(1, 16, 64, 3, b.F32, 8.0, 0)) == b.ERR_SHAPE
    assert prefill(shape=b.Shape(1, 16, 64, 2, b.F32, -1.0, 0)) == b.ERR_SHAPE
    assert prefill(shape=b.Shape(1, 16, 64, 2, 5, 8.0, 0)) == b.ERR_UNSUPPORTED
    assert prefill(shape=b.Shape(1, 16, 4096, 2, b.F32, 8.0, 0)) == b.ERR_UNSUPPORTED   # head width 2048
    assert prefill(x=odd) == b.ERR_ALIGN
    assert prefill(ws=good + 16) == b.ERR_ALIGN
    assert prefill(params=b.ParamPtrs(good, 0, odd, good, good, good, good)) == b.ERR_ALIGN
    assert prefill(params=b.ParamPtrs(good, 0, 0, good, good, good, good)) == b.ERR_NULL
    assert prefill(wsb=16) == b.ERR_WORKSPACE
    assert prefill(y=good) == b.ERR_ALIAS
    assert prefill(y=good + 64) == b.ERR_ALIAS                                            # partial overlap

    rc = lib.rglru_decode_step(ctypes.byref(sh), ctypes.byref(pp), vp(good), None, vp(good), vp(good + 0x10000), vp(good), 1 << 20, None)
    assert rc == b.ERR_NULL
    rc = lib.rglru_decode_step(ctypes.byref(sh), ctypes.byref(pp), vp(good), vp(good), vp(good), vp(good), vp(good), 1 << 20, None)
    assert rc == b.ERR_ALIAS
    args = [vp(good)] * 3 + [None, vp(good)] + [vp(good + 0x100000)] + [vp(good)] * 7
    rc = lib.rglru_backward(ctypes.byref(sh), ctypes.byref(pp), *args, None, vp(good), 16, None)
    assert rc == b.ERR_WORKSPACE
    args[5] = vp(good)
    rc = lib.rglru_backward(ctypes.byref(sh), ctypes.byref(pp), *args, None, vp(good), 1 << 30, None)
    assert rc == b.ERR_ALIAS
    rc = lib.rglru_prefill_host(ctypes.byref(sh), ctypes.byref(pp), vp(good), None, None, vp(good), vp(good), vp(good),
                                vp(good), 16, vp(good), 1 << 20, None)
    assert rc == b.ERR_WORKSPACE
    assert lib.rglru_query_status(None, None) == b.ERR_NULL


def test_binding_fails_loudly_without_library(monkeypatch):
    from paper_2402_19427_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/librglru_b200.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
