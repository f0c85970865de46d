"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1909_05073_b200 import binding, synth
from paper_1909_05073_b200 import build as pbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pbuild.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "pconv.h")).read()
    declared = set(re.findall(r"\b(pconv_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_status_strings(lib):
    assert binding.pconv_status_str(0) == "ok"
    for s in range(1, 11):
        assert binding.pconv_status_str(s) not in ("", "unknown status")
    assert binding.pconv_status_str(99) == "unknown status"


def _pack_status(lib, w, pats, stride=1, storage=0, flags=0, null_w=False, null_out=False):
    w = np.ascontiguousarray(w, dtype=np.float32)
    pats = np.ascontiguousarray(pats, dtype=np.uint16)
    out = ctypes.c_void_p()
    bo, bc = ctypes.c_int(-1), ctypes.c_int(-1)
    st = lib.pconv_pack(None if null_w else w.ctypes.data, w.shape[0], w.shape[1],
                        pats.ctypes.data, len(pats), stride, storage, flags, None,
                        None if null_out else ctypes.byref(out), ctypes.byref(bo),
                        ctypes.byref(bc))
    if st == 0:
        lib.pconv_free(out)
    return st, bo.value, bc.value


def test_pack_rejects_bad_arguments_on_the_host(lib):
    w = np.zeros((2, 3, 3, 3), np.float32)
    P = synth.PATTERNS8
    assert _pack_status(lib, w, P, null_w=True)[0] == 1
    assert _pack_status(lib, w, P, null_out=True)[0] == 1
    assert _pack_status(lib, w, P, stride=3)[0] == 2
    assert _pack_status(lib, w, P, storage=7)[0] == 6
    assert _pack_status(lib, w, P, flags=0x40)[0] == 6
    assert _pack_status(lib, w, [0x03A, 0x03A])[0] == 3          # duplicate
    assert _pack_status(lib, w, [0x03B])[0] == 3                 # five bits
    assert _pack_status(lib, w, [0x23A])[0] == 3                 # bit outside the 3x3
    assert _pack_status(lib, w, list(range(17)))[0] == 3         # too many
    bad = w.copy()
    bad[1, 2, 0, 0] = bad[1, 2, 2, 2] = 1.0                      # two opposite corners
    assert _pack_status(lib, bad, P) == (4, 1, 2)
    three = w.copy()
    three[0, 1, 1, 1] = 1.0                                      # legal unless strict
    assert _pack_status(lib, three, P, flags=binding.STRICT4) == (4, 0, 1)
    nan = w.copy()
    nan[1, 0, 1, 1] = np.nan
    assert _pack_status(lib, nan, P) == (5, 1, 0)
    big = w.copy()
    big[0, 2, 1, 1] = 7e4                                        # overflows fp16
    assert _pack_status(lib, big, P, storage=binding.F16) == (5, 0, 2)


def test_forward_rejects_bad_arguments_without_a_device(lib):
    assert lib.pconv_forward(None, None, None, None, 1, 4, 4, 0, None) == 1
    assert lib.pconv_maxpool2x2(None, None, 1, 1, 4, 4, 0, None) == 1
    assert lib.pconv_stats(None, None) == 1
    assert lib.pconv_unpack(None, None) == 1
    lib.pconv_free(None)
    lib.pconv_stack_free(None)
    out = ctypes.c_void_p()
    assert lib.pconv_stack_create(None, None, None, 1, 1, 4, 4, 0, ctypes.byref(out)) == 1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libpconv.so")
    with pytest.raises(RuntimeError, match="only implementation"):
        binding.lib()
