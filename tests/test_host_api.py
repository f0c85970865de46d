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


def test_launch_plans_are_well_formed_over_many_shapes(lib):
    """The planner is host arithmetic: for thousands of shapes the chosen geometry must fit the
    hardware (shared memory, ring depth, grid limits) and follow its own rules."""
    rng = np.random.default_rng(2024)
    seen_zs, seen_split = set(), set()
    for _ in range(4000):
        c_in = int(rng.choice([1, 3, 8, 16, 40, 64, 100, 128, 256, 512, 1024, 2048]))
        c_out = int(rng.choice([1, 8, 16, 33, 64, 128, 256, 512, 1000]))
        h = int(rng.choice([1, 2, 4, 7, 8, 14, 16, 28, 32, 56, 112, 224, 300]))
        w = int(rng.choice([1, 2, 3, 4, 7, 8, 14, 15, 16, 28, 32, 56, 112, 224, 333]))
        n = int(rng.choice([1, 1, 2, 8, 32, 256]))
        stride = int(rng.choice([1, 2]))
        storage = int(rng.choice([binding.F32, binding.F16]))
        keep = float(rng.choice([0.05, 0.3, 0.5, 1.0]))
        canonical = bool(rng.random() < 0.7)
        generic = bool(rng.random() < 0.15)
        ws = bool(rng.random() < 0.5)
        kept = int(keep * c_in * c_out)
        flags = binding.KERNEL_GENERIC_TAPS if generic else 0
        rows = int(rng.choice([0, 0, 4, 8])) if (canonical and not generic) else 0
        flags |= {0: 0, 4: binding.ROWS4, 8: binding.ROWS8}[rows]
        p = binding.pconv_plan_shape(c_out, c_in, kept, stride, storage, canonical, n, h, w, flags, ws)
        what = (c_out, c_in, h, w, n, stride, storage, keep, canonical, generic, ws, rows, p)
        assert p["rows_per_lane"] in (4, 8) and (rows == 0 or p["rows_per_lane"] == rows), what
        if not canonical or generic:
            assert p["rows_per_lane"] == 4, what
        if p["rows_per_lane"] == 8:     # eight consumer warps, two per Tensor-Memory lane quadrant
            assert p["warps_per_unit"] in (1, 2), what
            assert p["groups_per_cta"] * p["pixel_sets"] * p["warps_per_unit"] <= 8, what
            if rows == 0:               # the planner's own choice: unsplit plans only
                assert p["warps_per_unit"] == 1 and p["channel_splits"] == 1, what
        assert p["smem_bytes"] <= 227 * 1024, what
        assert p["stages"] >= 1 and p["ctas"] >= 1, what
        assert p["warps_per_unit"] in (1, 2, 4) and p["tile_width"] in (2, 4, 8, 16, 32), what
        n_chunks = (c_in + 7) // 8
        assert 1 <= p["channel_splits"] <= n_chunks, what
        if generic:
            assert p["generic_taps"] == 1 and p["warps_per_unit"] == 1 and p["channel_splits"] == 1, what
        if not ws:
            assert p["channel_splits"] == 1, what
        chunks_per_cta = -(-n_chunks // p["channel_splits"])
        # a ring shallower than the warps sharing a unit is only allowed when no slot is reused
        assert p["stages"] >= min(p["warps_per_unit"], chunks_per_cta) or p["stages"] == chunks_per_cta, what
        assert p["groups_per_cta"] * p["pixel_sets"] * p["warps_per_unit"] <= (8 if generic else 16), what
        seen_zs.add(p["warps_per_unit"])
        seen_split.add(p["channel_splits"] > 1)
    assert seen_zs == {1, 2, 4} and seen_split == {False, True}
