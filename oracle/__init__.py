"""CPU oracle for the PCONV forward pass -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline legs may import
this package.  It shares no code with the CUDA library and never imports it.

The arithmetic lives in ``pconv_oracle.c`` (plain C, fp64 accumulation, optional OpenMP over
(image, filter)); this module compiles it with gcc on first use, and adds what is pure data
handling: the fp16-storage reading (round weights and input to fp16 with round-to-nearest-even,
widen back, then run the same fp64 convolution; the result is NOT rounded to fp16) and the
structural invariants of a PCONV weight tensor (every kept kernel has its non-zeros inside one
pattern of the set -- exactly 4 of them in strict mode --, every pruned kernel is all zero;
"Sparse Convolution Pattern" section, and the 2.25x = 9/4 pattern rate of the pattern-count
tables).

Pins: see tests/test_oracle_pins.py.  `project` (the projection that produces PCONV weights from
dense ones; not part of the forward pass) is "parity unpinned": the paper's formulas for it are in
a supplement that is not available; it is the plain fp64 definition of the Euclidean projection,
and only that definition's properties are tested (exhaustive search on tiny tensors, invariants).
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pconv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force=False):
    """Compile the C oracle (gcc -O2 -fopenmp). Idempotent."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                           "-o", tmp, _SRC])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        lib.oracle_conv3x3.argtypes = [fp, fp, fp, fp] + [ctypes.c_int] * 7
        lib.oracle_conv3x3.restype = ctypes.c_int
        lib.oracle_maxpool2x2.argtypes = [fp, fp] + [ctypes.c_int] * 4
        lib.oracle_maxpool2x2.restype = ctypes.c_int
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads():
    """Threads the C oracle uses (OpenMP max threads)."""
    return int(_load().oracle_num_threads())


def _fp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def out_size(h, stride):
    return (h + 2 - 3) // stride + 1


def conv3x3(x, w, bias=None, stride=1, relu=False, storage="f32"):
    """Direct 3x3 cross-correlation (Eq. 1), zero padding 1, over the dense weights.

    x [N,C_in,H,W], w [C_out,C_in,3,3], bias [C_out] or None; returns fp32 [N,C_out,H_out,W_out].
    storage="f16": w and x are first rounded to fp16 (RNE) and widened back; bias stays fp32.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    if storage == "f16":
        x = x.astype(np.float16).astype(np.float32)
        w = w.astype(np.float16).astype(np.float32)
    elif storage != "f32":
        raise ValueError("storage must be 'f32' or 'f16'")
    n, c_in, h, wd = x.shape
    c_out = w.shape[0]
    assert w.shape == (c_out, c_in, 3, 3), (w.shape, x.shape)
    y = np.empty((n, c_out, out_size(h, stride), out_size(wd, stride)), dtype=np.float32)
    b = None
    if bias is not None:
        b = np.ascontiguousarray(bias, dtype=np.float32)
        assert b.shape == (c_out,)
    rc = _load().oracle_conv3x3(_fp(x), _fp(w), _fp(b) if b is not None else None, _fp(y),
                                n, c_in, h, wd, c_out, int(stride), int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_conv3x3 rejected its arguments")
    return y


def maxpool2x2(x):
    """2x2 / stride-2 max-pool, NCHW fp32 (fp16 inputs are widened first; max is exact)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    n, c, h, wd = x.shape
    y = np.empty((n, c, h // 2, wd // 2), dtype=np.float32)
    if _load().oracle_maxpool2x2(_fp(x), _fp(y), n, c, h, wd) != 0:
        raise ValueError("oracle_maxpool2x2 rejected its arguments")
    return y


def classify(w, patterns):
    """Per (filter, channel): -1 if the kernel is all zero, else the lowest pattern id whose
    mask (bit 3u+v) contains the kernel's support; raises if some support fits no pattern."""
    w = np.asarray(w)
    c_out, c_in = w.shape[:2]
    bits = (1 << np.arange(9)).reshape(3, 3)
    support = ((w != 0) * bits).sum(axis=(2, 3)).astype(np.int64)
    ids = np.full((c_out, c_in), -2, dtype=np.int64)
    ids[support == 0] = -1
    for pid in range(len(patterns) - 1, -1, -1):
        fits = (support & ~int(patterns[pid])) == 0
        ids[fits & (support != 0)] = pid
    if (ids == -2).any():
        o, c = np.argwhere(ids == -2)[0]
        raise ValueError("kernel (%d,%d) fits no pattern of the set" % (o, c))
    return ids


def check_invariants(w, patterns, strict4=True):
    """PCONV structure: masks have 4 of 9 bits and are distinct; each kernel is all zero or has
    its support inside one mask (exactly 4 non-zeros when strict4). Returns per-kernel ids."""
    pats = [int(p) for p in patterns]
    assert len(set(pats)) == len(pats), "duplicate pattern"
    for p in pats:
        assert 0 < p < 512 and bin(p).count("1") == 4, "pattern %#x is not 4-of-9" % p
    ids = classify(w, pats)
    if strict4:
        nnz = (np.asarray(w) != 0).sum(axis=(2, 3))
        assert set(np.unique(nnz)) <= {0, 4}, "a kernel has a non-zero count other than 0 or 4"
    return ids


def project(w, patterns, keep):
    """Projection of dense 3x3 kernels onto the PCONV constraint set: the step that turns trained
    weights into pattern- and connectivity-pruned ones (the training section says only that, inside
    an ADMM framework, each kernel is given a pattern or is removed as a whole; its formulas are in
    a supplement that is not available, so this is a reading of that sentence: the Euclidean
    projection, which is what the constrained-variable update of that framework computes --
    parity unpinned beyond the properties tested in tests/test_oracle_pins.py).

    Definition, in fp64: for each kernel the pattern that retains the largest sum of squares
    (lowest pattern id among exact ties); then the k = round(keep * kernels) kernels with the
    largest retained sum survive, together with every kernel that ties exactly with the k-th.
    Where two candidates differ by less than rounding, an implementation that sums in a lower
    precision may legitimately choose the other one; tests allow for that with a relative slack
    on the retained sums and compare exactly where the sums are exact (integer-valued weights).

    w: [c_out, c_in, 3, 3].  Returns (projected weights float32, pattern ids int8 with -1 for
    pruned kernels)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    c_out, c_in = w.shape[:2]
    flat = w.reshape(c_out * c_in, 9)
    n = flat.shape[0]
    sq = flat.astype(np.float64) ** 2
    masks = np.array([[(int(m) >> t) & 1 for t in range(9)] for m in patterns], np.float64)
    scores = masks @ sq.T                               # [pattern, kernel] retained sum of squares
    pid = np.argmax(scores, axis=0)                    # first maximum = lowest id on ties
    best = scores[pid, np.arange(n)]
    k = int(np.floor(keep * n + 0.5))
    k = min(max(k, 0), n)
    if k == 0:
        kept = np.zeros(n, bool)
    else:
        threshold = np.sort(best)[n - k]              # the k-th largest value
        kept = best >= threshold
    out = flat * masks[pid].astype(np.float32) * kept[:, None]
    ids = np.where(kept, pid, -1).astype(np.int8)
    return out.reshape(w.shape).astype(np.float32), ids.reshape(c_out, c_in)


def retained_energy(w, patterns):
    """fp64 sum of squares that each pattern of the set retains of each kernel: [pattern, kernel]
    (the quantity `project` maximises; tests use it to judge choices that differ by rounding)."""
    flat = np.ascontiguousarray(w, dtype=np.float32).reshape(-1, 9).astype(np.float64)
    masks = np.array([[(int(m) >> t) & 1 for t in range(9)] for m in patterns], np.float64)
    return masks @ (flat ** 2).T
