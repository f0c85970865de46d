"""Shared helpers of the GPU parity tests (comparison rule and case construction)."""
import numpy as np

TOL = {"f32": 1e-4, "f16": 2e-2}


def check_close(gpu, ref, storage="f32", what=""):
    """The parity bar: |gpu - oracle| <= tol * (1 + |oracle|) element-wise (tol 1e-4 for fp32,
    2e-2 for fp16 storage), plus the scale-aware form max|gpu - oracle| / (rms(oracle) +
    |oracle|) against the same tol, which stays meaningful when activations are tiny."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), what + ": non-finite output"
    tol = TOL[storage]
    err = np.abs(gpu - ref)
    bad = err > tol * (1 + np.abs(ref))
    assert not bad.any(), "%s: %d elements over tolerance, worst %g at %s" % (
        what, bad.sum(), err.max(), np.unravel_index(err.argmax(), err.shape))
    rms = np.sqrt(np.mean(ref ** 2))
    if rms > 0:
        rel = (err / (rms + np.abs(ref))).max()
        assert rel <= tol, "%s: scale-aware error %g > %g" % (what, rel, tol)
    return err.max()
