"""Shared helpers of the GPU parity tests: the comparison rule, and guard bands around device
buffers (the stand-in for a memory checker: an out-of-bounds write of a few elements lands in a
band instead of a neighbouring allocation, and is caught)."""
import numpy as np

TOL = {"f32": 1e-4, "f16": 2e-2}

GUARD_BYTES = 4096          # a multiple of 256, so guarded buffers keep the alignment the ABI asks for
GUARD_FILL = 0xA5


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


class Guarded:
    """A CUDA tensor of `shape` / `dtype` placed between two bands of GUARD_BYTES sentinel bytes.
    `.t` is the tensor to hand to the library; `.check(what)` asserts both bands are untouched."""

    def __init__(self, shape, dtype, fill=None, device="cuda"):
        import torch
        numel = int(np.prod(shape)) if len(shape) else 1
        nbytes = numel * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 255) // 256 * 256
        self.raw = torch.full((padded + 2 * GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device=device)
        self.nbytes = nbytes
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        import torch
        torch.cuda.synchronize()
        lo = self.raw[:GUARD_BYTES]
        hi = self.raw[GUARD_BYTES + self.nbytes:]
        assert bool((lo == GUARD_FILL).all()), "%s: bytes before the buffer were written" % what
        assert bool((hi == GUARD_FILL).all()), "%s: bytes after the buffer were written" % what
