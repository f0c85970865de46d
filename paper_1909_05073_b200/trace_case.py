"""Phase timing of one synthetic layer inside the tiled kernel, from the trace build of the library
(`python -m paper_1909_05073_b200.trace_case 512 512 28 1 1 0.3 [f32|f16] [split] [zs=<1|2|4>] [ks=<n>]`):
where a launch spends its time (set-up, first chunk, loop, epilogue, finishing of split tiles) for
CTA (0,0,0) and the latest CTA, and how long a consumer warp waited for chunks.  `zs=` / `ks=`
force the launch plan (warps per unit, channel splits) instead of the library's choice."""
import os
import sys

import torch

from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth


def run(c_in, c_out, h, n, stride, keep, storage="f32", split=False, zs=None, ks=None):
    B.LIB_PATH = pbuild.build(trace=True)
    for key, val in (("PCONV_FORCE_ZS", zs), ("PCONV_FORCE_KS", ks)):
        if val is None:
            os.environ.pop(key, None)
        else:
            os.environ[key] = str(val)
    st = B.F16 if storage == "f16" else B.F32
    spec = synth.LayerSpec("t", c_in, c_out, h, h, stride, keep)
    w, b, _ = synth.gen_weights(spec, 1)
    layer = B.Layer(w, synth.PATTERNS8, stride, st, b)
    x = torch.from_numpy(synth.gen_input(spec, n, 1)).cuda()
    if st == B.F16:
        x = x.half()
    y = None
    for _ in range(3):
        y = layer.forward(x, relu=True, kernel=B.KERNEL_TILED, out=y, split=split)
        torch.cuda.synchronize()
    m = B.pconv_trace_read(layer.handle)
    plan = B.pconv_plan(layer.handle, n, h, h, 0, split)
    us = lambda i: (m[i] - m[0]) / 1e3 if m[i] else float("nan")
    clk = 1.965e3   # SM cycles per microsecond at the maximum clock
    print("plan: %s" % plan)
    print("CTA 0:   set-up %.1f  first chunk %.1f  loop end %.1f  sums issued %.1f  epilogue end %.1f us"
          % (us(1), us(2), us(3), us(4), us(5)))
    print("all CTAs: last start %.1f  last loop end %.1f  last sums issued %.1f  last end %.1f us"
          % (us(8), us(9), us(10), us(7)))
    print("warp 0:  waited %.1f us for chunks, worked %.1f us on %d chunks" % (m[11] / clk, m[12] / clk, m[13]))
    assert B.pconv_device_status(layer.handle)[0] == 0


if __name__ == "__main__":
    a = [v for v in sys.argv[1:] if "=" not in v and v not in ("split", "f32", "f16")]
    kw = dict(v.split("=") for v in sys.argv[1:] if "=" in v)
    run(int(a[0]), int(a[1]), int(a[2]), int(a[3]), int(a[4]), float(a[5]),
        storage="f16" if "f16" in sys.argv else "f32", split="split" in sys.argv,
        zs=kw.get("zs"), ks=kw.get("ks"))
