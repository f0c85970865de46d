"""One synthetic layer, a warm-up launch and `reps` timed launches: the small case used for ncu
captures and for the pattern-count sweep
(`python -m paper_1909_05073_b200.profile_case 64 64 56 32 1 0.35 [tiled|generic|simple|auto] [f32|f16] [4|8|12] [split]`;
the ninth argument is the number of patterns in the set: the four designed ones, the canonical
eight, or those plus four arbitrary masks; `split` passes the channel-split workspace, as a layer
stack does)."""
import sys

import numpy as np
import torch

from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import synth


def run(c_in, c_out, h, n, stride, keep, kernel="tiled", storage="f32", n_patterns=8, split=False, reps=3):
    sel = {"tiled": B.KERNEL_TILED, "generic": B.KERNEL_GENERIC_TAPS, "simple": B.KERNEL_SIMPLE,
           "auto": 0}[kernel]
    st = B.F16 if storage == "f16" else B.F32
    spec = synth.LayerSpec("p", c_in, c_out, h, h, stride, keep)
    patterns = {4: synth.SCP4, 8: synth.PATTERNS8, 12: synth.PATTERNS12}[int(n_patterns)]
    w, b, ids = synth.gen_weights(spec, 1, patterns)
    layer = B.Layer(w, patterns, stride, st, b)
    x = torch.from_numpy(synth.gen_input(spec, n, 1)).cuda()
    if st == B.F16:
        x = x.half()
    y = layer.forward(x, kernel=sel, split=split)
    print("plan:", B.pconv_plan(layer.handle, n, h, h, 0, split))
    torch.cuda.synchronize()
    us = []
    for _ in range(int(reps)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        layer.forward(x, kernel=sel, out=y, split=split)
        e1.record()
        torch.cuda.synchronize()
        us.append(e0.elapsed_time(e1) * 1e3)
    flops = 8 * int((ids >= 0).sum()) * n * spec.h_out * spec.w_out
    t = float(np.median(us))
    print("%.1f us  %.2f effective TFLOP/s  (%.1f%% of 74.45)" % (t, flops / t / 1e6,
                                                                flops / t / 1e6 / 0.7445))
    assert B.pconv_device_status(layer.handle)[0] == 0
    return t


if __name__ == "__main__":
    a = sys.argv[1:]
    split = "split" in a
    a = [v for v in a if v != "split"]
    run(int(a[0]), int(a[1]), int(a[2]), int(a[3]), int(a[4]), float(a[5]), *(a[6:9]), split=split)
