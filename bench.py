#!/usr/bin/env python
"""Benchmark of the PCONV forward path: the VGG-16 conv stack (13 pattern-sparse 3x3 layers and
the four 2x2 max-pools after conv2/4/7/10, fused into those layers' epilogues) on one 224x224 image
per GPU, fp32.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-configs]
    python bench.py --layer C_IN,C_OUT,H,N,STRIDE,KEEP[,f32|f16[,4|8|12[,split][,rows4|rows8]]]  [--steps K]
    python bench.py --layer cfg5:0          (layer 0 of benchmark configuration 5, at its batch)

A step is one pass of the whole stack over one image (per rank).  `value` is effective TFLOP/s
(2 x surviving multiply-adds of all ranks / device time, inputs resident in HBM); `e2e` is the same
figure through the host entry point (input copied from pinned host memory and the result copied
back inside the timed region).  `configs` holds, for the other four benchmark configurations, the
time, effective TFLOP/s and roofline fraction of every layer.  `--impl reference` times the CPU
oracle on the same workload.  Under torchrun every rank runs its own image (batch sharding, no
collective on the data path).  `--layer` times one layer alone (the small case used for profiler
captures) and prints its launch plan.
"""
import argparse
import json
import os
import re
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1909_05073_b200 import synth  # noqa: E402

CID = 2
METRIC = "pattern-conv effective TFLOP/s (2 x surviving MACs / s), VGG-16 conv stack, batch 1 per GPU"
WORKLOAD = ("config 2: VGG-16 conv stack (13 conv + 4 fused max-pool), 224x224x3, batch 1 per GPU, "
            "fp32, 8 patterns, keep 1.0 (conv1) / 0.3")
# FP32 FMA peak of the part: SMs x 128 lanes x 2 flop x max SM clock (derived; a register-only
# fma.rn.f32x2 loop measured 74.1 TFLOP/s on this machine, see profiles/fp32_peak.md)
ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def hbm_peak_gbs():
    """(GB/s, source): the measured copy bandwidth of this machine's B200s, else the stated fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback (earlier measurement on this pool)"


def recorded_traffic():
    """dram__bytes_read + dram__bytes_write of the conv launches of one bench step, from the
    profiler summary under profiles/ (a line `traffic_bytes_per_step = N`), or None."""
    try:
        text = open(os.path.join(ROOT, "profiles", "bench_vgg16_n1_launch_list.md")).read()
        m = re.search(r"traffic_bytes_per_step\s*=\s*([0-9.eE+]+)", text)
        return float(m.group(1)) if m else None
    except OSError:
        return None


def build_workload():
    cfg = synth.config(CID)
    layers = []
    for li, spec in enumerate(cfg.layers):
        w, b, ids = synth.gen_weights(spec, synth.layer_seed(CID, li), cfg.patterns)
        layers.append((spec, w, b, int((ids >= 0).sum())))
    x = synth.gen_input(cfg.layers[0], 1, synth.layer_seed(CID, 0))
    return cfg, layers, x


def layer_flops(spec, kept, n=1):
    return 2 * 4 * kept * spec.h_out * spec.w_out * n


def layer_bytes(spec, kept, n=1, es=4):
    """Minimal HBM bytes of a layer: input once, output once, 4 values + 2 index bytes per
    surviving kernel, bias."""
    return (es * n * (spec.c_in * spec.h * spec.w + spec.c_out * spec.h_out * spec.w_out)
            + kept * (4 * es + 2) + 4 * spec.c_out)


def layer_roof_us(spec, kept, n, es, hbm_gbs):
    return max(layer_flops(spec, kept, n) / (ALU_PEAK_TFLOPS * 1e12),
               layer_bytes(spec, kept, n, es) / (hbm_gbs * 1e9)) * 1e6


def surviving_flops(layers):
    return sum(layer_flops(s, kept) for s, _, _, kept in layers)


def algorithmic_bytes(layers):
    return sum(layer_bytes(s, kept) for s, _, _, kept in layers)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        clocks, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                clocks.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(clocks) if clocks else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(clocks)}


def run_reference(args):
    """The CPU oracle, as it stands, on the same stack: one image per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg, layers, x = build_workload()
    flops = surviving_flops(layers)

    def step():
        a = x
        for spec, w, b, _ in layers:
            a = oracle.conv3x3(a, w, b, spec.stride, True)
            if spec.pool_after:
                a = oracle.maxpool2x2(a)
        return a

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    val = flops / (ms * 1e-3) / 1e12
    cores = oracle.num_threads()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "images_per_step": 1},
        "ms_per_image": ms,
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": "whole stack (13 conv + 4 pool), 1 image per step, dense "
                                   "direct convolution in fp64"},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def _time_launch(torch, flush, fn, reps):
    """Median device time (us) of fn() over `reps` launches, L2 flushed before each."""
    us = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        us.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(us))


def measure_config(torch, B, flush, cid, batch, reps, hbm_gbs):
    """Every layer of one benchmark configuration, each launch timed alone with CUDA events after
    an L2 flush, as a layer stack launches it (workspace for the channel split, fused pool)."""
    cfg = synth.config(cid, batch)
    half = cfg.storage == "f16"
    st, es = (B.F16, 2) if half else (B.F32, 4)
    tdtype = torch.float16 if half else torch.float32
    rows, layers = [], []
    x_next = None
    for li, spec in enumerate(cfg.layers):
        w, b, ids = synth.gen_weights(spec, synth.layer_seed(cid, li), cfg.patterns)
        kept = int((ids >= 0).sum())
        layer = B.Layer(w, cfg.patterns, spec.stride, st, b, strict4=True)
        layers.append(layer)
        if cfg.chained and x_next is not None:
            x = x_next
        else:
            x = torch.from_numpy(synth.gen_input(spec, cfg.batch, synth.layer_seed(cid, li))).cuda().to(tdtype)
        pool = bool(cfg.chained and spec.pool_after)
        n_, c_, h_, w_ = layer.out_shape(x.shape)
        y = torch.empty((n_, c_, h_ // 2, w_ // 2) if pool else (n_, c_, h_, w_), dtype=tdtype, device="cuda")
        plan = B.pconv_plan(layer.handle, cfg.batch, spec.h, spec.w, 0, True)
        if pool and plan["tensor_path"]:
            # what a stack launches here: the dense tensor-core kernel, then the plain max-pool kernel
            y_full = torch.empty((n_, c_, h_, w_), dtype=tdtype, device="cuda")

            def run(layer=layer, x=x, y=y, y_full=y_full):
                layer.forward(x, relu=True, out=y_full, split=True)
                B.pconv_maxpool2x2(y_full, y)
        else:
            def run(layer=layer, x=x, y=y, pool=pool):
                layer.forward(x, relu=True, out=y, split=True, pool=pool)
        run()                                                          # warm-up (and the chain's data)
        us = _time_launch(torch, flush, run, reps)
        roof = layer_roof_us(spec, kept, cfg.batch, es, hbm_gbs)
        row = {"layer": spec.name, "us": round(us, 2), "roof_us": round(roof, 3),
               "frac": round(roof / us, 4),
               "tflops": round(layer_flops(spec, kept, cfg.batch) / us / 1e6, 3),
               "kernel": "tensor" if plan["tensor_path"] else "tiled"}
        if plan["tensor_path"]:
            # the dense path's own roof: zero-inserted multiply-adds at the measured bf16 tensor peak
            dense = 2.0 * 9 * spec.c_in * spec.c_out * spec.h_out * spec.w_out * cfg.batch
            row["dense_tflops"] = round(dense / us / 1e6, 1)
        if cid == 5:
            s = layer.stats()
            mean = s.kept_kernels / max(s.n_groups, 1)
            row["group_kernels_max_over_mean"] = round(s.max_group_kernels / mean, 4)
        rows.append((row, layer_flops(spec, kept, cfg.batch), roof))
        x_next = y if cfg.chained else None
    status = [B.pconv_device_status(l.handle)[0] for l in layers]
    if any(status):
        raise SystemExit("device reported an abandoned wait in config %d" % cid)
    total_us = sum(r["us"] for r, _, _ in rows)
    stack_us = None
    if cfg.chained:
        s0 = cfg.layers[0]
        stack = B.Stack(layers, [l.pool_after for l in cfg.layers], cfg.batch, s0.h, s0.w, B.RELU)
        xs = torch.from_numpy(synth.gen_input(s0, cfg.batch, synth.layer_seed(cid, 0))).cuda().to(tdtype)
        ys = torch.empty(stack.out_shape, dtype=tdtype, device="cuda")
        stack.forward(xs, ys)
        stack_us = _time_launch(torch, flush, lambda: stack.forward(xs, ys), reps)
        if stack.status()[0]:
            raise SystemExit("device reported an abandoned wait in the stack of config %d" % cid)
        stack.close()
    flops = sum(f for _, f, _ in rows)
    roof = sum(r for _, _, r in rows)
    out = {"workload": "config %d: %s, batch %d, %s" % (cid, cfg.name, cfg.batch, cfg.storage),
           "ms": round(total_us / 1e3, 4), "ms_per_image": round(total_us / 1e3 / cfg.batch, 5),
           "tflops": round(flops / total_us / 1e6, 3), "roof_us": round(roof, 2),
           "frac": round(roof / total_us, 4), "timing": "sum of the layers' launches timed alone",
           "layers": [r for r, _, _ in rows]}
    if stack_us is not None:
        out["stack_ms"] = round(stack_us / 1e3, 4)
        out["stack_tflops"] = round(flops / stack_us / 1e6, 3)
        out["stack_frac"] = round(roof / stack_us, 4)
    for l in layers:
        l.close()
    return out


def run_layer(args):
    """One layer alone: plan, median time, effective TFLOP/s (the case profiler captures use)."""
    import torch
    from paper_1909_05073_b200 import binding as B
    from paper_1909_05073_b200 import build as pbuild
    pbuild.build()
    torch.cuda.set_device(0)
    a = args.layer.split(",")
    split = "split" in a
    kernel = {"rows4": B.ROWS4, "rows8": B.ROWS8}                       # pin the tiled kernel's rows per lane
    kflags = sum(f for k, f in kernel.items() if k in a)
    a = [v for v in a if v != "split" and v not in kernel]
    if a[0].startswith("cfg"):
        cid, li = a[0][3:].split(":")[:2]
        cfg = synth.config(int(cid), int(a[1]) if len(a) > 1 else None)
        spec, n, patterns = cfg.layers[int(li)], cfg.batch, cfg.patterns
        storage = cfg.storage
        seed = synth.layer_seed(int(cid), int(li))
        split = True
    else:
        c_in, c_out, h, n, stride = (int(v) for v in a[:5])
        spec = synth.LayerSpec("layer", c_in, c_out, h, h, stride, float(a[5]))
        storage = a[6] if len(a) > 6 else "f32"
        patterns = {4: synth.SCP4, 8: synth.PATTERNS8, 12: synth.PATTERNS12}[int(a[7]) if len(a) > 7 else 8]
        seed = 1
    half = storage == "f16"
    w, b, ids = synth.gen_weights(spec, seed, patterns)
    kept = int((ids >= 0).sum())
    layer = B.Layer(w, patterns, spec.stride, B.F16 if half else B.F32, b)
    x = torch.from_numpy(synth.gen_input(spec, n, seed)).cuda()
    if half:
        x = x.half()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    y = layer.forward(x, split=split, kernel=kflags)
    for _ in range(max(args.warmup - 1, 0)):
        layer.forward(x, out=y, split=split, kernel=kflags)
    us = _time_launch(torch, flush, lambda: layer.forward(x, out=y, split=split, kernel=kflags), args.steps)
    hbm, src = hbm_peak_gbs()
    roof = layer_roof_us(spec, kept, n, 2 if half else 4, hbm)
    assert B.pconv_device_status(layer.handle)[0] == 0
    print(json.dumps({
        "layer": {"c_in": spec.c_in, "c_out": spec.c_out, "h": spec.h, "w": spec.w, "n": n,
                  "stride": spec.stride, "keep": spec.keep, "storage": storage,
                  "patterns": len(patterns), "kept_kernels": kept, "workspace": split},
        "plan": B.pconv_plan(layer.handle, n, spec.h, spec.w, kflags, split),
        "us": round(us, 2), "tflops": round(layer_flops(spec, kept, n) / us / 1e6, 3),
        "frac_of_alu_peak": round(layer_flops(spec, kept, n) / us / 1e6 / ALU_PEAK_TFLOPS, 4),
        "roof_us": round(roof, 3), "frac": round(roof / us, 4), "hbm_peak": src,
        "l2": "flushed before every timed launch"}))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1909_05073_b200 import binding as B
    from paper_1909_05073_b200 import build as pbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if local == 0:
        pbuild.build()
    if world > 1:
        dist.barrier()
    B.lib()

    cfg, layers, x_np = build_workload()
    flops = surviving_flops(layers)
    conv_layers = [B.Layer(w, cfg.patterns, s.stride, B.F32, b, strict4=True) for s, w, b, _ in layers]
    pools = [s.pool_after for s, _, _, _ in layers]
    spec0 = layers[0][0]
    stack = B.Stack(conv_layers, pools, 1, spec0.h, spec0.w, B.RELU)
    x = torch.from_numpy(x_np).cuda()
    y = torch.empty(stack.out_shape, dtype=torch.float32, device="cuda")
    x_host = torch.from_numpy(x_np).pin_memory()
    y_host = torch.empty(stack.out_shape, dtype=torch.float32).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB of L2

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing -----------------------------------------------------------------
    for _ in range(args.warmup):
        stack.forward(x, y)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    sync_all()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    for e0, e1 in ev:
        flush.zero_()
        e0.record()
        stack.forward(x, y)
        e1.record()
    sync_all()
    ms_total = sum(e0.elapsed_time(e1) for e0, e1 in ev)

    # ---- the same step replayed from a CUDA graph (reported beside the eager figure) ------------
    side = torch.cuda.Stream()
    y_graph = torch.empty_like(y)
    stack.capture(x, y_graph, side)
    with torch.cuda.stream(side):
        for _ in range(args.warmup):
            stack.replay(side)
        side.synchronize()
        gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
        for e0, e1 in gev:
            flush.zero_()
            e0.record(side)
            stack.replay(side)
            e1.record(side)
        side.synchronize()
    graph_ms = sum(e0.elapsed_time(e1) for e0, e1 in gev) / args.steps
    # (not bit-equal: the grouping of the fp32 partial sums varies from launch to launch)
    graph_same = bool(torch.allclose(y_graph, y, rtol=1e-4, atol=1e-6))

    # ---- the same step as chains: runs of layers in one persistent kernel (PCONV_CHAIN) --------
    chain_stack = B.Stack(conv_layers, pools, 1, spec0.h, spec0.w, B.RELU | B.CHAIN)
    y_chain = torch.empty_like(y)
    for _ in range(args.warmup):
        chain_stack.forward(x, y_chain)
    torch.cuda.synchronize()
    cev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(args.steps)]
    for e0, e1 in cev:
        flush.zero_()
        e0.record()
        chain_stack.forward(x, y_chain)
        e1.record()
    torch.cuda.synchronize()
    chain_ms = sum(e0.elapsed_time(e1) for e0, e1 in cev) / args.steps
    chain_same = bool(torch.allclose(y_chain, y, rtol=1e-4, atol=1e-6))
    chain_launches = chain_stack.launches()
    if chain_stack.status()[0]:
        raise SystemExit("device reported an abandoned wait in the chained stack")
    chain_stack.close()

    # ---- per-kernel pass: the dominant kernel's launches timed one by one ------------------------
    acts = []
    a = x
    for layer, pool in zip(conv_layers, pools):
        n_, c_, h_, w_ = layer.out_shape(a.shape)
        o = torch.empty((n_, c_, h_ // 2, w_ // 2) if pool else (n_, c_, h_, w_), dtype=torch.float32,
                        device="cuda")
        acts.append((a, o))
        a = o
    conv_ms = [0.0] * len(conv_layers)
    wss = [layer.workspace(xi.shape) for layer, (xi, _) in zip(conv_layers, acts)]
    for _ in range(args.steps):
        flush.zero_()
        pairs = []
        for layer, (xi, oi), ws, pool in zip(conv_layers, acts, wss, pools):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.pconv_forward(layer.handle, xi, layer.bias, oi, B.RELU | (B.POOL2X2 if pool else 0),
                            workspace=ws)
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        for i, (e0, e1) in enumerate(pairs):
            conv_ms[i] += e0.elapsed_time(e1) / args.steps
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end through the host entry point -------------------------------------------------
    # (on a stream of its own: the host entry point then replays its device part from a graph)
    for _ in range(min(args.warmup, 3)):
        stack.forward_host(x_host, y_host, side)
    sync_all()
    e2e_total = 0.0
    for _ in range(args.steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        stack.forward_host(x_host, y_host, side)   # synchronises its stream before returning
        e2e_total += time.perf_counter() - t0
    sync_all()

    from paper_1909_05073_b200.shard import max_over_ranks
    t = max_over_ranks([ms_total, e2e_total * 1e3], device="cuda")
    ms_step = t[0] / args.steps
    e2e_ms = t[1] / args.steps
    status, where = stack.status()
    if status != 0 or any(B.pconv_device_status(l.handle)[0] for l in conv_layers):
        raise SystemExit("device reported an abandoned wait (%d)" % where)

    if rank == 0:
        import oracle
        hbm_gbs, hbm_src = hbm_peak_gbs()
        t0 = time.perf_counter()
        a_ref = x_np
        for spec, w, b, _ in layers:
            a_ref = oracle.conv3x3(a_ref, w, b, spec.stride, True)
            if spec.pool_after:
                a_ref = oracle.maxpool2x2(a_ref)
        cpu_s = time.perf_counter() - t0
        got = y_host.numpy()
        err = np.abs(got - a_ref)
        parity_ok = bool((err <= 1e-4 * (1 + np.abs(a_ref))).all())
        conv_time_ms = sum(conv_ms)
        roofs = [layer_roof_us(s, kept, 1, 4, hbm_gbs) for s, _, _, kept in layers]
        # The timed region launches nothing but the 13 conv kernels (pools fused), so its duration
        # is theirs, overlap between consecutive launches included; the launches timed one by one
        # (no overlap) are reported beside it.
        achieved = flops / (ms_step * 1e-3) / 1e12
        achieved_alone = flops / (conv_time_ms * 1e-3) / 1e12
        value = world * flops / (ms_step * 1e-3) / 1e12
        out = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "images_per_step": world,
                       "l2": "flushed between timed steps (256 MB write)",
                       "parallelism": "batch sharding, no collective"},
            "ms_per_image": ms_step,
            "surviving_gflop_per_image": flops / 1e9,
            "roofline_time_us_per_image": sum(roofs),
            "clocks": clocks,
            "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "ms_per_step": e2e_ms, "h2d_bytes_per_step": int(x_host.numel() * 4),
                    "d2h_bytes_per_step": int(y_host.numel() * 4)},
            # one launch per conv layer: the four max-pools are fused into the epilogue of the layer before
            "gpu_launches": args.steps * stack.launches(),
            "graph_replay": {"ms_per_step": graph_ms, "value": flops / (graph_ms * 1e-3) / 1e12,
                             "unit": "TFLOP/s", "matches_eager_output": graph_same},
            # not the default: one persistent kernel per run of single-wave layers
            "chained": {"ms_per_step": chain_ms, "value": flops / (chain_ms * 1e-3) / 1e12,
                        "unit": "TFLOP/s", "launches_per_step": chain_launches,
                        "matches_eager_output": chain_same},
            "roofline": {"bound": "alu", "kernel": "tiled_kernel (13 conv launches per step)",
                         "achieved": achieved, "peak": ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                         "frac": achieved / ALU_PEAK_TFLOPS,
                         "peak_source": "148 SMs x 128 FP32 lanes x 2 x 1.965 GHz (derived; "
                                        "no FP32 figure in MEASURED_PEAKS.json; an FFMA2 loop "
                                        "measured 74.1, profiles/fp32_peak.md)",
                         "frac_of_layer_roofs": sum(roofs) / (ms_step * 1e3),
                         "hbm_peak_gbs": hbm_gbs, "hbm_peak_source": hbm_src,
                         "launch_ms_sum": conv_time_ms, "achieved_launches_timed_alone": achieved_alone,
                         # dram__bytes_read + dram__bytes_write of the conv launches of one step,
                         # from the profiler capture summarised in profiles/
                         "traffic": recorded_traffic(),
                         "algorithmic_bytes": algorithmic_bytes(layers),
                         "per_layer_us": [round(m * 1e3, 2) for m in conv_ms],
                         "per_layer_roof_us": [round(r, 3) for r in roofs],
                         "per_layer_frac": [round(r / (m * 1e3), 4) for r, m in zip(roofs, conv_ms)]},
            "cpu_baseline": {"value": flops / cpu_s / 1e12, "unit": "TFLOP/s",
                             "cores": oracle.num_threads(), "kind": "oracle", "seconds": cpu_s,
                             "sample": "whole stack, 1 image (dense direct convolution, fp64)"},
            "parity": {"ok": parity_ok, "max_abs_err": float(err.max())},
        }
        if not args.no_configs and world == 1:
            reps = max(3, min(args.steps, 10))
            stack.close()
            del x, y, y_graph, acts
            out["configs"] = {
                "note": "every layer launched alone (as a stack launches it), CUDA events, L2 flushed "
                        "before each launch, median of %d; frac = max(surviving flop / ALU peak, "
                        "minimal bytes / HBM peak) / time" % reps,
                "config1": measure_config(torch, B, flush, 1, 1, reps, hbm_gbs),
                "config3_n1": measure_config(torch, B, flush, 3, 1, reps, hbm_gbs),
                "config3_n32": measure_config(torch, B, flush, 3, 32, reps, hbm_gbs),
                "config4": measure_config(torch, B, flush, 4, 256, reps, hbm_gbs),
                "config5": measure_config(torch, B, flush, 5, 64, reps, hbm_gbs),
            }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layer", default=None, help="time one layer alone (see the module docstring)")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the per-layer measurement of configurations 1, 3, 4 and 5")
    args = ap.parse_args()
    if args.layer:
        run_layer(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
