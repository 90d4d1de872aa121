#!/usr/bin/env python
"""Benchmark of the integer-only inference hot path: images/s of a table-driven ResNet run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path (every layer of the table) over one batch of synthetic
images.  `value` is measured with the batch resident in HBM; `e2e` includes the copy of the
step's images from pinned host memory and the read-back of its logits.  Under torchrun every rank
runs the same batch size on its own GPU (independent images, no collective on the data path:
weak scaling); the time is the maximum over ranks.  `--impl reference` times the CPU oracle.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2011_10680_b200 import inputs

WORKLOADS = {
    # name: (depth, mixed, batch, seed)
    "resnet50_int8_b256": (50, False, 256, 3),
    "resnet50_int4_8_mixed_b256": (50, True, 256, 4),
    "resnet18_int8_b8": (18, False, 8, 2),
    # the same ResNet-50 with the residual stream kept in INT32 between blocks, as Fig. 2 draws it (element-wise adds)
    "resnet50_int8_int32stream_b256": (50, False, 256, 3),
    # Inception modules as Appendix E draws them (35x35 and 17x17 module shapes, 4-bit convolution inputs, INT32
    # pooling branch, per-branch DN and concatenation); image 299 / 4 -> 71x71 so that the stem lands on 35x35
    "inception_modules_int4_b256": (0, True, 256, 6),
}


def workload_table(name):
    depth, mixed, batch, seed = WORKLOADS[name]
    if depth == 0:
        return inputs.inception_table(seed, conv_bits=4 if mixed else 8, image_hw=71, width=64, modules35=2, modules17=2)
    return inputs.resnet_table(depth, seed, mixed=mixed, int32_stream="int32stream" in name)
METRIC = "int-only ResNet-50 images/s @bs256; fused conv INT TOPS vs tcgen05 i8 peak"
NOMINAL_I8_TOPS = 4500.0
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
# Figures taken from profiler / measurement runs, kept beside their summaries under profiles/ (small tracked JSON):
# DRAM bytes of the conv launches of one pass (ncu capture at a reduced batch, scaled by images), and the
# MMA-only tcgen05 kind::i8 ceiling measured by `bench.py --mma-peak`.
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "resnet50_int8_conv_dram_traffic.json")
I8_PEAK_JSON = os.path.join(ROOT, "profiles", "mma_peak_kind_i8.json")


def tracked_json(path):
    try:
        return json.load(open(path))
    except (OSError, ValueError):
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return d["hbm_gbs"], d["bf16_tflops_sustained"], "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS * 1400.0 / 1590.0, "fallback"


def layer_work(table, batch):
    """Algorithmic ops and bytes of every layer: what the method itself must move, inputs read once."""
    shapes, bits = table["shapes"], table["bits"]
    hw_in = {-1: (table["image_hw"], table["image_hw"], 3, 8)}
    for i in range(len(table["layers"])):
        hw_in[i] = (*shapes[i], bits[i])
    rows = []
    for i, l in enumerate(table["layers"]):
        h, w, c, b_in = hw_in[l["in0"]]
        ho, wo, co = shapes[i]
        out_bytes = batch * ho * wo * co * l["out_bits"] // 8
        ops = 0
        if l["op"] in ("conv", "linear"):
            k = l["kh"] * l["kw"] * l["cin"]
            m = batch * ho * wo
            ops = 2 * m * co * k
            if l["kh"] == 1 and l["stride"] > 1:
                in_bytes = m * l["cin"] * b_in // 8          # only the sampled pixels
            else:
                in_bytes = batch * h * w * c * b_in // 8
            byt = in_bytes + co * k * l["bits"] // 8 + out_bytes + 13 * co
            if l["in1"] >= 0:
                byt += batch * ho * wo * co * hw_in[l["in1"]][3] // 8
        elif l["op"] == "concat":
            byt = out_bytes + sum(batch * hw_in[t][0] * hw_in[t][1] * hw_in[t][2] * hw_in[t][3] // 8 for t in l["ins"])
        else:
            byt = batch * h * w * c * b_in // 8 + out_bytes
            if l["in1"] >= 0:
                byt += batch * ho * wo * co * hw_in[l["in1"]][3] // 8
        rows.append(dict(layer=i, op=l["op"], ops=ops, bytes=byt))
    return rows


class ClockSampler:
    """nvidia-smi clock / throttle sampling while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax = float(f[1])
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def run_reference(args, rank):
    """The CPU oracle as it stands, on a bounded sample of the same workload per step."""
    if rank != 0:
        return
    from oracle import hqref
    from oracle.network import run_network
    depth, mixed, batch, seed = WORKLOADS[args.workload]
    table = workload_table(args.workload)
    t0 = time.perf_counter()
    run_network(table, inputs.random_images(seed, 1, table["image_hw"]))
    t1 = time.perf_counter() - t0
    total_steps = args.steps + args.warmup
    sample = int(max(1, min(batch, 90.0 / max(t1, 1e-3) / total_steps)))
    images = inputs.random_images(seed, sample, table["image_hw"])
    for _ in range(args.warmup):
        run_network(table, images)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run_network(table, images)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = hqref.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8" if not mixed else "int4/int8", "data": "synthetic",
        "config": {"workload": args.workload, "global_batch": batch, "sample_images_per_step": sample,
                   "note": "CPU oracle (int64, 7-loop conv, OpenMP over rows) on the first images of the batch"},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": cores, "kind": "oracle",
                         "sample": f"{sample} of {batch} images per step"},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Config 5: fused conv/GEMM sweep over the ResNet-50 layer shapes (INT8 and INT4, with and without the
    residual add); per shape device time (CUDA events, L2 flushed between repetitions by writing 256 MB and then reading another 256 MB),
    integer TOPS, achieved GB/s of the algorithmic bytes and the fraction of that shape's own roofline."""
    import torch
    from paper_2011_10680_b200 import binding, build
    build.build()
    hq = binding.Handle(0)
    hbm_peak, bf16_peak, peak_kind = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush_r = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")
    rows = []
    shapes = inputs.SWEEP_LAYERS if args.sweep_only < 0 else [inputs.SWEEP_LAYERS[args.sweep_only]]
    for (hw, cin, cout, k, stride, has_res) in shapes:
        n = max(1, args.sweep_pixels // (hw * hw))
        for bits in (8, 4):
            for residual in ((False, True) if has_res else (False,)):
                case = inputs.conv_case(5, n, hw, hw, cin, cout, k, stride, k // 2, bits=bits, residual=residual)
                dev = binding.upload_case(case)
                out = binding.alloc_out(case["n"], case["ho"], case["wo"], case["cout"], case["out_bits"], case["out_signed"])
                times = []
                for rep in range(args.warmup + args.steps):
                    flush.fill_(rep & 0xFF)
                    flush_r.view(torch.int32).sum()    # then 256 MB read: no backlog of dirty lines charged to the timed kernel
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    st, _ = hq.conv_case(case, dev, out)
                    e1.record()
                    assert st == binding.HQ_OK
                    torch.cuda.synchronize()
                    if rep >= args.warmup:
                        times.append(e0.elapsed_time(e1) * 1e3)
                hq.sync()
                us = float(np.median(times))
                m = n * case["ho"] * case["wo"]
                kk = k * k * cin
                ops = 2 * m * cout * kk
                byt = n * hw * hw * cin * bits // 8 + cout * kk * bits // 8 + m * cout + (m * cout if residual else 0) + 13 * cout
                t_roof = max(ops / (NOMINAL_I8_TOPS * 1e12), byt / (hbm_peak * 1e9)) * 1e6
                rows.append(dict(hw=hw, cin=cin, cout=cout, k=k, batch=n, bits=bits, residual=residual, M=m, N=cout, K=kk,
                                 us=us, best_us=float(min(times)), tops=ops / us / 1e6, gbs=byt / us / 1e3,
                                 frac_of_i8_nominal=ops / us / 1e6 / NOMINAL_I8_TOPS, roofline_us=t_roof,
                                 frac_of_own_roofline=t_roof / us, bound="tensor" if ops / (NOMINAL_I8_TOPS * 1e12) > byt / (hbm_peak * 1e9) else "hbm"))
    if args.layers_out:
        json.dump(rows, open(args.layers_out, "w"), indent=1)
    best = max(rows, key=lambda r: r["tops"])
    print(json.dumps({"metric": "fused conv INT TOPS vs tcgen05 i8 peak (sweep)", "shapes": len(rows),
                      "best_tops": best["tops"], "best_shape": {k: best[k] for k in ("hw", "cin", "cout", "k", "batch", "bits")},
                      "median_frac_of_own_roofline": float(np.median([r["frac_of_own_roofline"] for r in rows])),
                      "hbm_peak": hbm_peak, "peak_kind": f"of {peak_kind}", "i8_nominal_tops": NOMINAL_I8_TOPS,
                      "rows": [{k: (round(v, 3) if isinstance(v, float) else v) for k, v in r.items()} for r in rows]}), flush=True)
    hq.close()


def run_membound(args):
    """The memory-bound kernels on their own, at ResNet-50 batch-256 tensor sizes (each operand larger than L2):
    max pooling, dyadic requantization, the two-branch residual add, the average-pool requantization, and at
    InceptionV3 module sizes the concatenation with per-branch rescale and the INT32 window sums.  Device
    time per call (CUDA events; 256 MB written, then 256 MB read between repetitions), achieved GB/s of the algorithmic bytes
    (every operand read once, the result written once) and its fraction of the measured copy bandwidth."""
    import torch
    from paper_2011_10680_b200 import binding, build
    build.build()
    hq = binding.Handle(0)
    hbm_peak, _, peak_kind = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush_r = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    ri = lambda lo, hi, shape, dt: torch.randint(lo, hi, shape, generator=g, device="cuda", dtype=torch.int32).to(dt)
    u8 = lambda *shape: ri(0, 256, shape, torch.uint8)
    dy = lambda ch, lo, hi: (ri(1 << 30, (1 << 31) - 1, (ch,), torch.int32), ri(lo, hi, (ch,), torch.int32))
    n = args.batch or 256
    cases = []

    x = u8(n, 112, 112, 64); o = torch.empty((n, 56, 56, 64), dtype=torch.uint8, device="cuda")
    cases.append(("maxpool 3x3/2 u8 [%d,112,112,64]" % n, x.numel() + o.numel(),
                  lambda x=x, o=o: hq.maxpool(x, 64, 0, 3, 2, 1, o)))
    ch = 256
    m = u8(n, 56, 56, ch); r = u8(n, 56, 56, ch); o = torch.empty_like(m)
    mb, mc = dy(ch, 30, 33); rb, rc = dy(ch, 30, 33)
    cases.append(("requant u8->u8 [%d,56,56,256]" % n, 2 * m.numel(),
                  lambda m=m, o=o: hq.residual_add(m, 8, 0, mb, mc, None, 0, 0, None, None, ch, 1, 0, 255, o, 8, 0)))
    cases.append(("add u8+u8->u8 [%d,56,56,256]" % n, 3 * m.numel(),
                  lambda m=m, r=r, o=o: hq.residual_add(m, 8, 0, mb, mc, r, 8, 0, rb, rc, ch, 1, 0, 255, o, 8, 0)))
    o4 = torch.empty((n, 56, 56, ch // 2), dtype=torch.uint8, device="cuda")
    cases.append(("requant u8->u4 [%d,56,56,256]" % n, m.numel() + o4.numel(),
                  lambda m=m, o4=o4: hq.residual_add(m, 8, 0, mb, mc, None, 0, 0, None, None, ch, 1, 0, 15, o4, 4, 0)))
    a32 = ri(-(1 << 20), 1 << 20, (n, 56, 56, 64), torch.int32); o32 = torch.empty((n, 56, 56, 64), dtype=torch.uint8, device="cuda")
    b32, c32 = dy(64, 44, 48)
    cases.append(("requant s32->u8 [%d,56,56,64]" % n, 5 * a32.numel(),
                  lambda: hq.residual_add(a32, 32, 1, b32, c32, None, 0, 0, None, None, 64, 1, 0, 255, o32, 8, 0)))
    na = 8 * n
    xa = u8(na, 7, 7, 2048); oa = torch.empty((na, 1, 1, 2048), dtype=torch.uint8, device="cuda")
    ba, ca = dy(2048, 36, 38)
    cases.append(("avgpool requant u8 [%d,7,7,2048]" % na, xa.numel() + oa.numel(),
                  lambda: hq.avgpool_requant(xa, 2048, 8, 0, ba, ca, 0, 255, oa, 8, 0)))
    # Inception concatenation (Appendix E) at the 35x35 module's sizes: three 8-bit convolution branches and the
    # pooling branch in INT32, one dyadic pair per channel, 288 output channels
    cat = [{"x": u8(n, 35, 35, c), "bits": 8, "signed": 0, "ch": c} for c in (64, 64, 96)]
    cat.append({"x": ri(-(1 << 20), 1 << 20, (n, 35, 35, 64), torch.int32), "bits": 32, "signed": 1, "ch": 64})
    for br in cat:
        br["b"], br["c"] = dy(br["ch"], 44, 48) if br["bits"] == 32 else dy(br["ch"], 30, 33)
    ocat = torch.empty((n, 35, 35, 288), dtype=torch.uint8, device="cuda")
    cases.append(("concat 3x u8 + s32 -> u8 [%d,35,35,288]" % n,
                  sum(br["x"].numel() * br["x"].element_size() for br in cat) + ocat.numel(),
                  lambda: hq.concat_requant(cat, 1, 0, 255, ocat, 8, 0)))
    cat17 = [{"x": u8(4 * n, 17, 17, 192), "bits": 8, "signed": 0, "ch": 192} for _ in range(4)]
    for br in cat17:
        br["b"], br["c"] = dy(192, 34, 37)
    ocat17 = torch.empty((4 * n, 17, 17, 768), dtype=torch.uint8, device="cuda")
    cases.append(("concat 4x u8 -> u8 [%d,17,17,768]" % (4 * n), 2 * ocat17.numel(),
                  lambda: hq.concat_requant(cat17, 1, 0, 255, ocat17, 8, 0)))
    # the same two calls with ONE pair per branch, DN(S_i / S_a) of per-tensor activation scales (the form Appendix E
    # writes down; the rows above draw a pair per channel)
    def one_pair(brs):
        res = []
        for br in brs:
            b, c = br["b"], br["c"]
            res.append({**br, "b": b[:1].repeat(br["ch"]).contiguous(), "c": c[:1].repeat(br["ch"]).contiguous()})
        return res
    cat_u, cat17_u = one_pair(cat), one_pair(cat17)
    cases.append(("concat 3x u8 + s32 -> u8 [%d,35,35,288], one pair per branch" % n,
                  sum(br["x"].numel() * br["x"].element_size() for br in cat) + ocat.numel(),
                  lambda: hq.concat_requant(cat_u, 1, 0, 255, ocat, 8, 0)))
    cases.append(("concat 4x u8 -> u8 [%d,17,17,768], one pair per branch" % (4 * n), 2 * ocat17.numel(),
                  lambda: hq.concat_requant(cat17_u, 1, 0, 255, ocat17, 8, 0)))
    # the pooling branch of that module: 3x3 / stride 1 window sums over the INT32 feature map
    xp = ri(-(1 << 20), 1 << 20, (n, 35, 35, 192), torch.int32); op_ = torch.empty_like(xp)
    cases.append(("sumpool 3x3/1 s32 -> s32 [%d,35,35,192]" % n, 2 * xp.numel() * 4,
                  lambda: hq.sumpool(xp, 192, 32, 1, 3, 1, 1, op_)))
    rows = []
    for name, byt, fn in cases:
        times = []
        for rep in range(args.warmup + args.steps):
            flush.fill_(rep & 0xFF)
            flush_r.view(torch.int32).sum()    # then 256 MB read: no backlog of dirty lines charged to the timed kernel
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            st = fn()
            e1.record()
            assert st == binding.HQ_OK, (name, st)
            torch.cuda.synchronize()
            if rep >= args.warmup:
                times.append(e0.elapsed_time(e1) * 1e3)
        us = float(np.median(times))
        # back to back, no flush: every operand is larger than the L2, and each launch pays for the write-back of
        # the output lines the launch before it left behind
        reps = 10
        fn(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record(); torch.cuda.synchronize()
        us_b2b = e0.elapsed_time(e1) * 1e3 / reps
        rows.append(dict(kernel=name, bytes=int(byt), us=round(us, 2), gbs=round(byt / us / 1e3, 1),
                         frac_of_hbm=round(byt / us / 1e3 / hbm_peak, 3), us_back_to_back=round(us_b2b, 2),
                         gbs_back_to_back=round(byt / us_b2b / 1e3, 1), frac_back_to_back=round(byt / us_b2b / 1e3 / hbm_peak, 3)))
    hq.sync()
    print(json.dumps({"metric": "memory-bound kernels, achieved GB/s of algorithmic bytes", "hbm_peak": hbm_peak,
                      "peak_kind": f"of {peak_kind}", "rows": rows}), flush=True)
    hq.close()


def run_sweep_grid(args):
    """Config 5 as a full grid: M in {3136, 12544, 50176, 200704} (= batch x H x W of a ResNet stage), N in
    {64 .. 2048}, K in {64 (1x1, Cin 64), 576 / 1152 / 2304 / 4608 (3x3, Cin 64 / 128 / 256 / 512)}, INT8 and INT4
    operands, epilogue with and without the residual add: 480 points.  Inputs are drawn on the device (timing only;
    parity of these shapes is the tests' job).  Per point: device time, integer TOPS, GB/s of the algorithmic bytes,
    fraction of the point's own roofline."""
    import torch
    from paper_2011_10680_b200 import binding, build
    build.build()
    hq = binding.Handle(0)
    hbm_peak, bf16_peak, peak_kind = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush_r = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    ri = lambda lo, hi, shape, dt: torch.randint(lo, hi, shape, generator=g, device="cuda", dtype=torch.int32).to(dt)
    rows = []
    for (kk, cin, k, hw) in ((64, 64, 1, 56), (576, 64, 3, 56), (1152, 128, 3, 28), (2304, 256, 3, 14), (4608, 512, 3, 7)):
        for m in (3136, 12544, 50176, 200704):
            n = m // (hw * hw)
            for cout in (64, 128, 256, 512, 1024, 2048):
                for bits in (8, 4):
                    for residual in (False, True):
                        per = 8 // bits
                        x = ri(0, 256, (n, hw, hw, cin // per), torch.uint8)
                        w = ri(-128, 128, (cout, k, k, cin // per), torch.int8)
                        bias = ri(-(1 << 15), 1 << 15, (cout,), torch.int32)
                        b = ri(1 << 30, (1 << 31) - 1, (cout,), torch.int32)
                        lo_c = 36 + int(np.log2(kk)) // 2 - (8 if bits == 4 else 0)
                        c = ri(lo_c, lo_c + 4, (cout,), torch.int32)
                        res = ri(0, 256, (n, hw, hw, cout), torch.uint8) if residual else None
                        rb = ri(1 << 30, (1 << 31) - 1, (cout,), torch.int32) if residual else None
                        rc = ri(28, 35, (cout,), torch.int32) if residual else None
                        out = torch.empty((n, hw, hw, cout), dtype=torch.uint8, device="cuda")
                        times = []
                        for rep in range(args.warmup + args.steps):
                            flush.fill_(rep & 0xFF)
                            flush_r.view(torch.int32).sum()    # then 256 MB read: no backlog of dirty lines charged to the timed kernel
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record()
                            st = hq.conv2d(x, bits, 0, cin, w, cout, k, k, 1, k // 2, bias, b, c, out, 8, 0,
                                           res, 8 if residual else 0, 0, rb, rc, 1, 0, 255)
                            e1.record()
                            assert st == binding.HQ_OK, st
                            torch.cuda.synchronize()
                            if rep >= args.warmup:
                                times.append(e0.elapsed_time(e1) * 1e3)
                        us = float(np.median(times))
                        ops = 2 * m * cout * kk
                        byt = m * cin * bits // 8 + cout * kk * bits // 8 + m * cout + (m * cout if residual else 0) + 13 * cout
                        t_ops, t_byt = ops / (NOMINAL_I8_TOPS * 1e12), byt / (hbm_peak * 1e9)
                        rows.append(dict(M=m, N=cout, K=kk, bits=bits, residual=residual, us=round(us, 2), tops=round(ops / us / 1e6, 1),
                                         gbs=round(byt / us / 1e3, 1), frac_of_own_roofline=round(max(t_ops, t_byt) * 1e6 / us, 3),
                                         bound="tensor" if t_ops > t_byt else "hbm"))
                        del x, w, res, out
    hq.sync()
    if args.layers_out:
        json.dump(rows, open(args.layers_out, "w"), indent=1)
    best = max(rows, key=lambda r: r["tops"])
    med = lambda sel: float(np.median([r["frac_of_own_roofline"] for r in rows if sel(r)]))
    big = lambda r: r["M"] == 200704 and r["bits"] == 8
    print(json.dumps({"metric": "fused conv INT TOPS vs tcgen05 i8 peak (sweep grid)", "points": len(rows),
                      "best_tops": best["tops"], "best_point": best,
                      "median_frac_of_own_roofline": {"all": med(lambda r: True),
                                                       "int8_M200704_tensor_bound": med(lambda r: big(r) and r["bound"] == "tensor"),
                                                       "int8_M200704_hbm_bound": med(lambda r: big(r) and r["bound"] == "hbm")},
                      "max_frac_of_i8_nominal": round(best["tops"] / NOMINAL_I8_TOPS, 3),
                      "hbm_peak": hbm_peak, "peak_kind": f"of {peak_kind}", "i8_nominal_tops": NOMINAL_I8_TOPS}), flush=True)
    hq.close()


def run_mma_peak(args):
    """The MMA-only ceiling of tcgen05 kind::i8 on this GPU (hq_mma_peak_launch): every SM issues 128 x 256 x 32
    instructions back to back from pseudo-random operands resident in shared memory, for at least --min-seconds
    (default 2 s) of device time, with the SM clock sampled meanwhile.  Prints integer POPS (2 per MAC) for the
    whole run and for the best launch."""
    import torch
    from paper_2011_10680_b200 import binding, build
    build.build()
    hq = binding.Handle(0)
    stream = torch.cuda.Stream()
    want_s = args.min_seconds if args.min_seconds > 0 else 2.0
    rounds, blocks = 8, 4096                       # 8 x 4096 blocks of 128 x 256 x 128 B: about 10 ms per launch
    with torch.cuda.stream(stream):
        for _ in range(3):
            hq.mma_peak_launch(rounds, blocks)
        hq.sync()
        sampler = ClockSampler(0)
        sampler.start()
        time.sleep(0.25)
        times, ops_total, total_ms = [], 0, 0.0
        while total_ms < want_s * 1e3:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ops = 0
            for _ in range(10):
                ops += hq.mma_peak_launch(rounds, blocks)
            e1.record(stream)
            e1.synchronize()
            ms = e0.elapsed_time(e1)
            times.append((ms, ops)); total_ms += ms; ops_total += ops
        clocks = sampler.stop()
        hq.sync()
    best_pops = max(o / m for m, o in times) / 1e12          # ops per ms / 1e12 = peta-ops per second
    pops = ops_total / total_ms / 1e12
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    mhz = clocks.get("sm_mhz") or 1965.0
    line = {"metric": "tcgen05.mma kind::i8 MMA-only ceiling", "pops": pops, "best_launch_group_pops": best_pops,
            "seconds": total_ms / 1e3, "launches": 10 * len(times), "nominal_pops": NOMINAL_I8_TOPS / 1e3,
            "frac_of_nominal": pops / (NOMINAL_I8_TOPS / 1e3), "clocks": clocks,
            "mac_per_clk_per_sm_at_median_clock": (ops_total / 2) / (total_ms * 1e-3) / sms / (mhz * 1e6),
            "operands": "pseudo-random bytes resident in shared memory, s8 x u8 -> s32, 128 x 256 x 32 per instruction"}
    if args.layers_out:
        json.dump(line, open(args.layers_out, "w"), indent=1)
    print(json.dumps(line), flush=True)
    hq.close()


def run_ilp(args):
    """Hardware-aware bit-width selection (Section 3.4): per-layer latencies of the INT8 and INT4 forms measured
    on this GPU feed the ILP, together with model size, BOPS and a synthetic sensitivity; every answer is then
    built and timed as a network of its own."""
    import torch
    from paper_2011_10680_b200 import binding, build

    build.build()
    depth, seed = 50, 3
    batch = args.batch or 256
    units = inputs.resnet_choice_units(depth)
    hq = binding.Handle(0)
    images_d = torch.from_numpy(inputs.random_images(seed, batch)).cuda()
    stream = torch.cuda.Stream()

    def measure(conv_bits):
        table = inputs.resnet_table(depth, seed, conv_bits=conv_bits)
        net = binding.Network(hq, table, batch)
        logits = torch.empty(net.logits_shape, dtype=torch.int32, device="cuda")
        with torch.cuda.stream(stream):
            for _ in range(max(args.warmup, 3)):
                assert net.run(images_d, logits) == binding.HQ_OK
            hq.sync()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                net.run(images_d, logits)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            ns = np.zeros(len(table["layers"]))
            for _ in range(3):
                ns += np.array(net.time_layers(images_d, logits), dtype=np.float64)
            hq.sync()
        net.close()
        return table, ns / 3.0, ms

    def per_unit(table, layer_ns):
        q, m, g = np.zeros(units), np.zeros(units), np.zeros(units)
        fixed = 0.0
        for l, ns in zip(table["layers"], layer_ns):
            u = l.get("unit", -1)
            if u is None or u < 0:
                fixed += ns
                continue
            q[u] += ns
            if l["op"] == "conv":
                m[u] += l["params"] * l["bits"] / 8.0
                g[u] += float(l["bits"]) ** 2 * l["macs"]
        return q, m, g, fixed

    t8, ns8, ms8 = measure([8] * units)
    t4, ns4, ms4 = measure([4] * units)
    q8, m8, g8, fixed8 = per_unit(t8, ns8)
    q4, m4, g4, _ = per_unit(t4, ns4)
    lat = np.stack([q4, q8], axis=1).round().astype(np.int64)              # ns per batch, choice 0 = INT4, 1 = INT8
    size = np.stack([m4, m8], axis=1).round().astype(np.int64)             # bytes
    bops = (np.stack([g4, g8], axis=1) / 1e6).round().astype(np.int64)     # mega bit-operations per image
    omega = inputs.synthetic_sensitivity(t8, seed)
    rows = [{"case": "uniform INT8", "bits": "8" * units, "step_ms": ms8, "layer_sum_us": float(ns8.sum() / 1e3)},
            {"case": "uniform INT4 (first and last layer INT8)", "bits": "4" * units, "step_ms": ms4,
             "layer_sum_us": float(ns4.sum() / 1e3)}]

    def span(t, frac):
        lo, hi = int(t.min(axis=1).sum()), int(t.max(axis=1).sum())
        return lo + int(frac * (hi - lo))

    cases = [("size", 0, 0.5), ("size", 0, 0.25), ("bops", 1, 0.5), ("latency", 2, 0.5), ("latency", 2, 0.1),
             ("size+latency", -1, 0.5)]
    for name, which, frac in cases:
        lims = [-1, -1, -1]
        if which >= 0:
            lims[which] = span((size, bops, lat)[which], frac)
        else:
            lims[0], lims[2] = span(size, frac), span(lat, frac)
        t0 = time.time()
        st, choice, obj = binding.ilp_solve(omega, size, bops, lat, *lims)
        solve_s = time.time() - t0
        if st != binding.HQ_OK:
            rows.append({"case": name, "fraction_of_range": frac, "status": binding.status_string(st)})
            continue
        bits = [8 if c else 4 for c in choice]
        table, ns, ms = measure(bits)
        idx = np.arange(units)
        rows.append({"case": f"{name} limit at {frac} of the INT4..INT8 range", "limits": lims, "solve_s": solve_s,
                     "bits": "".join(str(b) for b in bits), "n_int4": int(sum(1 for b in bits if b == 4)), "omega": obj,
                     "size_MB": float(size[idx, choice].sum() / 2 ** 20), "gbops_per_image": float(bops[idx, choice].sum() / 1e3),
                     "predicted_us": float((lat[idx, choice].sum() + fixed8) / 1e3), "layer_sum_us": float(ns.sum() / 1e3),
                     "step_ms": ms})
    print(json.dumps({"metric": "bit-width ILP on measured B200 layer latencies (ResNet-50 block convs)", "batch": batch,
                      "units": units, "latency_ns": lat.tolist(), "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50_int8_b256", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers-out", default=None, help="write the per-layer table (JSON) to this file")
    ap.add_argument("--sweep", action="store_true", help="run the fused conv/GEMM sweep (config 5) instead of the network")
    ap.add_argument("--sweep-grid", action="store_true", help="run the full 480-point M x N x K x bits x residual grid of config 5")
    ap.add_argument("--membound", action="store_true", help="time the memory-bound kernels (pooling, requantization, residual add) on their own")
    ap.add_argument("--ilp", action="store_true", help="measure per-layer INT4/INT8 latencies and solve the bit-width ILP of Section 3.4 for several limits")
    ap.add_argument("--sweep-pixels", type=int, default=200704, help="output pixels per sweep shape (batch is derived)")
    ap.add_argument("--sweep-only", type=int, default=-1, help="run a single sweep shape (index), e.g. for profiling")
    ap.add_argument("--mma-peak", action="store_true", help="measure the MMA-only tcgen05 kind::i8 ceiling (>= --min-seconds, default 2 s)")
    ap.add_argument("--min-seconds", type=float, default=-1.0,
                    help="after the K timed steps, keep repeating K-step blocks until this much device time has passed and report "
                         "the sustained figure beside the K-step one (default 3 s; 0 switches it off)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.mma_peak:
        if rank == 0:
            run_mma_peak(args)
        return
    if args.min_seconds < 0:
        args.min_seconds = 3.0
    if args.sweep_grid:
        if rank == 0:
            run_sweep_grid(args)
        return
    if args.membound:
        if rank == 0:
            run_membound(args)
        return
    if args.ilp:
        if rank == 0:
            run_ilp(args)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2011_10680_b200 import binding, build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    depth, mixed, batch, seed = WORKLOADS[args.workload]
    batch = args.batch or batch
    table = workload_table(args.workload)
    hq = binding.Handle(local_rank)
    net = binding.Network(hq, table, batch)
    images_h = torch.from_numpy(inputs.random_images(seed + 1000 * rank, batch, table["image_hw"])).pin_memory()
    images_d = images_h.cuda()
    logits_d = torch.empty(net.logits_shape, dtype=torch.int32, device="cuda")
    stream = torch.cuda.Stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---------------- device-resident throughput -------------------------------------------
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            assert net.run(images_d, logits_d) == binding.HQ_OK
        hq.sync()
        sampler = ClockSampler(local_rank)
        barrier()
        if rank == 0:
            sampler.start()
            time.sleep(0.25)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            net.run(images_d, logits_d)
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        clocks = sampler.stop() if rank == 0 else None
        hq.sync()

        # ---------------- sustained: K-step blocks back to back for at least --min-seconds -----
        sustained = None
        if args.min_seconds > 0:
            sampler2 = ClockSampler(local_rank)
            barrier()
            if rank == 0:
                sampler2.start()
            blocks_ms, n_blocks = 0.0, 0
            g0 = torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            while True:
                g1 = torch.cuda.Event(enable_timing=True)
                for _ in range(args.steps):
                    net.run(images_d, logits_d)
                g1.record(stream)
                g1.synchronize()
                n_blocks += 1
                blocks_ms = g0.elapsed_time(g1)
                go = torch.tensor([1.0 if blocks_ms < args.min_seconds * 1e3 else 0.0], device="cuda")
                if world > 1:
                    dist.all_reduce(go, op=dist.ReduceOp.MAX)      # every rank runs the same number of blocks
                if float(go[0]) == 0.0:
                    break
            barrier()
            c2 = sampler2.stop() if rank == 0 else None
            sustained = {"seconds": blocks_ms / 1e3, "steps": n_blocks * args.steps,
                         "ms_per_step": blocks_ms / (n_blocks * args.steps), "clocks": c2}
            hq.sync()

        # ---------------- end to end: pinned host images in, logits out, double-buffered ----
        copy_stream, back_stream = torch.cuda.Stream(), torch.cuda.Stream()     # images in, logits out
        img_bufs = [torch.empty_like(images_d) for _ in range(2)]
        log_bufs = [torch.empty_like(logits_d) for _ in range(2)]
        logits_h = [torch.empty(net.logits_shape, dtype=torch.int32).pin_memory() for _ in range(2)]
        ready = [torch.cuda.Event() for _ in range(2)]
        ran = [torch.cuda.Event() for _ in range(2)]
        done = [torch.cuda.Event() for _ in range(2)]

        def e2e_steps(k):
            for i in range(k):
                j = i & 1
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(done[j])              # buffer pair j free again: its logits have left
                    img_bufs[j].copy_(images_h, non_blocking=True)
                    ready[j].record(copy_stream)
                stream.wait_event(ready[j])
                net.run(img_bufs[j], log_bufs[j])
                ran[j].record(stream)
                with torch.cuda.stream(back_stream):             # the read-back does not hold the next step up
                    back_stream.wait_event(ran[j])
                    logits_h[j].copy_(log_bufs[j], non_blocking=True)
                    done[j].record(back_stream)

        e2e_steps(max(args.warmup, 4))
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        e2e_steps(args.steps)
        stream.wait_event(done[0]); stream.wait_event(done[1])      # the timed region ends when the last logits are on the host
        f1.record(stream)
        copy_stream.synchronize(); back_stream.synchronize()
        barrier()
        ms_e2e = f0.elapsed_time(f1)
        hq.sync()
        assert torch.equal(logits_h[0], logits_d.cpu()) and torch.equal(logits_h[1], logits_d.cpu())

        # ---------------- per-layer device times (CUDA events around each layer) -------------
        reps = 3
        layer_ns = np.zeros(len(table["layers"]))
        for _ in range(reps):
            layer_ns += np.array(net.time_layers(images_d, logits_d), dtype=np.float64)
        layer_ns /= reps

    if world > 1:
        t = torch.tensor([ms, ms_e2e, sustained["ms_per_step"] if sustained else 0.0], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, ms_e2e = float(t[0]), float(t[1])
        if sustained:
            sustained["ms_per_step"] = float(t[2])

    if rank == 0:
        hbm_peak, bf16_peak, peak_kind = measured_peaks()
        work = layer_work(table, batch)
        rows, tc_bytes, tc_ops, tc_ns = [], 0, 0, 0.0
        for wk, ns, l in zip(work, layer_ns, table["layers"]):
            # layers that run conv_tc_kernel: every conv / linear with a channel count the tensor maps take (4-bit
            # operands included: widened, or kept one value per byte inside the network) and the 3-channel stem
            # (space-to-depth form; its two helper kernels are part of the layer's time)
            on_tc = l["op"] in ("conv", "linear") and (l["cin"] % 32 == 0 or (l["cin"] == 3 and l["kh"] == 7 and l["stride"] == 2))
            if on_tc:
                tc_bytes += wk["bytes"]; tc_ops += wk["ops"]; tc_ns += ns
            rows.append({**wk, "us": ns / 1e3, "tensor_core": on_tc, "gbs": wk["bytes"] / max(ns, 1),
                         "tops": wk["ops"] / max(ns, 1) / 1e3})
        if args.layers_out:
            json.dump(rows, open(args.layers_out, "w"), indent=1)
        n_conv_tc = sum(1 for r in rows if r["tensor_core"])
        total_ops = sum(r["ops"] for r in rows)
        value = world * batch * args.steps / (ms / 1e3)
        step_ms = ms / args.steps
        # The dominant kernel is conv_tc_kernel (all its launch shapes).  Its time per step is the graph-replay step
        # time times its share of the summed per-layer event times (plain launches with an event pair per layer run
        # slower than the graph, so only their RATIO is used); achieved = its algorithmic bytes per step / that time.
        share = tc_ns / max(layer_ns.sum(), 1)
        conv_ms = step_ms * share
        achieved = tc_bytes / (conv_ms * 1e-3) / 1e9                  # GB/s
        # layer by layer: the time each layer would take at its own roofline (tensor peak or HBM bandwidth)
        i8_meas = tracked_json(I8_PEAK_JSON)
        i8_meas_tops = i8_meas["pops"] * 1e3 if i8_meas else None
        def layerwise_ms(tops):
            return sum(max(r["ops"] / (tops * 1e12), r["bytes"] / (hbm_peak * 1e9)) for r in rows) * 1e3
        lw_nominal = layerwise_ms(NOMINAL_I8_TOPS)
        lw_measured = layerwise_ms(i8_meas_tops) if i8_meas_tops else None
        traffic = tracked_json(TRAFFIC_JSON)
        traffic_per_launch = None
        if traffic and args.workload == "resnet50_int8_b256":
            per_image = (traffic["conv_tc_kernel"]["dram_read_bytes"] + traffic["conv_tc_kernel"]["dram_write_bytes"]) / traffic["batch"]
            traffic_per_launch = per_image * batch / max(n_conv_tc, 1)
        tensor_tops = tc_ops / (conv_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8" if not mixed else "int4/int8", "data": "synthetic",
            "config": {"workload": args.workload + (f" (batch overridden to {batch})" if args.batch else ""),
                       "global_batch": world * batch, "image": f"{table['image_hw']}x{table['image_hw']}x3 uint8",
                       "parallelism": f"dp{world}" if world > 1 else "single",
                       "l2": "activations per step (GBs) exceed the 126 MB L2; no explicit flush",
                       "launch": "CUDA graph replay of the whole layer table"},
            "int_tops": total_ops * args.steps / (ms / 1e3) / 1e12 * world,
            "e2e": {"value": world * batch * args.steps / (ms_e2e / 1e3), "unit": "images/s",
                    "h2d_bytes_per_step": int(images_h.numel()), "d2h_bytes_per_step": int(logits_d.numel() * 4),
                    "note": "pinned host images -> device -> hq_run_network -> logits to pinned host, two buffers"},
            "gpu_launches": net.launch_count() * args.steps,
            "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                         "frac": achieved / hbm_peak,
                         "traffic": traffic_per_launch,
                         "traffic_note": (f"avg DRAM bytes per conv launch: ncu capture at batch {traffic['batch']}, caches left alone "
                                          f"({os.path.basename(TRAFFIC_JSON)}), scaled by images") if traffic_per_launch else None,
                         "algorithmic_bytes_per_launch": tc_bytes / max(n_conv_tc, 1),
                         "peak_kind": f"of {peak_kind}",
                         "kernel": "conv_tc_kernel", "launches_per_step": n_conv_tc,
                         "avg_launch_us": conv_ms * 1e3 / max(n_conv_tc, 1),
                         "kernel_ms_per_step": conv_ms, "share_of_step": share,
                         "how": "algorithmic bytes of the conv launches / (ms_per_step x their share of the per-layer event times)",
                         "algorithmic_bytes_per_step": tc_bytes,
                         "layerwise_frac": lw_nominal / step_ms,
                         "layerwise_roofline_ms": lw_nominal,
                         "layerwise_note": "sum over layers of max(ops / 4.5 POPS nominal, algorithmic bytes / measured HBM) / ms_per_step",
                         "layerwise_frac_measured_i8_peak": (lw_measured / step_ms) if lw_measured else None,
                         "tensor_tops": tensor_tops,
                         "tensor_frac_of_nominal_4500": tensor_tops / NOMINAL_I8_TOPS,
                         "tensor_frac_of_measured_i8_peak": (tensor_tops / i8_meas_tops) if i8_meas_tops else None,
                         "measured_i8_peak_tops": i8_meas_tops,
                         "tensor_frac_of_2x_measured_bf16": tensor_tops / (2 * bf16_peak)},
        }
        if sustained:
            sustained["value"] = world * batch / (sustained["ms_per_step"] / 1e3)
            sustained["unit"] = "images/s"
            mhz = (sustained.get("clocks") or {}).get("sm_mhz")
            sustained["ms_per_step_x_sm_ghz"] = sustained["ms_per_step"] * mhz / 1e3 if mhz else None
            line["sustained"] = sustained
        if world == 1 and not args.no_cpu_baseline:
            from oracle import hqref
            from oracle.network import run_network
            one = inputs.random_images(seed, 1, table["image_hw"])
            t0 = time.perf_counter(); run_network(table, one); t1 = time.perf_counter() - t0
            sample = int(max(1, min(batch, 15.0 / max(t1, 1e-3))))
            imgs = inputs.random_images(seed, sample, table["image_hw"])
            t0 = time.perf_counter(); ref = run_network(table, imgs); dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": sample / dt, "unit": "images/s", "cores": hqref.num_threads(),
                                    "kind": "oracle", "sample": f"first {sample} of {batch} images, one pass"}
        print(json.dumps(line), flush=True)
    net.close()
    hq.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
