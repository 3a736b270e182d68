#!/usr/bin/env python
"""Benchmark of the fused-CNN inference path: MobileNetV2-224, fp16 storage, batch 256 per GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--net v2|v1|seg|fire] [--batch B]

One step = one gi_run of the whole network (layout conversion in, 54 fused ops, layout
conversion out) on a batch of synthetic images.  Prints ONE JSON line on rank 0.

* value        images/s with the input batch already resident in HBM (CUDA events on the run
               stream around each gi_run, L2 flushed by an untimed 256 MiB memset between steps).
* e2e          the same metric through the public call with HOST buffers: every step copies its
               pinned fp16 NHWC images to the device, calls gi_run and copies the logits back, all
               inside the timed region; the copy of the next step runs on a second stream while the
               kernels of the current one execute (paper_1907_01989_b200/pipeline.py).
* roofline     the kernel family with the largest share of the step, from gi_run_timed (one CUDA
               event pair per executed op, same stream): algorithmic bytes / measured time against
               the measured HBM peak (or flops against the tensor peak where that binds).
* cpu_baseline the CPU oracle as it stands on this machine's host cores, on a bounded sample of images.
* batch1       latency of the same network at batch 1, plain launches and CUDA-graph replay.
* sustained    the same step (and the same host-buffer pipeline) repeated back to back for at least 3 s of
               device time, with the SM clock sampled throughout: what the GPU holds under its power cap,
               next to the 20-step burst the headline is.

--gpus N without a torchrun environment starts the N ranks itself (re-executes under torch.distributed.run).

N > 1 runs independent replicas (one process per GPU, the batch is the only sharded axis and
the path has no exchange step): weak scaling, no collective on the data path.
--impl reference times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

NETS = {"v2": ("mobilenet_v2", "MobileNetV2-224"), "v1": ("mobilenet_v1", "MobileNetV1-224"),
        "seg": ("mobilenet_v2_segmentation", "MobileNetV2-513-OS16-seg"), "fire": ("fire_network", "fire-module-network-96")}
PW_MODES = {"auto": 0, "simt": 1, "pair": 2, "lane": 3, "wide": 4, "rule": 5}
XOP_MODES = {"auto": 0, "off": 1, "on": 2, "chain": 3}
# dram__bytes_read.sum + dram__bytes_write.sum over algorithmic bytes, from the ncu captures summarised
# under profiles/ (depthwise: batch 128, 112x112x96, stride 1: 560.3 MB over 616.6 MB; pointwise_tc:
# batch 64, 112x112, 16->96: 119.6 MB over 179.8 MB, the tail of the output still being in L2)
NCU_DRAM_TO_ALGORITHMIC = {"depthwise": 0.909, "pointwise_tc": 0.665}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            p = json.load(fh)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi (read-only query) from before the warm-up on; stop(t0, t1) keeps the
    samples whose timestamp lies inside the timed region [t0, t1] (wall clock, seconds)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        return summarize_clock_rows(self.rows, t0, t1)


def summarize_clock_rows(rows, t0=None, t1=None):
    """rows: (arrival wall time, csv line).  A sample counts if it arrived inside [t0, t1 + 50 ms]."""
    sm, mx, reasons = [], [], set()
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for when, row in rows:
        if t0 is not None and not (t0 <= when <= t1 + 0.05):
            continue
        f = [x.strip() for x in row.split(",")]
        if len(f) < 8:
            continue
        try:
            sm.append(float(f[1]))
            mx.append(float(f[2]))
        except ValueError:
            continue
        for n, v in zip(names, f[4:8]):
            if v.lower().startswith("active"):
                reasons.add(n)
    return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
            "samples": len(sm), "reasons": sorted(reasons)}


def shard_images(rank: int, batch_per_gpu: int):
    """Weak scaling by batch: rank r owns images [r*B, (r+1)*B) of the global batch; no exchange step."""
    return [rank * batch_per_gpu + i for i in range(batch_per_gpu)]


def job_throughput(local_ms: float, images_per_rank: int, steps: int, world: int, dist=None, device=None):
    """Whole-job images/s: all ranks' images over the slowest rank's device time (max over ranks)."""
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    return world * images_per_rank * steps / (total_ms * 1e-3), total_ms


def oracle_images_per_s(spec_fn, budget_s=15.0):
    """Time the CPU oracle on a bounded sample of the workload's images."""
    from oracle import graph as og
    from oracle import ops as oops
    from paper_1907_01989_b200 import workloads as wl
    spec1 = spec_fn(1)
    x1 = wl.make_input(spec1, images=[0])
    t0 = time.perf_counter()
    og.run(spec1, [x1], storage="f16", fused=True)
    t1 = time.perf_counter() - t0
    cores = oops.num_threads()
    n = int(max(1, min(64, budget_s / max(t1, 1e-3) * min(cores, 8) / 4)))
    spec = spec_fn(n)
    x = wl.make_input(spec, images=list(range(n)))
    t0 = time.perf_counter()
    og.run(spec, [x], storage="f16", fused=True)
    dt = time.perf_counter() - t0
    return n / dt, cores, f"{n} images of the workload, evaluated once as one batch of {n} ({dt:.1f} s)", n, dt


def respawn_under_torchrun(n: int) -> int:
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one per GPU) and return their exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def clock_bins(chunks, rows):
    """chunks: (wall start, wall end, device ms, images); rows: the sampler's (arrival time, csv line).  Each chunk gets
    the median SM clock of the samples that arrived while it ran; returns images/s per 100 MHz clock bin."""
    bins = {}
    for w0, w1, ms, images in chunks:
        mhz = []
        for when, row in rows:
            if w0 <= when <= w1:
                try:
                    mhz.append(float(row.split(",")[1]))
                except (ValueError, IndexError):
                    pass
        if not mhz:
            continue
        key = int(statistics.median(mhz) // 100 * 100)
        b = bins.setdefault(key, [0.0, 0])
        b[0] += ms
        b[1] += images
    return {f"{k}-{k + 99} MHz": {"images_per_s": round(v[1] / v[0] * 1e3, 1), "seconds": round(v[0] * 1e-3, 3)}
            for k, v in sorted(bins.items())}


def sustained_leg(torch, stream, run_chunk, images_per_chunk, gpu_index, seconds=3.0):
    """Repeat `run_chunk()` (which enqueues work and returns the device milliseconds it took, synchronised) until
    at least `seconds` of device time have passed; SM clock sampled from before the first chunk."""
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.1)
    chunks, total_ms = [], 0.0
    t0 = time.time()
    while total_ms < seconds * 1e3 and len(chunks) < 100000:
        w0 = time.time()
        ms = run_chunk()
        w1 = time.time()
        chunks.append((w0, w1, ms, images_per_chunk))
        total_ms += ms
    t1 = time.time()
    rows = list(sampler.rows)
    clocks = sampler.stop(t0, t1)
    images = images_per_chunk * len(chunks)
    return {"images_per_s": images / total_ms * 1e3, "device_seconds": round(total_ms * 1e-3, 3), "wall_seconds": round(t1 - t0, 3),
            "steps": None, "sm_mhz_median": clocks["sm_mhz"], "clock_samples": clocks.get("samples"),
            "reasons": clocks["reasons"], "by_sm_clock": clock_bins(chunks, rows)}


def run_reference(args, spec_fn, label):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    sample = ""
    for step in range(args.warmup + args.steps):
        budget = args.budget_s if args.budget_s else max(1.0, 100.0 / (args.warmup + args.steps))
        v, cores, sample, n, dt = oracle_images_per_s(spec_fn, budget_s=budget)
        if step >= args.warmup:
            vals.append((n, dt))
    n_tot, t_tot = sum(n for n, _ in vals), sum(t for _, t in vals)
    value = n_tot / t_tot
    line = {"impl": "reference", "metric": f"{label} fp16 images/s (batch {args.batch})", "value": value,
            "unit": "images/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * t_tot / len(vals), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16", "data": "synthetic",
            "config": {"workload": f"{NETS[args.net][0]}_batch{args.batch}", "note": "CPU oracle on host cores; "
                       "each step is a bounded sample of the workload's images"},
            "cpu_baseline": {"value": value, "unit": "images/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def measure_fp16_peak():
    """Dense fp16 matmul throughput of this GPU, measured the way the bf16 figure of MEASURED_PEAKS.json was:
    torch.matmul 8192^3, best of 10 (burst) and back to back for 4 s (sustained).  A library GEMM as a yardstick
    for the roofline denominators; nothing of the inference path runs here."""
    import torch
    torch.cuda.set_device(0)
    out = {}
    for name, dt in (("fp16", torch.float16), ("bf16", torch.bfloat16)):
        a = torch.randn(8192, 8192, device="cuda", dtype=dt)
        b = torch.randn(8192, 8192, device="cuda", dtype=dt)
        flops = 2 * 8192 ** 3
        for _ in range(3):
            a @ b
        best = 1e9
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            a @ b
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        sampler = ClockSampler(0)
        sampler.start()
        t0 = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 0
        e0.record()
        while time.time() - t0 < 4.0:
            for _ in range(50):
                a @ b
            n += 50
            torch.cuda.synchronize()
        e1.record()
        e1.synchronize()
        t1 = time.time()
        clocks = sampler.stop(t0, t1)
        out[name] = {"tflops_burst": round(flops / best / 1e9, 1), "tflops_sustained": round(n * flops / e0.elapsed_time(e1) / 1e9, 1),
                     "sm_mhz_median_sustained": clocks["sm_mhz"], "reasons": clocks["reasons"]}
        time.sleep(2.0)
    print(json.dumps({"fp16_peak": out, "how": "torch.matmul 8192^3: best of 10 (burst); back to back for 4 s (sustained)"}), flush=True)


def run_sweep(args):
    """Single fused operators (1x1 convolution, 3x3 depthwise) with PHWC4 buffers in and out, so
    one kernel runs per call.  Each point is timed with a CUDA event pair per iteration on the run
    stream, the L2 flushed by an untimed memset in between; prints one JSON line per point."""
    import torch
    from paper_1907_01989_b200 import api
    from paper_1907_01989_b200 import workloads as wl
    peaks, peak_kind = load_peaks()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    if args.points:
        points = [tuple(int(v) for v in pt.split(",")) for pt in args.points.split(";") if pt]
    elif args.sweep == "conv3":
        points = [(256, 224, 3, 32, 2), (64, 224, 3, 32, 2), (16, 513, 3, 32, 2), (1, 224, 3, 32, 2)]
    elif args.sweep == "stem":
        points = [(256, 224, 32), (64, 224, 32), (1, 224, 32)]
    elif args.sweep == "dwpw":  # the depthwise -> projection pairs of MobileNetV2 that have at least one tile per SM
        points = [(256, 112, 32, 16, 1), (256, 112, 96, 24, 2), (256, 56, 144, 24, 1), (256, 56, 144, 32, 2), (256, 28, 192, 32, 1),
                  (256, 28, 192, 64, 2), (256, 14, 384, 64, 1), (256, 14, 576, 96, 1)]
    elif args.sweep == "block":  # the inverted-residual blocks of MobileNetV2 on 14x14 and 7x7 planes
        points = [(256, 14, 64, 384, 64, 1), (256, 14, 64, 384, 96, 1), (256, 14, 96, 576, 96, 1), (256, 14, 96, 576, 160, 2),
                  (256, 7, 160, 960, 160, 1), (256, 7, 160, 960, 320, 1)]
    elif args.sweep == "pair":  # the projection -> expansion seams of MobileNetV2 (B, HW, Cin, Cmid, Cout)
        points = [(256, 112, 32, 16, 96), (256, 56, 96, 24, 144), (256, 56, 144, 24, 144), (256, 28, 144, 32, 192),
                  (256, 28, 192, 32, 192), (256, 14, 192, 64, 384), (256, 14, 384, 64, 384), (256, 14, 384, 96, 576),
                  (256, 14, 576, 96, 576), (256, 7, 576, 160, 960), (256, 7, 960, 160, 960)]
    elif args.sweep == "dw":
        points = [(b, hw, c, s) for b in (64, 256) for hw, c in ((112, 32), (112, 96), (56, 144), (28, 192), (14, 384),
                                                                 (14, 576), (7, 960)) for s in (1, 2)]
    else:
        points = [(256, 112, 16, 96), (256, 112, 32, 16), (256, 56, 24, 144), (256, 56, 144, 24), (256, 28, 32, 192),
                  (256, 28, 192, 32), (256, 14, 64, 384), (256, 14, 384, 64), (256, 14, 96, 576), (256, 14, 576, 96),
                  (256, 7, 160, 960), (256, 7, 960, 160), (256, 7, 320, 1280), (256, 14, 576, 576), (256, 14, 960, 960),
                  (256, 14, 1280, 1280), (64, 56, 192, 192), (8, 28, 384, 384), (1, 14, 96, 576)]
    rows = []
    for pt in points:
        in_layout = api.GI_PHWC4
        if args.sweep == "stem":
            b, hw, cout = pt
            spec = wl.single_conv3x3(b, hw, 3, cout, 2)
            name = f"conv3x3 b{b} {hw}x{hw} 3->{cout} s2, NHWC input"
            in_layout = api.GI_NHWC
        elif args.sweep == "conv3":
            b, hw, cin, cout, stride = pt
            spec = wl.single_conv3x3(b, hw, cin, cout, stride)
            name = f"conv3x3 b{b} {hw}x{hw} {cin}->{cout} s{stride}"
        elif args.sweep == "block":
            b, hw, cin, hidden, cout, stride = pt
            spec = wl.inverted_residual_block(b, hw, hw, cin, hidden, cout, stride)
            name = f"block b{b} {hw}x{hw} {cin}->{hidden}->{cout} s{stride}"
        elif args.sweep == "pair":
            b, hw, cin, cmid, cout = pt
            spec = wl.pointwise_pair(b, hw, hw, cin, cmid, cout, residual=args.residual)
            name = f"pw1x1+pw1x1 b{b} {hw}x{hw} {cin}->{cmid}->{cout}"
        elif args.sweep == "dwpw":
            b, hw, c, cout, stride = pt
            spec = wl.depthwise_then_pointwise(b, hw, hw, c, cout, stride, residual=args.residual)
            name = f"dw3x3+pw1x1 b{b} {hw}x{hw} {c}->{cout} s{stride}"
        elif args.sweep == "dw":
            b, hw, c, stride = pt
            spec = wl.single_depthwise(b, hw, c, stride, 1, residual=args.residual)
            name = f"dw3x3 b{b} {hw}x{hw}x{c} s{stride}"
        else:
            b, hw, cin, cout = pt
            spec = wl.single_pointwise(b, hw, cin, cout, residual=args.residual)
            name = f"pw1x1 b{b} {hw}x{hw} {cin}->{cout}"
        g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=in_layout, out_layout=api.GI_PHWC4)
        ex = g.compile(pointwise=PW_MODES[args.pointwise], cross_op=XOP_MODES[args.cross_op])
        ex.bind(dev)
        ops = ex.ops()
        assert len(ops) == {"dwpw": 2, "stem": 2, "block": 3, "pair": 2}.get(args.sweep, 1)
        # seeded images (the workload recipe), at most 8 distinct ones: image k of the batch is drawn image k % 8
        n_img = min(b, 8)
        xs_np = [wl.make_input(spec, images=list(range(n_img)), index=i) for i in range(len(spec.inputs))]

        def to_device(x_np, layout):
            x = torch.from_numpy(x_np).to(dev).half()
            x = x.repeat((b + n_img - 1) // n_img, 1, 1, 1)[:b].contiguous()
            return x if layout == api.GI_NHWC else to_phwc4(x)

        def to_phwc4(x):  # layout only: [B,H,W,C] -> [S][B][plane][4], zero filled
            B_, H_, W_, C_ = x.shape
            S_, P_ = (C_ + 3) // 4, (H_ * W_ + 1) // 2 * 2
            x = torch.nn.functional.pad(x.reshape(B_, H_ * W_, C_), (0, S_ * 4 - C_, 0, P_ - H_ * W_))
            flat = x.reshape(B_, P_, S_, 4).permute(2, 0, 1, 3).contiguous().reshape(-1)
            full = torch.zeros(api.gi_tensor_bytes(B_, H_, W_, C_) // 2, dtype=torch.float16, device=dev)
            full[: flat.numel()] = flat
            return full

        def image_of(raw, t, img):  # one image of a PHWC4 tensor back as [1,H,W,C] fp32 on the host
            H_, W_, C_ = spec.shapes[t]
            S_, P_ = (C_ + 3) // 4, (H_ * W_ + 1) // 2 * 2
            a = raw[: S_ * b * P_ * 4].reshape(S_, b, P_, 4)[:, img, : H_ * W_, :]
            return a.permute(1, 0, 2).reshape(1, H_, W_, S_ * 4)[..., :C_].float().cpu().numpy()

        if args.sweep == "stem":  # the layout conversion must have been taken over by the convolution
            assert [api.KERNEL_NAMES[q.kernel] for q in ops] == ["none", "conv3x3_tc"], "this shape keeps its layout conversion"
        ins = [to_device(x, in_layout) for x in xs_np]
        outs = [torch.full((api.gi_tensor_bytes(b, *spec.shapes[t]) // 2,), float("nan"), dtype=torch.float16, device=dev)
                for t in spec.outputs]
        checked, worst = False, None
        if not args.no_check:
            # what is timed below is first compared with the CPU oracle on sampled images (first and last of the batch)
            from oracle import graph as og
            ex.run(ins, outs, stream)
            torch.cuda.synchronize()
            sel = sorted({0, b - 1})
            ref = og.run(spec, [x[[i % n_img for i in sel]] for x in xs_np], storage="f16", fused=True)
            worst = 0.0
            for t, o in zip(spec.outputs, outs):
                for k, img in enumerate(sel):
                    got, want = image_of(o, t, img), ref[t][k:k + 1]
                    assert np.isfinite(got).all(), f"{name}: non-finite output"
                    worst = max(worst, float((np.abs(got - want) / (1e-2 + 1e-2 * np.abs(want))).max()))
            assert worst <= 1.0, f"{name}: disagrees with the oracle (normalised error {worst:.3f})"
            checked = True
        for _ in range(3):
            ex.run(ins, outs, stream)
        ms = []
        for _ in range(args.iters):
            flush.zero_()
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            ex.run(ins, outs, stream)
            z.record(stream)
            z.synchronize()
            ms.append(a.elapsed_time(z))
        t = statistics.median(ms)

        class o:  # the graph's ops together (one op, or the depthwise + 1x1 pair: two kernels, or one for both)
            bytes = sum(q.bytes for q in ops)
            flops = sum(q.flops for q in ops)
            kernel = "+".join(api.KERNEL_NAMES[q.kernel] for q in ops if api.KERNEL_NAMES[q.kernel] != "none")
        t_hbm = o.bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_tc = o.flops / (peaks["bf16_tflops"] * 1e12) * 1e3
        row = {"op": name, "kernel": o.kernel, "ms": round(t, 5), "bytes": int(o.bytes),
               "flops": int(o.flops), "gbs": round(o.bytes / t / 1e6, 1), "tflops": round(o.flops / t / 1e9, 2),
               "bound": "tensor" if t_tc > t_hbm else "hbm", "frac_of_roofline": round(max(t_hbm, t_tc) / t, 4),
               "peak_source": peak_kind, "checked": checked,
               "max_error_over_tolerance": None if worst is None else round(worst, 4),
               # the operator's tensors would fit in L2 (126 MB), but the untimed flush before each launch evicts
               # them: the inputs of every timed launch come from DRAM, only the output may still sit in L2 at the end
               "smaller_than_l2": bool(o.bytes < 126e6), "inputs_from": "dram (L2 flushed before each timed launch)"}
        rows.append(row)
        print(json.dumps(row), flush=True)
    if args.out:
        with open(args.out, "w") as fh:
            fh.write("# op | kernel | ms | GB/s | TFLOP/s | bound | fraction of roofline (burst peaks, %s)\n" % peak_kind)
            for r in rows:
                fh.write(f"{r['op']} | {r['kernel']} | {r['ms']} | {r['gbs']} | {r['tflops']} | {r['bound']} | "
                         f"{r['frac_of_roofline']}\n")


def run_slice8_sweep(args):
    """The layout comparison (slices of 8 channels against the library's slices of 4) on single 1x1 layers: the same
    seeded layer and images through (a) the library's own kernel choice on PHWC4 tensors, (b) the wide-tile kernel on
    PHWC4 tensors (tiled copy + rearrangement in shared memory), (c) the wide-tile kernel on tensors stored in slices of
    8 channels (gi_slice8_pointwise_run: the tiled copy lands operand rows directly).  Timing and checking as in
    run_sweep: CUDA event pair per launch, L2 flushed before each, sampled images against the oracle."""
    import torch
    from paper_1907_01989_b200 import api
    from paper_1907_01989_b200 import workloads as wl
    from oracle import graph as og
    dev = "cuda:0"
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    points = ([tuple(int(v) for v in pt.split(",")) for pt in args.points.split(";") if pt] if args.points else
              [(256, 14, 512, 512), (256, 14, 1280, 1280), (256, 28, 256, 256), (256, 7, 960, 320)])

    def sliced(x, width, total_halves):  # layout only: [B,H,W,C] -> [S][B][plane][width], zero filled
        B_, H_, W_, C_ = x.shape
        S_, P_ = (C_ + width - 1) // width, (H_ * W_ + 1) // 2 * 2
        x = torch.nn.functional.pad(x.reshape(B_, H_ * W_, C_), (0, S_ * width - C_, 0, P_ - H_ * W_))
        flat = x.reshape(B_, P_, S_, width).permute(2, 0, 1, 3).contiguous().reshape(-1)
        full = torch.zeros(total_halves, dtype=torch.float16, device=dev)
        full[: flat.numel()] = flat
        return full

    def image_of(raw, width, b, hw, c, img):  # one image back as [1,H,W,C] fp32 on the host
        S_, P_ = (c + width - 1) // width, (hw * hw + 1) // 2 * 2
        a = raw[: S_ * b * P_ * width].reshape(S_, b, P_, width)[:, img, : hw * hw, :]
        return a.permute(1, 0, 2).reshape(1, hw, hw, S_ * width)[..., :c].float().cpu().numpy()

    def timed(launch):
        for _ in range(3):
            launch()
        ms = []
        for _ in range(args.iters):
            flush.zero_()
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            launch()
            z.record(stream)
            z.synchronize()
            ms.append(a.elapsed_time(z))
        return statistics.median(ms)

    for b, hw, cin, cout in points:
        spec = wl.single_pointwise(b, hw, cin, cout)
        n_img = min(b, 8)
        x_np = wl.make_input(spec, images=list(range(n_img)))
        x = torch.from_numpy(x_np).to(dev).half().repeat((b + n_img - 1) // n_img, 1, 1, 1)[:b].contiguous()
        sel = sorted({0, b - 1})
        ref = og.run(spec, [x_np[[i % n_img for i in sel]]], storage="f16", fused=True)[spec.outputs[0]]
        flops = 2.0 * b * hw * hw * cin * cout

        def report(layout, kernel, ms, raw, width):
            worst = 0.0
            for k, img in enumerate(sel):
                got, want = image_of(raw, width, b, hw, cout, img), ref[k:k + 1]
                assert np.isfinite(got).all(), f"{layout}: non-finite output"
                worst = max(worst, float((np.abs(got - want) / (1e-2 + 1e-2 * np.abs(want))).max()))
            assert worst <= 1.0, f"{layout}: disagrees with the oracle (normalised error {worst:.3f})"
            print(json.dumps({"op": f"pw1x1 b{b} {hw}x{hw} {cin}->{cout}", "layout": layout, "kernel": kernel, "ms": round(ms, 5),
                              "tflops": round(flops / ms / 1e9, 1), "checked": True, "max_error_over_tolerance": round(worst, 4)}), flush=True)

        for mode in ("auto", "wide"):
            g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4, out_layout=api.GI_PHWC4)
            ex = g.compile(pointwise=PW_MODES[mode])
            ex.bind(dev)
            ins = [sliced(x, 4, api.gi_tensor_bytes(b, hw, hw, cin) // 2)]
            outs = [torch.full((api.gi_tensor_bytes(b, hw, hw, cout) // 2,), float("nan"), dtype=torch.float16, device=dev)]
            ms = timed(lambda: ex.run(ins, outs, stream))
            kernel = "+".join(api.KERNEL_NAMES[q.kernel] for q in ex.ops())
            report("slices of 4 channels, " + ("the library's choice" if mode == "auto" else "wide-tile kernel"), kernel, ms, outs[0], 4)
        conv = [o for o in spec.ops if o.kind == wl.CONV2D][0]
        blob = torch.from_numpy(api.gi_slice8_pointwise_pack(conv.weights.reshape(cout, cin), conv.bias)).to(dev)
        x8 = sliced(x, 8, api.gi_slice8_tensor_bytes(b, hw, hw, cin) // 2)
        out8 = torch.full((api.gi_slice8_tensor_bytes(b, hw, hw, cout) // 2,), float("nan"), dtype=torch.float16, device=dev)
        act = {wl.ACT_NONE: api.GI_ACT_NONE, wl.ACT_RELU: api.GI_ACT_RELU, wl.ACT_RELU6: api.GI_ACT_RELU6}[
            [o for o in spec.ops if o.kind == wl.ACTIVATION][0].act if any(o.kind == wl.ACTIVATION for o in spec.ops) else wl.ACT_NONE]
        ms = timed(lambda: api.gi_slice8_pointwise_run(x8.data_ptr(), out8.data_ptr(), blob.data_ptr(), b, hw, hw, cin, cout, act, stream))
        report("slices of 8 channels, wide-tile kernel", "pointwise_mm", ms, out8, 8)


def run_host_check(args):
    """The multi-rank plumbing without a GPU: rank and world size from the launcher's environment, a gloo group,
    the batch shard of this rank, and the whole-job throughput from the slowest rank's (synthetic) time."""
    import torch.distributed as dist
    from paper_1907_01989_b200 import workloads as wl
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    images = shard_images(rank, 3)
    x = wl.make_input(wl.separable_block(3), images=images)
    value, total_ms = job_throughput(100.0 + 10.0 * rank, 3, 4, world, dist, "cpu")
    gathered = [None] * world
    if world > 1:
        dist.all_gather_object(gathered, (images, float(x.sum())))
    else:
        gathered = [(images, float(x.sum()))]
    if rank == 0:
        print(json.dumps({"host_check": True, "n_gpus": world, "value": value, "total_ms": total_ms, "shards": gathered}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--net", default="v2", choices=sorted(NETS))
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--pointwise", default="auto", choices=["auto", "simt", "pair", "lane", "wide", "rule"])
    ap.add_argument("--cross-op", default="auto", choices=["auto", "off", "on", "chain"],
                    help="cross-operator kernels: the library's choice, none, blocks and depthwise + 1x1 pairs wherever supported, 1x1 -> 1x1 pairs wherever supported")
    ap.add_argument("--per-op", default=None, help="write the per-op timing table to this file")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-batch1", action="store_true", help="skip the batch-1 latency leg (keeps profiler runs short)")
    ap.add_argument("--sweep", default=None, choices=["pw", "dw", "conv3", "dwpw", "stem", "block", "pair", "slice8"],
                    help="time single fused operators instead of a network (slice8: the layout comparison on 1x1 layers, points 'B,HW,Cin,Cout;...')")
    ap.add_argument("--points", default=None, help="sweep points 'B,HW,Cin,Cout;...' (pw), 'B,HW,C,stride;...' (dw), "
                    "'B,HW,Cin,Cout,stride;...' (conv3), 'B,HW,C,Cout,stride;...' (dwpw: depthwise then 1x1, see --cross-op), "
                    "'B,HW,Cout;...' (stem: 3x3 stride-2 convolution of a 3-channel NHWC input, read in that layout), "
                    "'B,HW,Cin,hidden,Cout,stride;...' (block: one inverted-residual block, see --cross-op)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--no-check", action="store_true", help="sweep: skip the comparison of sampled images with the CPU oracle")
    ap.add_argument("--budget-s", type=float, default=None, help="--impl reference: seconds of oracle work per step")
    ap.add_argument("--sustained-s", type=float, default=3.0, help="device seconds of the sustained legs (0: skip them)")
    ap.add_argument("--host-check", action="store_true",
                    help="no GPU work: every rank joins a gloo group, takes its shard of the batch and the ranks reduce a "
                         "synthetic per-rank time with the same max-over-ranks code the timed run uses (tests the N > 1 plumbing)")
    ap.add_argument("--fp16-peak", action="store_true", help="measure the dense fp16 matmul peak (burst and sustained) and exit")
    ap.add_argument("--out", default=None)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.batch is None:
        args.batch = 16 if args.net == "seg" else 256

    if args.fp16_peak:
        measure_fp16_peak()
        return
    if args.sweep == "slice8":
        run_slice8_sweep(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    # started as plain `python bench.py --gpus N`: start the N ranks here (one process per GPU)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_torchrun(args.gpus))
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={os.environ['WORLD_SIZE']}: launch one rank per GPU")
    from paper_1907_01989_b200 import workloads as wl
    fn_name, label = NETS[args.net]
    spec_fn = getattr(wl, fn_name)
    if args.host_check:
        run_host_check(args)
        return
    if args.impl == "reference":
        run_reference(args, spec_fn, label)
        return

    import torch
    import torch.distributed as dist
    from paper_1907_01989_b200 import api
    from paper_1907_01989_b200.pipeline import HostPipeline

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    spec = spec_fn(args.batch)
    graph, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = graph.compile(pointwise=PW_MODES[args.pointwise], cross_op=XOP_MODES[args.cross_op])
    ex.bind(dev)
    ops = ex.ops()
    # ops that run inside another op's kernel, or need no kernel at all, launch nothing
    n_launch = sum(1 for o in ops if api.KERNEL_NAMES[o.kernel] != "none")
    # every rank draws its own images: rank r holds images [r*B, (r+1)*B) of the global batch
    x_host = wl.make_input(spec, images=shard_images(rank, args.batch)).astype(np.float16)
    x_pin = torch.from_numpy(x_host).pin_memory()
    x_dev = x_pin.to(dev, non_blocking=False)
    out_shape = (args.batch,) + tuple(spec.shapes[spec.outputs[0]])
    out_dev = torch.empty(out_shape, dtype=torch.float16, device=dev)
    out_pin = torch.empty(out_shape, dtype=torch.float16).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step_resident():
        ex.run([x_dev], [out_dev], stream)

    # ---- resident-input throughput -------------------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()  # started before the warm-up so that it is sampling when the timed region begins
    # no garbage-collection pause between two launches of a timed step: the host only enqueues work here
    import gc
    gc.collect()
    gc.disable()
    for _ in range(args.warmup):
        flush.zero_()
        step_resident()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    wall0 = time.perf_counter()
    t_region0 = time.time()
    for i in range(args.steps):
        flush.zero_()
        starts[i].record(stream)
        step_resident()
        ends[i].record(stream)
    barrier()
    t_region1 = time.time()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop(t_region0, t_region1) if rank == 0 else None
    ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    value, total_ms = job_throughput(sum(ms), args.batch, args.steps, world, dist, dev)
    ms_per_step = total_ms / args.steps

    # ---- end to end with host buffers ------------------------------------------------------
    # every step copies its images from pinned host memory and reads its logits back; the copy of
    # step i+1 runs on a second stream while the kernels of step i execute (HostPipeline)
    def time_e2e(graphs):
        pipe = HostPipeline(ex, [tuple(x_dev.shape)], [tuple(out_dev.shape)], torch.float16, dev, graphs=graphs)
        if graphs and not pipe.graphs:
            return None
        for _ in range(3):
            pipe.submit([x_pin], [out_pin])
        pipe.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        pipe.copy.wait_event(e0)  # the first timed copy starts after the start event
        for _ in range(args.steps):
            pipe.submit([x_pin], [out_pin])
        e1.record(stream)         # after the last step's kernels and read-back
        pipe.synchronize()
        barrier()
        return job_throughput(e0.elapsed_time(e1), args.batch, args.steps, world, dist, dev)[0]

    # the pipeline's plain launches are the end-to-end number; the same pipeline replaying one CUDA graph per
    # slot (HostPipeline(graphs=True), one launch per batch) is reported next to it
    e2e_value = time_e2e(False)
    e2e_graph_value = time_e2e(True) if world == 1 else None
    logits_checksum = float(out_pin.float().abs().mean())

    # ---- sustained: the same step, and the same host pipeline, for seconds instead of a burst of K steps ----
    sustained = None
    if args.sustained_s > 0:
        chunk = max(1, int(40.0 / max(ms_per_step, 0.05)))  # about 40 ms of device time between synchronisations

        def chunk_back_to_back():
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(chunk):
                step_resident()
            z.record(stream)
            z.synchronize()
            return a.elapsed_time(z)

        def chunk_flushed():
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(chunk)]
            for a, z in ev:
                flush.zero_()
                a.record(stream)
                step_resident()
                z.record(stream)
            ev[-1][1].synchronize()
            return sum(a.elapsed_time(z) for a, z in ev)

        pipe_s = HostPipeline(ex, [tuple(x_dev.shape)], [tuple(out_dev.shape)], torch.float16, dev, graphs=False)
        for _ in range(3):
            pipe_s.submit([x_pin], [out_pin])
        pipe_s.synchronize()

        def chunk_e2e():
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            pipe_s.copy.wait_event(a)
            for _ in range(chunk):
                pipe_s.submit([x_pin], [out_pin])
            z.record(stream)
            pipe_s.synchronize()
            return a.elapsed_time(z)

        barrier()
        sustained = {"protocol": f"steps back to back in chunks of {chunk} (one synchronisation per chunk) until "
                                 f"{args.sustained_s:g} s of device time; SM clock sampled every 20 ms; rank 0's replica",
                     "back_to_back": sustained_leg(torch, stream, chunk_back_to_back, chunk * args.batch, local, args.sustained_s),
                     "l2_flushed_between_steps": sustained_leg(torch, stream, chunk_flushed, chunk * args.batch, local, args.sustained_s),
                     "e2e_host_buffers": sustained_leg(torch, stream, chunk_e2e, chunk * args.batch, local, args.sustained_s)}
        for leg in ("back_to_back", "l2_flushed_between_steps", "e2e_host_buffers"):
            sustained[leg]["steps"] = int(round(sustained[leg]["images_per_s"] * sustained[leg]["device_seconds"] / args.batch))
        barrier()

    # ---- per-op times for the roofline (rank 0) ---------------------------------------------
    line = None
    if rank == 0:
        peaks, peak_kind = load_peaks()
        per_op = np.zeros(len(ops))
        reps = max(3, min(args.steps, 10))
        for _ in range(2):
            ex.run_timed([x_dev], [out_dev], stream)
        for _ in range(reps):
            flush.zero_()
            per_op += np.array(ex.run_timed([x_dev], [out_dev], stream))
        per_op /= reps
        fam = {}
        for o, t in zip(ops, per_op):
            name = api.KERNEL_NAMES[o.kernel]
            if name == "none":  # nothing was launched for this op (it ran inside another op's kernel, or needs none)
                continue
            f = fam.setdefault(name, {"launches": 0, "ms": 0.0, "bytes": 0, "flops": 0, "roof_ms": 0.0})
            f["launches"] += 1
            f["ms"] += float(t)
            f["bytes"] += int(o.bytes)
            f["flops"] += int(o.flops)
            f["roof_ms"] += max(o.bytes / (peaks["hbm_gbs"] * 1e9), o.flops / (peaks["bf16_tflops_sustained"] * 1e12)) * 1e3
        total_op_ms = sum(f["ms"] for f in fam.values())
        kernels = []
        for name, f in sorted(fam.items(), key=lambda kv: -kv[1]["ms"]):
            kernels.append({"kernel": name, "launches": f["launches"], "ms": round(f["ms"], 4),
                            "share": round(f["ms"] / total_op_ms, 4), "gbs": round(f["bytes"] / f["ms"] / 1e6, 1),
                            "tflops": round(f["flops"] / f["ms"] / 1e9, 2),
                            "frac_of_roofline": round(f["roof_ms"] / f["ms"], 4)})
        top_name = kernels[0]["kernel"]
        top = fam[top_name]
        hbm_time = top["bytes"] / (peaks["hbm_gbs"] * 1e9)
        tensor_time = top["flops"] / (peaks["bf16_tflops_sustained"] * 1e12)
        if tensor_time > hbm_time:
            roofline = {"bound": "tensor", "achieved": top["flops"] / top["ms"] / 1e9, "peak": peaks["bf16_tflops_sustained"],
                        "unit": "TFLOP/s"}
        else:
            roofline = {"bound": "hbm", "achieved": top["bytes"] / top["ms"] / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
        # DRAM bytes per launch of the dominant kernel: not measurable here (no profiler in a timed run);
        # scaled from the ncu capture of the same kernel on a smaller case (ratio of dram read + write
        # to algorithmic bytes, see profiles/), which is valid because its traffic grows with the tensor
        ratio = NCU_DRAM_TO_ALGORITHMIC.get(top_name)
        traffic = None if ratio is None else ratio * top["bytes"] / top["launches"]
        # the whole step against the sum of its ops' roofline times: free of the per-launch event overhead below
        step_roof_ms = sum(f["roof_ms"] for f in fam.values())
        roofline["step_frac"] = step_roof_ms / ms_per_step
        roofline["step_roofline_ms"] = round(step_roof_ms, 4)
        roofline["per_kernel_note"] = ("per-kernel times come from gi_run_timed, one event pair per launch: a launch then cannot "
                                       "overlap its predecessor's tail as it does in the timed step, so they sum to "
                                       f"{total_op_ms:.3f} ms against a {ms_per_step:.3f} ms step and the per-kernel fractions "
                                       "are lower bounds; step_frac has neither problem")
        roofline.update({"traffic": traffic, "traffic_source": None if ratio is None else
                         f"ncu capture of a smaller case x {ratio} (dram bytes / algorithmic bytes), mean per launch",
                         "kernel": top_name, "launches_per_step": top["launches"],
                         "bytes_per_step": top["bytes"], "ms_per_step": round(top["ms"], 4), "peak_source": peak_kind,
                         "per_kernel": kernels})
        if args.per_op:
            with open(args.per_op, "w") as fh:
                fh.write("# op kernel in_shape out_shape bytes flops ms GB/s TFLOP/s frac_of_roofline\n")
                for i, (o, t) in enumerate(zip(ops, per_op)):
                    ti = ex.tensor(o.inputs[0]) if o.inputs[0] >= 0 else None
                    to = ex.tensor(o.output) if o.output >= 0 else None
                    roof = max(o.bytes / (peaks["hbm_gbs"] * 1e9), o.flops / (peaks["bf16_tflops_sustained"] * 1e12)) * 1e3
                    fh.write(f"{i} {api.KERNEL_NAMES[o.kernel]} "
                             f"{(ti.h, ti.w, ti.c) if ti else '-'} {(to.h, to.w, to.c) if to else '-'} {o.bytes} {o.flops} "
                             f"{t:.4f} {o.bytes / t / 1e6:.0f} {o.flops / t / 1e9:.1f} {roof / t:.3f}\n".replace(", ", ","))

        # ---- the same step replayed as a CUDA graph (an extra next to the headline, never the headline):
        # same flush and event protocol as the timed region above
        graph_step = None
        if not args.no_batch1:
            side = torch.cuda.Stream()
            try:
                with torch.cuda.stream(side):
                    ex.run([x_dev], [out_dev], side)
                    side.synchronize()
                    cgs = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(cgs, stream=side):
                        ex.run([x_dev], [out_dev], torch.cuda.current_stream())
                    gms = []
                    for i in range(3 + min(args.steps, 20)):
                        flush.zero_()
                        torch.cuda.synchronize()
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record(side)
                        cgs.replay()
                        b.record(side)
                        side.synchronize()
                        if i >= 3:
                            gms.append(a.elapsed_time(b))
                    graph_step = {"ms_per_step": statistics.median(gms), "images_per_s": args.batch / statistics.median(gms) * 1e3,
                                  "protocol": "gi_run captured once, replayed; 3 warm-up replays, median of the next "
                                              f"{len(gms)}, L2 flushed before each"}
            except Exception as exc:
                graph_step = f"capture failed: {type(exc).__name__}"

        # ---- batch-1 latency (the paper's protocol: 10 warm-up runs, mean of the next 100) ----
        b1_ms, graph_ms, b1_launches = None, None, None
        if not args.no_batch1:
            spec1 = spec_fn(1)
            g1, _ = api.graph_from_spec(spec1, api.GI_F16)
            ex1 = g1.compile(pointwise=PW_MODES[args.pointwise], cross_op=XOP_MODES[args.cross_op])
            ex1.bind(dev)
            x1 = torch.from_numpy(wl.make_input(spec1).astype(np.float16)).to(dev)
            o1 = torch.empty((1,) + tuple(spec1.shapes[spec1.outputs[0]]), dtype=torch.float16, device=dev)
            for _ in range(10):
                ex1.run([x1], [o1], stream)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(100):
                ex1.run([x1], [o1], stream)
            b.record(stream)
            torch.cuda.synchronize()
            b1_ms = a.elapsed_time(b) / 100
            side = torch.cuda.Stream()
            try:
                with torch.cuda.stream(side):
                    ex1.run([x1], [o1], side)
                    side.synchronize()
                    cg = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(cg, stream=side):
                        ex1.run([x1], [o1], torch.cuda.current_stream())
                    for _ in range(10):
                        cg.replay()
                    side.synchronize()
                    a.record(side)
                    for _ in range(100):
                        cg.replay()
                    b.record(side)
                    side.synchronize()
                    graph_ms = a.elapsed_time(b) / 100
            except Exception as exc:  # graph capture is an extra, never the headline
                graph_ms = f"capture failed: {type(exc).__name__}"
            b1_launches = sum(1 for o in ex1.ops() if api.KERNEL_NAMES[o.kernel] != "none")

        gc.enable()
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v, cores, sample, _, _ = oracle_images_per_s(spec_fn)
            cpu = {"value": v, "unit": "images/s", "cores": cores, "kind": "oracle", "sample": sample}

        line = {"metric": f"{label} fp16 images/s (batch {args.batch})", "value": value, "unit": "images/s",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
                "config": {"workload": f"{fn_name}_batch{args.batch}", "batch_per_gpu": args.batch,
                           "launches_per_step": n_launch, "arena_mib": round(ex.info.arena_bytes / 2 ** 20, 1),
                           "l2": "flushed between steps by an untimed 256 MiB memset; a step moves ~"
                                 f"{sum(o.bytes for o in ops) / 1e9:.1f} GB", "parallelism": f"replicas x{world}",
                           "pointwise": args.pointwise},
                "roofline": roofline, "cpu_baseline": cpu,
                "e2e": {"value": e2e_value, "unit": "images/s", "with_cuda_graph_per_slot": e2e_graph_value,
                        "h2d_bytes_per_step": int(x_pin.numel() * 2),
                        "d2h_bytes_per_step": int(out_pin.numel() * 2)},
                "gpu_launches": args.steps * n_launch, "clocks": clocks,
                "cuda_graph_step": graph_step, "sustained": sustained,
                "batch1": {"ms": b1_ms, "cuda_graph_ms": graph_ms, "launches": b1_launches,
                           "protocol": "10 warm-up runs, mean of the next 100"},
                "step_ms_min_median_max": [min(ms), statistics.median(ms), max(ms)], "wall_s_timed_region": wall,
                "logits_abs_mean": logits_checksum}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
