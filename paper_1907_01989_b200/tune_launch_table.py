#!/usr/bin/env python
"""Measure every 1x1 kernel variant on every 1x1 shape of the benchmark networks and write the launch table.

The paper picks a launch configuration per operator from measurements on the device (Section 4, "Work Group:
Choosing the Right Size", and its table of optimal work-group sizes).  The counterpart here is the choice between
the three tensor-core 1x1 kernels (pixel-pair, lane-per-pixel, wide-tile); the tile sizes, stage counts and CTA
counts inside a kernel are functions of the shape that each kernel derives itself.  This script needs a B200:

    python -m paper_1907_01989_b200.tune_launch_table [--iters 20]

It times each supported variant of each shape (CUDA events, median; before every launch the L2 is flushed and the
input tensor is then written by a device copy, which leaves it where the producing kernel of a network leaves it: in L2
as far as it fits.  With the input cold instead, the pixel-pair kernel measured 8 % ahead on the expansion layers 24 -> 144,
32 -> 192 and 96 -> 576, where inside MobileNetV2 the lane-per-pixel kernel is 1.8 % of the whole step faster), and writes
  csrc/launch_table.inc                  the table gi_lower.cc consults before its rule (rebuild the library afterwards)
  ../profiles/pointwise_variant_choice.md  the measurements, and where the table and the rule differ
Shapes: the distinct 1x1 layers of MobileNetV1-224, MobileNetV2-224 (batch 256 and 64) and of the 513x513
segmentation network (batch 16).  Only argument marshalling and timing happen here; nothing is computed in Python.

    python -m paper_1907_01989_b200.tune_launch_table --depthwise [--iters 20]

does the same for the staged depthwise 3x3 stencil: for every depthwise layer (dilation 1) of those networks it times
the kernel under a grid of staging sizes - the largest staging buffer and the shared memory of one CTA, which together
decide planes per work item, buffers in flight and CTAs per SM - and writes
  csrc/dw_table.inc                      {batch, H, W, C, stride, buffer KB, CTA KB, ms default, ms best}; 0, 0 = keep the defaults
  ../profiles/depthwise_staging_choice.md
(gi_compile reads GI_DW_BUF_KB / GI_DW_CTA_KB from the environment as an override of the table: that is how the grid is
walked here.  The stencil is timed with a cold input: a table measured with the input left in L2, as for the 1x1 kernels,
was A/B-ed inside the networks and lost - MobileNetV2 batch 256 1.432 against 1.426 ms, MobileNetV1 1.099 against 1.095.)
"""
import argparse
import os
import statistics
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

VARIANTS = [("pair", 2, "pointwise_tc", 4), ("lane", 3, "pointwise_ts", 10), ("wide", 4, "pointwise_mm", 16)]


def shapes_of(spec):
    from paper_1907_01989_b200 import workloads as wl
    out = []
    for op in spec.ops:
        if op.kind == wl.CONV2D and op.kh == 1 and op.stride == (1, 1):
            h, w, cin = spec.shapes[op.inputs[0]]
            out.append((spec.batch, h, w, cin, op.cout))
    return out


def time_graph(torch, api, spec, dev, stream, flush, iters, **compile_kw):
    g, _ids = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
    ex = g.compile(**compile_kw)
    ex.bind(dev)
    b = spec.batch
    ins = [(torch.rand(api.gi_tensor_bytes(b, *spec.shapes[t]) // 2, device=dev) * 2 - 1).half() for t in spec.inputs]
    outs = [torch.empty(api.gi_tensor_bytes(b, *spec.shapes[t]) // 2, dtype=torch.float16, device=dev) for t in spec.outputs]
    for _ in range(3):
        ex.run(ins, outs, stream)
    ms = []
    for _ in range(iters):
        flush.zero_()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ex.run(ins, outs, stream)
        z.record(stream)
        z.synchronize()
        ms.append(a.elapsed_time(z))
    return statistics.median(ms), [api.KERNEL_NAMES[o.kernel] for o in ex.ops()]


def tune_depthwise(args):
    import torch
    from paper_1907_01989_b200 import api
    from paper_1907_01989_b200 import workloads as wl
    dev = "cuda:0"
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    seen, shapes = set(), []
    for spec in (wl.mobilenet_v2(256), wl.mobilenet_v1(256), wl.mobilenet_v2(64), wl.mobilenet_v1(64), wl.mobilenet_v2_segmentation(16)):
        for op in spec.ops:
            if op.kind == wl.DEPTHWISE and op.dilation == (1, 1) and op.stride[0] == op.stride[1]:
                h, w, c = spec.shapes[op.inputs[0]]
                s = (spec.batch, h, w, c, op.stride[0])
                if s not in seen and h == w:
                    seen.add(s)
                    shapes.append(s)
    grid = [(0, 0)] + [(b, c) for b in (64, 48, 36, 24, 16) for c in (110, 75, 56) if (b, c) != (64, 110)]
    rows = []
    for b, h, w, c, stride in shapes:
        spec = wl.single_depthwise(b, h, c, stride, 1)
        times = {}
        for buf_kb, cta_kb in grid:
            for k, v in (("GI_DW_BUF_KB", buf_kb), ("GI_DW_CTA_KB", cta_kb)):
                if v:
                    os.environ[k] = str(v)
                else:
                    os.environ.pop(k, None)
            ms, kernels = time_graph(torch, api, spec, dev, stream, flush, args.iters)
            assert kernels == ["depthwise"], kernels
            times[(buf_kb, cta_kb)] = ms
        os.environ.pop("GI_DW_BUF_KB", None)
        os.environ.pop("GI_DW_CTA_KB", None)
        best = min(times, key=times.get)
        # the defaults stay unless another setting is more than 3 % faster (the event timer resolves about 2 us)
        if times[(0, 0)] <= 1.03 * times[best]:
            best = (0, 0)
        rows.append(((b, h, w, c, stride), times[(0, 0)], best, times[best]))
        print((b, h, w, c, stride), "default", round(times[(0, 0)], 4), "best", best, round(times[best], 4), flush=True)
    with open(os.path.join(HERE, "csrc", "dw_table.inc"), "w") as fh:
        fh.write("// GENERATED by paper_1907_01989_b200/tune_launch_table.py --depthwise on one B200 - do not edit.\n"
                 "// {batch, H, W, channels, stride, largest staging buffer in KB, shared memory of one CTA in KB (0, 0 = the kernel's\n"
                 "//  defaults, 64 and 110), milliseconds with the defaults, milliseconds with this entry}\n")
        for (b, h, w, c, stride), t0, best, t1 in rows:
            fh.write(f"{{{b}, {h}, {w}, {c}, {stride}, {best[0]}, {best[1]}, {t0:.5f}f, {t1:.5f}f}},\n")
    with open(os.path.join(ROOT, "profiles", "depthwise_staging_choice.md"), "w") as fh:
        fh.write("# Staging sizes of the depthwise 3x3 stencil, measured per depthwise layer of the benchmark networks\n\n"
                 "The paper picks a launch configuration per operator from measurements (Section 4, work-group selection); for the\n"
                 "staged stencil the configuration is how much it stages at a time: the largest staging buffer (planes per work\n"
                 "item) and the shared memory of one CTA (buffers in flight, CTAs per SM).  Generated by\n\n"
                 "    python -m paper_1907_01989_b200.tune_launch_table --depthwise\n\n"
                 "(CUDA events, median of %d launches, L2 flushed before each; 14 settings besides the defaults 64 KB / 110 KB; an\n"
                 "entry replaces the defaults only where it is more than 3 %% faster).  The same run writes `csrc/dw_table.inc`, which\n"
                 "`gi_lower.cc` consults.\n\n"
                 "| batch | plane | channels | stride | defaults ms | table entry (buffer KB, CTA KB) | ms | gain |\n|---|---|---|---|---|---|---|---|\n" % args.iters)
        for (b, h, w, c, stride), t0, best, t1 in rows:
            entry = "defaults" if best == (0, 0) else f"{best[0]}, {best[1]}"
            fh.write(f"| {b} | {h}x{w} | {c} | {stride} | {t0:.4f} | {entry} | {t1:.4f} | {100 * (1 - t1 / t0):.0f} % |\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--depthwise", action="store_true", help="tune the staging sizes of the depthwise stencil instead of the 1x1 kernel choice")
    args = ap.parse_args()
    if args.depthwise:
        tune_depthwise(args)
        return
    import torch
    from paper_1907_01989_b200 import api
    from paper_1907_01989_b200 import workloads as wl
    dev = "cuda:0"
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    seen, shapes = set(), []
    for spec in (wl.mobilenet_v2(256), wl.mobilenet_v1(256), wl.mobilenet_v2(64), wl.mobilenet_v1(64), wl.mobilenet_v2_segmentation(16)):
        for s in shapes_of(spec):
            if s not in seen and s[1] * s[2] > 1:  # the classifier behind the pool is a single pixel: the one-wave rule covers it
                seen.add(s)
                shapes.append(s)
    rows = []
    for b, h, w, cin, cout in shapes:
        spec = wl.single_pointwise(b, h, cin, cout) if h == w else None
        if spec is None:
            continue
        times = {}
        for name, mode, kernel, _ in VARIANTS + [("rule", 5, None, 0)]:
            g, _ids = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
            ex = g.compile(pointwise=mode)
            ran = api.KERNEL_NAMES[ex.ops()[0].kernel]
            if kernel is not None and ran != kernel:
                continue  # this variant does not support the shape
            ex.bind(dev)
            ins = [(torch.rand(api.gi_tensor_bytes(b, *spec.shapes[t]) // 2, device=dev) * 2 - 1).half() for t in spec.inputs]
            src = [x.clone() for x in ins]
            outs = [torch.empty(api.gi_tensor_bytes(b, *spec.shapes[t]) // 2, dtype=torch.float16, device=dev) for t in spec.outputs]
            for _ in range(3):
                ex.run(ins, outs, stream)
            ms = []
            for _ in range(args.iters):
                flush.zero_()
                for x, y in zip(ins, src):
                    x.copy_(y)  # the input as its producer leaves it: written last, in L2 as far as it fits
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                ex.run(ins, outs, stream)
                z.record(stream)
                z.synchronize()
                ms.append(a.elapsed_time(z))
            times[name] = (statistics.median(ms), ran)
            del ex, g, ins, outs, src
        rows.append(((b, h, w, cin, cout), times))
        print((b, h, w, cin, cout), {k: round(v[0], 4) for k, v in times.items()}, "rule ->", times["rule"][1], flush=True)

    def pick(t):
        """The table's entry: the rule's own kernel unless another one is more than 3 % faster (the event timer
        resolves about 2 us, so closer calls are ties and a tie must not flip the choice from run to run)."""
        rule_variant = [n for n, _, k, _ in VARIANTS if k == t["rule"][1]][0]
        fastest = min((v[0], k) for k, v in t.items() if k != "rule")
        if t[rule_variant][0] <= 1.03 * fastest[0]:
            return (t[rule_variant][0], rule_variant)
        return fastest

    kid = {v[2]: v[3] for v in VARIANTS}
    with open(os.path.join(HERE, "csrc", "launch_table.inc"), "w") as fh:
        fh.write("// GENERATED by paper_1907_01989_b200/tune_launch_table.py on one B200 - do not edit.\n"
                 "// {batch * stored pixels per plane, input channels, output channels, GI_KERNEL_* of the fastest 1x1 kernel,\n"
                 "//  milliseconds of the pixel-pair / lane-per-pixel / wide-tile kernel (0 = does not support the shape)}\n")
        for (b, h, w, cin, cout), t in rows:
            best = pick(t)
            kern = dict((n, k) for n, _, k, _ in VARIANTS)[best[1]]
            px = b * ((h * w + 1) // 2 * 2)
            ms = [t[n][0] if n in t else 0.0 for n, _, _, _ in VARIANTS]
            fh.write(f"{{{px}LL, {cin}, {cout}, {kid[kern]}, {ms[0]:.5f}f, {ms[1]:.5f}f, {ms[2]:.5f}f}},\n")
    with open(os.path.join(ROOT, "profiles", "pointwise_variant_choice.md"), "w") as fh:
        fh.write("# Which tensor-core kernel runs a 1x1 convolution: every variant measured on every 1x1 shape of the benchmark networks\n\n"
                 "The paper picks a launch configuration per operator from measurements (Section 4, work-group selection, and its\n"
                 "table of optimal sizes); here the choice is between the three tensor-core 1x1 kernels.  Generated by\n\n"
                 "    python -m paper_1907_01989_b200.tune_launch_table\n\n"
                 "(CUDA events, median of %d launches; before each the L2 is flushed and the input then written by a device copy, so that it\n"
                 "lies where a producing kernel would leave it; PHWC4 buffers in and out so one kernel runs per call).\n"
                 "The same run writes `csrc/launch_table.inc`, which `gi_lower.cc` consults before its rule.\n\n"
                 "| batch | plane | Cin -> Cout | pixel-pair ms | lane-per-pixel ms | wide-tile ms | table entry | the rule picks | rule / table |\n"
                 "|---|---|---|---|---|---|---|---|---|\n" % args.iters)
        worse = 0
        for (b, h, w, cin, cout), t in rows:
            best = pick(t)
            rule_kernel = t["rule"][1]
            rule_variant = [n for n, _, k, _ in VARIANTS if k == rule_kernel][0]
            ratio = t[rule_variant][0] / best[0]
            worse += ratio > 1.03
            cell = lambda n: f"{t[n][0]:.4f}" if n in t else "-"
            fh.write(f"| {b} | {h}x{w} | {cin} -> {cout} | {cell('pair')} | {cell('lane')} | {cell('wide')} | {best[1]} | {rule_variant} | {ratio:.2f} |\n")
        fh.write(f"\n{len(rows)} shapes; on {worse} of them the rule's kernel is more than 3 % slower than the fastest one "
                 "(the table overrides the rule there).\n")


if __name__ == "__main__":
    main()
