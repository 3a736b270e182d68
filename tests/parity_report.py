"""Per-tensor parity report: max and 99.9-percentile of |gpu - oracle| / (atol + rtol |oracle|) for every stored
tensor of a network (naive planner, so every tensor survives), fp16 and fp32 storage.

    python tests/parity_report.py [v1|v2|seg|fire] [batch]

Needs a B200 and the built library; the oracle is the CPU reference (test infrastructure).  A value <= 1 is inside
the tolerance the tests enforce (fp16: 1e-2 + 1e-2 |oracle|, fp32: 1e-4 + 1e-4 |oracle|).
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from gpu_util import DeviceRun, error_report  # noqa: E402
from oracle import graph as og  # noqa: E402
from paper_1907_01989_b200 import api  # noqa: E402
from paper_1907_01989_b200 import workloads as wl  # noqa: E402

NETS = {"v1": wl.mobilenet_v1, "v2": wl.mobilenet_v2, "seg": wl.mobilenet_v2_segmentation, "fire": wl.fire_network}


def main():
    net = sys.argv[1] if len(sys.argv) > 1 else "v2"
    batch = int(sys.argv[2]) if len(sys.argv) > 2 else 1
    spec = NETS[net](batch)
    xs = [wl.make_input(spec, index=i) for i in range(len(spec.inputs))]
    print(f"# {spec.name}, batch {batch}: normalised error per stored tensor (max / 99.9 %)")
    for storage, name in ((api.GI_F16, "f16"), (api.GI_F32, "f32")):
        ref = og.run(spec, xs, storage=name, fused=True, keep_all=True)
        run = DeviceRun(spec, storage, planner=api.GI_PLAN_NAIVE)
        outs = run.run(xs)
        rows = []
        for t, r in sorted(ref.items()):
            if t in run.on_chip:  # never stored (the converted copy of an NHWC input the stem reads itself, a fused block's hidden tensors)
                continue
            got = outs[t] if t in outs else run.fetch(t)
            worst, q999 = error_report(got, r, storage)
            rows.append((t, tuple(spec.shapes[t]), worst, q999))
        print(f"## storage {name}: {len(rows)} tensors, worst max {max(r[2] for r in rows):.3f}, worst 99.9 % {max(r[3] for r in rows):.3f}")
        print("tensor shape max q99.9")
        for t, shape, worst, q999 in rows:
            print(t, "x".join(map(str, shape)), f"{worst:.3f}", f"{q999:.3f}")
    assert api.gi_device_status() == 0


if __name__ == "__main__":
    main()
