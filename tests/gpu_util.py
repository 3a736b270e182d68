"""Helpers for the GPU parity tests: run a workload through the C ABI and fetch tensors back."""
import numpy as np

from paper_1907_01989_b200 import api

TOL = {api.GI_F16: (1e-2, 1e-2), api.GI_F32: (1e-4, 1e-4)}  # |gpu - oracle| <= atol + rtol * |oracle|


def np_dtype(storage):
    return np.float16 if storage == api.GI_F16 else np.float32


def unpack_phwc4(raw: np.ndarray, B: int, H: int, W: int, Cc: int) -> np.ndarray:
    """[S][B][plane][4] physical array -> NHWC (test-side restatement of the layout in include/gi.h)."""
    S, P = (Cc + 3) // 4, (H * W + 1) // 2 * 2
    a = raw[: S * B * P * 4].reshape(S, B, P, 4)[:, :, : H * W, :]
    return np.ascontiguousarray(a.transpose(1, 2, 0, 3).reshape(B, H, W, S * 4)[..., :Cc])


def pack_slice8(x: np.ndarray) -> np.ndarray:
    """NHWC -> [ceil(C/8)][B][plane][8] (the 8-channel-slice layout of include/gi.h's layout experiment), zero padded."""
    B, H, W, Cc = x.shape
    S, P = (Cc + 7) // 8, (H * W + 1) // 2 * 2
    a = np.zeros((B, P, S * 8), dtype=x.dtype)
    a[:, : H * W, :Cc] = x.reshape(B, H * W, Cc)
    return np.ascontiguousarray(a.reshape(B, P, S, 8).transpose(2, 0, 1, 3))


def unpack_slice8(raw: np.ndarray, B: int, H: int, W: int, Cc: int) -> np.ndarray:
    S, P = (Cc + 7) // 8, (H * W + 1) // 2 * 2
    a = raw[: S * B * P * 8].reshape(S, B, P, 8)[:, :, : H * W, :]
    return np.ascontiguousarray(a.transpose(1, 2, 0, 3).reshape(B, H, W, S * 8)[..., :Cc])


# Every byte of the arena (and of the output buffers) starts as 0xFF: in fp16 and in fp32 storage that is a NaN.
# The 1x1 tensor-core kernels multiply neighbouring pixels and padding lanes by structural zeros, and
# 0 x NaN = NaN, so a kernel that leaves a padding lane or the padding pixel of an odd plane unwritten - harmless
# when the memory happens to hold small finite numbers - shows up as a NaN in the compared result.
POISON = 0xFF


class DeviceRun:
    def __init__(self, spec, storage=api.GI_F16, planner=api.GI_PLAN_GREEDY_BY_SIZE, pointwise=api.GI_PW_AUTO,
                 fuse=True, guard_bytes=0, cross_op=api.GI_XOP_AUTO):
        import torch
        self.torch = torch
        self.spec, self.storage = spec, storage
        self.graph, _ = api.graph_from_spec(spec, storage)
        self.ex = self.graph.compile(planner=planner, fuse=fuse, pointwise=pointwise, cross_op=cross_op)
        # tensors that stay on chip: the input of an op that runs inside the previous op's kernel (the kernel that runs
        # two 1x1 convolutions stores the tensor between them as well, so there it is compared like any other)
        self.on_chip, launcher = set(), None
        for o in self.ex.ops():
            name = api.KERNEL_NAMES[o.kernel]
            if name != "none":
                launcher = name
            elif o.kind in (api.GI_OP_CONV2D, api.GI_OP_DEPTHWISE_CONV2D) and launcher != "pointwise_chain":
                self.on_chip.add(o.inputs[0])
        # ... and the converted copy of an NHWC input that the first convolution reads in the caller's layout itself
        self.on_chip |= {o.output for o in self.ex.ops() if api.KERNEL_NAMES[o.kernel] == "none" and o.kind == api.GI_EXEC_PACK}
        dev = "cuda:0"
        nb = int(self.ex.info.arena_bytes)
        self.guard = guard_bytes
        self.arena = torch.full((max(nb, 256) + guard_bytes,), POISON, dtype=torch.uint8, device=dev)
        self.weights = torch.empty(max(int(self.ex.info.weight_bytes), 256), dtype=torch.uint8, device=dev)
        self.ex.bind_raw(self.weights.data_ptr(), self.weights.numel())
        tdt = torch.float16 if storage == api.GI_F16 else torch.float32
        self.outs = [torch.full((spec.batch,) + tuple(spec.shapes[t]), float("nan"), dtype=tdt, device=dev) for t in spec.outputs]
        self.tdt = tdt

    def run(self, inputs):
        torch = self.torch
        self.ins = [torch.from_numpy(np.ascontiguousarray(x)).to("cuda:0").to(self.tdt).contiguous() for x in inputs]
        self.ex.run_raw([t.data_ptr() for t in self.ins], [t.data_ptr() for t in self.outs], self.arena.data_ptr(),
                        max(int(self.ex.info.arena_bytes), 256))
        torch.cuda.synchronize()
        return {t: o.float().cpu().numpy() for t, o in zip(self.spec.outputs, self.outs)}

    def guard_intact(self) -> bool:
        if not self.guard:
            return True
        g = self.arena[-self.guard:]
        return bool((g == POISON).all().item())

    def fetch(self, t: int) -> np.ndarray:
        """Read an intermediate tensor out of the arena (meaningful for every tensor only under the naive planner)."""
        ti = self.ex.tensor(t)
        assert ti.alive and ti.intermediate
        raw = self.arena[ti.offset: ti.offset + ti.bytes].cpu().numpy().view(np_dtype(self.storage))
        return unpack_phwc4(raw, self.spec.batch, ti.h, ti.w, ti.c).astype(np.float32)

    def fetch_raw(self, t: int) -> np.ndarray:
        ti = self.ex.tensor(t)
        return self.arena[ti.offset: ti.offset + ti.bytes].cpu().numpy().view(np_dtype(self.storage))


def error_report(got: np.ndarray, ref: np.ndarray, storage):
    atol, rtol = TOL[storage]
    norm = np.abs(got.astype(np.float64) - ref.astype(np.float64)) / (atol + rtol * np.abs(ref.astype(np.float64)))
    return float(norm.max()), float(np.quantile(norm, 0.999))


def assert_close(got, ref, storage, what=""):
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what
    worst, q999 = error_report(got, ref, storage)
    assert worst <= 1.0, f"{what}: max normalised error {worst:.3f} (99.9%: {q999:.3f})"
    return worst
