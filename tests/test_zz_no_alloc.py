"""gi_run_static: the entry point for callers that cannot allocate device memory (an embedding
application owns all of it, the budget is spent, or cudaMalloc is off limits in their loop).
Its intermediates live in an array built into the library, so the test checks that it gives
exactly what gi_run gives with a caller-provided arena - on two calls in a row with different
images, because the array keeps whatever the previous call left in it."""
import numpy as np
import pytest

from paper_1907_01989_b200 import api
from paper_1907_01989_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_arena_matches_caller_arena_twice():
    import torch
    spec = wl.mobilenet_v2(2, size=128)
    g, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = g.compile()
    assert 0 < ex.info.arena_bytes <= api.GI_STATIC_ARENA_BYTES
    ex.bind("cuda:0")  # weights and the reference arena: the test may allocate, the entry point may not
    out_shape = (spec.batch,) + tuple(spec.shapes[spec.outputs[0]])
    for images in ([0, 1], [5, 9]):
        x = torch.from_numpy(wl.make_input(spec, images=images)).to("cuda:0").half().contiguous()
        ref = torch.zeros(out_shape, dtype=torch.float16, device="cuda:0")
        got = torch.zeros(out_shape, dtype=torch.float16, device="cuda:0")
        ex.run([x], [ref])
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        ex.run_static([x], [got])
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        r, o = ref.float().cpu().numpy(), got.float().cpu().numpy()
        assert np.isfinite(o).all() and np.abs(r).max() > 0
        # same kernels, same order: identical bits; the suite's fp16 tolerance is the outer bound
        assert np.all(np.abs(o - r) <= 1e-2 + 1e-2 * np.abs(r))
        assert np.array_equal(o, r)


def test_static_arena_rejects_oversized_executable():
    import torch
    spec = wl.mobilenet_v2(16)
    g, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = g.compile()
    assert ex.info.arena_bytes > api.GI_STATIC_ARENA_BYTES
    ex.bind("cuda:0")
    x = torch.zeros((16, 224, 224, 3), dtype=torch.float16, device="cuda:0")
    out = torch.zeros((16, 1, 1, 1001), dtype=torch.float16, device="cuda:0")
    with pytest.raises(api.GiError) as ei:
        ex.run_static([x], [out])
    assert ei.value.status == api.GI_E_ARENA
    assert "built-in arena" in str(ei.value)
