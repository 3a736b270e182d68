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


def _free_bytes(torch):
    # what the driver reports, not what PyTorch's caching allocator counts: a cudaMalloc inside the library
    # (it links its own CUDA runtime) would lower this and leave torch.cuda.memory_allocated() untouched
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_static_arena_matches_caller_arena_twice():
    import torch
    spec = wl.mobilenet_v2(2, size=128)
    g, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = g.compile()
    assert 0 < ex.info.arena_bytes <= api.GI_STATIC_ARENA_BYTES
    ex.bind("cuda:0")  # weights and the reference arena: the test may allocate, the entry point may not
    # a second, different executable that also runs in the built-in array: between our two calls it leaves
    # foreign data there, as another user of the library in the same process would
    other_spec = wl.fire_network(3)
    og_, _ = api.graph_from_spec(other_spec, api.GI_F16)
    other = og_.compile()
    other.bind("cuda:0")
    ox = torch.from_numpy(wl.make_input(other_spec)).to("cuda:0").half().contiguous()
    oo = torch.zeros((other_spec.batch,) + tuple(other_spec.shapes[other_spec.outputs[0]]), dtype=torch.float16, device="cuda:0")
    out_shape = (spec.batch,) + tuple(spec.shapes[spec.outputs[0]])
    first_call = True
    for images in ([0, 1], [5, 9]):
        x = torch.from_numpy(wl.make_input(spec, images=images)).to("cuda:0").half().contiguous()
        ref = torch.zeros(out_shape, dtype=torch.float16, device="cuda:0")
        got = torch.zeros(out_shape, dtype=torch.float16, device="cuda:0")
        ex.run([x], [ref])
        torch.cuda.synchronize()
        # the caller's arena now holds exactly the right intermediates: destroy them (0xFF bytes are fp16 NaNs), so
        # that a static run that read the caller's arena by mistake could not come out equal
        ex.arena.fill_(0xFF)
        other.run_static([ox], [oo])  # foreign contents in the built-in array (and its address looked up, first time)
        torch.cuda.synchronize()
        assert torch.isfinite(oo.float()).all()
        free_before = _free_bytes(torch)
        ex.run_static([x], [got])
        free_after = _free_bytes(torch)
        if not first_call:
            # (the very first launch of a kernel may make the driver load its code; from the second call on the
            # free memory the driver reports must not move at all)
            assert free_after == free_before, (free_before, free_after)
        first_call = False
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
