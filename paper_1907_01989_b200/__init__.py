"""B200-native fused-CNN graph inference (after arXiv 1907.01989).

The product is the C-ABI library declared in include/gi.h (CUDA, sm_100a only);
`paper_1907_01989_b200.api` is the thin ctypes binding over it and
`paper_1907_01989_b200.workloads` the seeded synthetic workload generator.
There is no CPU fallback: using the binding without the built library raises.
"""
