"""CPU oracle for the fused-CNN inference path of arXiv 1907.01989.

TEST INFRASTRUCTURE ONLY: imported by tests/, by __graft_entry__.smoke() and by the
cpu_baseline / reference legs of bench.py.  The CUDA library and its binding never
import it, and it imports nothing from them.

  ops.c / ops.py  operator definitions (fp32 storage, double accumulation), PHWC4
                  indexing, fp16 rounding
  compile.py      graph clean-up, fusion pass, tensor lifetimes, size formula and the memory
                  planners, each written step by step from its defining text
  graph.py        evaluates a graph description (unfused or fused) with the operators
"""
