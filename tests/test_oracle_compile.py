"""Pins for the oracle's compile step: fusion, lifetimes and the memory planners."""
import itertools
import os
import random
from types import SimpleNamespace as NS

import pytest

from oracle import compile as oc
from paper_1907_01989_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MIB = float(2 ** 20)


def problem(ops, size, intermediate=None):
    inter = set(size) if intermediate is None else set(intermediate)
    return oc.PlanProblem(ops=[(list(r), list(w)) for r, w in ops], size=dict(size), intermediate=inter)


# The hand example: x -> t0 (10), x -> t1 (40), add(t0, t1) -> t2 (3), f(t2) -> t3 (20), g(t3) -> out
X, OUT = 100, 101


def hand_example(t3=20):
    ops = [([X], [0]), ([X], [1]), ([0, 1], [2]), ([2], [3]), ([3], [OUT])]
    return problem(ops, {0: 10, 1: 40, 2: 3, 3: t3})


# ---------------------------------------------------------------------- the memory table of Section 5
def _memory_table():
    rows = {}
    with open(os.path.join(GOLDEN, "section5_memory_table.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, v1, v2 = line.split()
                rows[k] = (float(v1), float(v2))
    return rows


def test_section5_memory_table_totals():
    """Algorithm 1 and the naive strategy reproduce the paper's printed totals for MobileNet v1 and
    MobileNetV2.  This pins 'outputs get their object before inputs are released' (the opposite
    order gives 1.53 for v1) and 'the pool is used whenever it is not empty, growing the object'."""
    t4 = _memory_table()
    for col, (g, fold_add) in enumerate(((wl.mobilenet_v1(1), True), (wl.mobilenet_v2(1), False))):
        fused = oc.fuse(g, fold_add=fold_add)
        p = oc.plan_problem(g, fused, elem_bytes=2, align=1, convert_io=False)
        naive = oc.plan_naive(p)[1] / MIB
        greedy = oc.plan_greedy_shared_objects(p)[1] / MIB
        assert round(naive, 1) == t4["naive"][col]
        assert round(greedy, 1) == t4["greedy"][col]
        # the minimum-cost flow strategy: larger than Algorithm 1 on MobileNet, smaller on MobileNetV2, as printed
        mcfp = oc.plan_min_cost_flow(p)[1] / MIB
        assert round(mcfp, 1) == t4["mcfp"][col]


def test_release_before_allocate_would_not_match_the_memory_table():
    # the other reading of Algorithm 1's order, kept here only to show that the memory table of Section 5 tells them apart
    g = wl.mobilenet_v1(1)
    p = oc.plan_problem(g, oc.fuse(g), 2, 1, convert_io=False)
    life = oc.lifetimes(p)
    sizes, avail, obj = [], [], {}
    for i, (reads, writes) in enumerate(p.ops):
        for t in reads:
            if t in p.intermediate and life[t][1] == i:
                avail.append(obj[t])
        for t in writes:
            if t in p.intermediate:
                if not avail:
                    sizes.append(p.size[t])
                    s = len(sizes) - 1
                else:
                    s = min(avail, key=lambda k: abs(sizes[k] - p.size[t]))
                    avail.remove(s)
                    sizes[s] = max(sizes[s], p.size[t])
                obj[t] = s
    assert round(sum(sizes) / MIB, 1) != 2.3


# ---------------------------------------------------------------------- Algorithm 1 details
def test_alg1_hand_example_closest_by_absolute_difference():
    p = hand_example()
    off, total, obj, sizes = oc.plan_greedy_shared_objects(p)
    # t2 (3) finds an empty pool -> third object; t3 (20) sees pool {10, 40}: |10-20| < |40-20| -> grows the 10
    assert sizes == [20, 40, 3] and total == 63
    assert obj == {0: 0, 1: 1, 2: 2, 3: 0}
    assert off == {0: 0, 1: 20, 2: 60, 3: 0}


def test_alg1_tie_prefers_larger_object():
    p = hand_example(t3=25)  # |10-25| == |40-25|: the larger object is taken, nothing grows
    off, total, obj, sizes = oc.plan_greedy_shared_objects(p)
    assert sizes == [10, 40, 3] and obj[3] == 1 and total == 53


def test_alg1_chain_uses_two_objects():
    sizes = [7, 3, 9, 4, 12, 1, 5]
    ops = [([X], [0])] + [([i - 1], [i]) for i in range(1, len(sizes))] + [([len(sizes) - 1], [OUT])]
    p = problem(ops, dict(enumerate(sizes)))
    _, total, obj, osz = oc.plan_greedy_shared_objects(p)
    assert len(osz) == 2
    assert sorted(osz) == sorted([max(sizes[0::2]), max(sizes[1::2])])
    assert all(obj[i] == i % 2 for i in range(len(sizes)))
    assert total == max(sizes[0::2]) + max(sizes[1::2])


def test_alg1_same_tensor_twice_released_once():
    ops = [([X], [0]), ([0, 0], [1]), ([1], [2]), ([2], [OUT])]
    p = problem(ops, {0: 8, 1: 8, 2: 8})
    _, total, obj, sizes = oc.plan_greedy_shared_objects(p)
    assert sizes == [8, 8] and obj == {0: 0, 1: 1, 2: 0}


def test_shared_object_size_is_max_of_its_tensors():
    rnd = random.Random(5)
    for _ in range(50):
        p = random_problem(rnd, 12)
        _, _, obj, sizes = oc.plan_greedy_shared_objects(p)
        for k, s in enumerate(sizes):
            assert s == max(p.size[t] for t, o in obj.items() if o == k)


# ---------------------------------------------------------------------- minimum-cost flow
def cheapest_assignment(p):
    """Brute force over the problem the flow network encodes: every tensor either opens an object (cost: its
    size) or takes over the object of a tensor that is dead before it is born, each donor used once
    (cost: the growth max(0, size_y - size_x))."""
    life = oc.lifetimes(p)
    ts = sorted(p.intermediate)
    best = [None]

    def rec(k, used, cost):
        if best[0] is not None and cost >= best[0]:
            return
        if k == len(ts):
            best[0] = cost
            return
        y = ts[k]
        rec(k + 1, used, cost + p.size[y])
        for x in ts:
            if x not in used and life[x][1] < life[y][0]:
                rec(k + 1, used | {x}, cost + max(0, p.size[y] - p.size[x]))

    rec(0, frozenset(), 0)
    return best[0]


def test_mcfp_hand_example():
    # t3 (20) may take over t0 (10, growth 10) or t1 (40, growth 0); t2 overlaps both: 10 + 40 + 3 + 0
    p = hand_example()
    off, total, obj, sizes, cost = oc.plan_min_cost_flow(p)
    assert cost == 53 and total == 53 and sizes == [10, 40, 3]
    assert obj[3] == obj[1] and off == {0: 0, 1: 10, 2: 50, 3: 10}
    oc.check_no_overlap(p, off)


def test_mcfp_chain_of_equal_tensors_uses_two_objects():
    n = 9
    p = problem([([X], [0])] + [([i - 1], [i]) for i in range(1, n)] + [([n - 1], [OUT])], {i: 7 for i in range(n)})
    off, total, obj, sizes, cost = oc.plan_min_cost_flow(p)
    assert cost == 14 and sizes == [7, 7]
    assert all(obj[i] == i % 2 for i in range(n))


def test_mcfp_flow_cost_is_the_minimum_and_bounds_the_total():
    rnd = random.Random(5)
    for trial in range(150):
        p = random_problem(rnd, rnd.randint(2, 8))
        off, total, obj, sizes, cost = oc.plan_min_cost_flow(p)
        assert cost == cheapest_assignment(p)
        # the growth charged per re-use is what the object grows by at most (the paper: "a good approximation")
        assert oc.lower_bound(p) <= total <= cost <= oc.plan_naive(p)[1]
        oc.check_no_overlap(p, off)
        assert set(off) == p.intermediate
        for t, k in obj.items():
            assert p.size[t] <= sizes[k]


def test_mcfp_invariants_larger_random_dags():
    rnd = random.Random(6)
    for trial in range(40):
        p = random_problem(rnd, rnd.randint(10, 40))
        off, total, obj, sizes, cost = oc.plan_min_cost_flow(p)
        oc.check_no_overlap(p, off)
        assert oc.lower_bound(p) <= total <= cost <= oc.plan_naive(p)[1]
        assert total == sum(sizes)


# ---------------------------------------------------------------------- greedy by size
def test_by_size_hand_example():
    p = hand_example()
    off, total = oc.plan_greedy_by_size(p)
    assert off == {1: 0, 3: 0, 0: 40, 2: 50} and total == 53 == oc.lower_bound(p)


def test_by_size_prefers_smallest_fitting_gap():
    # G1 (30) and G2 (15) die early; A (20) and B (12) live to the end; F (4) is born after G1, G2 died.
    # Placement by size: G1@0, A@30, G2@50, B@65.  F conflicts with A [30,50) and B [65,77):
    # free gaps are [0,30) and [50,65); the smaller one that fits wins -> 50 (first fit would say 0).
    G1, A, G2, B, F = 0, 1, 2, 3, 4
    ops = [([X], [G1, A, G2, B]), ([G1, G2], [OUT]), ([X], [OUT]), ([X], [F]), ([A, B, F], [OUT])]
    p = problem(ops, {G1: 30, A: 20, G2: 15, B: 12, F: 4})
    off, total = oc.plan_greedy_by_size(p)
    oc.check_no_overlap(p, off)
    assert off == {G1: 0, A: 30, G2: 50, B: 65, F: 50} and total == 77


def random_problem(rnd, n):
    """A random DAG of n single-output ops over random sizes; op i reads 1-2 earlier tensors or the input."""
    ops, size = [], {}
    for i in range(n):
        k = rnd.choice([1, 1, 2])
        reads = [rnd.choice([X] + list(range(max(0, i - 4), i))) for _ in range(k)] if i else [X]
        ops.append((reads, [i]))
        size[i] = rnd.choice([1, 2, 3, 4, 6, 8, 12, 16]) * rnd.choice([1, 16])
    ops.append(([n - 1], [OUT]))
    return problem(ops, size)


def optimal_first_fit(p):
    """Minimum arena over all placement orders of lowest-offset first fit (tiny problems only)."""
    life = oc.lifetimes(p)
    best = None
    for order in itertools.permutations(sorted(p.intermediate)):
        off = {}
        for t in order:
            a, b = life[t]
            placed = sorted((off[u], off[u] + p.size[u]) for u in off if not (life[u][1] < a or b < life[u][0]))
            cur = 0
            for lo, hi in placed:
                if lo - cur >= p.size[t]:
                    break
                cur = max(cur, hi)
            off[t] = cur
        total = max(off[t] + p.size[t] for t in off)
        best = total if best is None else min(best, total)
    return best


def test_by_size_invariants_random_dags():
    rnd = random.Random(11)
    for trial in range(300):
        p = random_problem(rnd, rnd.randint(2, 25))
        off, total = oc.plan_greedy_by_size(p)
        oc.check_no_overlap(p, off)
        assert set(off) == p.intermediate
        naive = oc.plan_naive(p)[1]
        assert oc.lower_bound(p) <= total <= naive
        a1 = oc.plan_greedy_shared_objects(p)
        oc.check_no_overlap(p, a1[0])
        assert oc.lower_bound(p) <= a1[1] <= naive


def test_by_size_never_beats_true_optimum_on_tiny_problems():
    rnd = random.Random(3)
    for trial in range(40):
        p = random_problem(rnd, rnd.randint(2, 6))
        total = oc.plan_greedy_by_size(p)[1]
        opt = optimal_first_fit(p)
        assert oc.lower_bound(p) <= opt <= total


def test_expected_totals_on_the_networks():
    # the greedy-by-size arena equals the live-bytes lower bound on all three networks
    for g, want_mib in ((wl.mobilenet_v1(1), 2.297), (wl.mobilenet_v2(1), 2.871), (wl.mobilenet_v2_segmentation(1), 15.14)):
        p = oc.plan_problem(g, oc.fuse(g), 2, 256, convert_io=True)
        off, total = oc.plan_greedy_by_size(p)
        oc.check_no_overlap(p, off)
        assert total == oc.lower_bound(p)
        assert abs(total / MIB - want_mib) < 2e-3
        assert all(o % 256 == 0 for o in off.values())


def test_planner_speed_on_large_graph():
    import time
    rnd = random.Random(2)
    p = random_problem(rnd, 2000)
    t0 = time.time()
    oc.plan_greedy_shared_objects(p)
    assert time.time() - t0 < 5.0


# ---------------------------------------------------------------------- lifetimes, sizes
def test_lifetimes_and_lower_bound_hand_example():
    p = hand_example()
    assert oc.lifetimes(p) == {0: (0, 2), 1: (1, 2), 2: (2, 3), 3: (3, 4)}
    assert oc.lower_bound(p) == 53


def test_tensor_bytes_formula():
    assert oc.tensor_bytes(1, (8, 6, 12), 2, 1) == 8 * 6 * 12 * 2
    assert oc.tensor_bytes(1, (8, 6, 5), 2, 1) == oc.tensor_bytes(1, (8, 6, 8), 2, 1)  # C=5 costs like C=8
    assert oc.tensor_bytes(1, (7, 7, 4), 2, 1) == 50 * 4 * 2                            # odd plane gets a pad pixel
    assert oc.tensor_bytes(3, (7, 7, 4), 2, 256) == 1280
    assert oc.tensor_bytes(2, (1, 1, 1001), 4, 256) == oc.round_up(2 * 251 * 8 * 4, 256)


# ---------------------------------------------------------------------- fusion
def test_fusion_counts():
    assert len(oc.fuse(wl.separable_block())) == 2
    assert len(oc.fuse(wl.mobilenet_v1())) == 29
    assert len(oc.fuse(wl.mobilenet_v2())) == 54
    assert len(oc.fuse(wl.mobilenet_v2_segmentation())) == 54
    assert len(oc.fuse(wl.mobilenet_v2(), enable=False)) == 99
    assert len(oc.fuse(wl.mobilenet_v2(), fold_add=False)) == 64


def test_fusion_v2_block_structure():
    g = wl.mobilenet_v2()
    f = oc.fuse(g)
    with_add = [x for x in f if any(k == "add" for k, _ in x.epilogue)]
    assert len(with_add) == 10
    for x in with_add:
        assert x.kind == "conv2d" and x.epilogue[0][0] == "add" and len(x.epilogue) == 1
        res = x.epilogue[0][1]
        assert g.shapes[res] == g.shapes[x.output]
    assert sum(1 for x in f if x.kind == "depthwise_conv2d" and x.epilogue == [("act", "relu6")]) == 17


def _g(shapes, inputs, outputs, ops):
    return NS(batch=1, shapes=shapes, inputs=inputs, outputs=outputs,
              ops=[NS(kind=k, inputs=i, output=o, act=a) for k, i, o, a in ops])


def test_fusion_rules_small_cases():
    s = (4, 4, 4)
    # activation with two consumers of the conv output: not folded
    g = _g({i: s for i in range(5)}, [0], [3, 4],
           [("conv2d", [0], 1, None), ("activation", [1], 2, "relu"), ("activation", [1], 3, "relu6"),
            ("add", [2, 3], 4, None)])
    f = oc.fuse(g)
    assert [x.kind for x in f] == ["conv2d", "activation", "activation", "add"]
    # conv output that is a graph output: not folded
    g = _g({i: s for i in range(3)}, [0], [1, 2], [("conv2d", [0], 1, None), ("activation", [1], 2, "relu")])
    assert len(oc.fuse(g)) == 2
    # act, add, act all fold; a fourth element-wise op does not
    g = _g({i: s for i in range(7)}, [0], [6],
           [("conv2d", [0], 1, None), ("activation", [1], 2, "relu"), ("add", [0, 2], 3, None),
            ("activation", [3], 4, "relu6"), ("activation", [4], 5, "relu"), ("activation", [5], 6, "relu")])
    f = oc.fuse(g)
    assert len(f) == 3 and f[0].epilogue == [("act", "relu"), ("add", 0), ("act", "relu6")] and f[0].output == 4
    # add of a tensor with itself is not folded; add whose other operand is produced later is folded into the later conv
    g = _g({i: s for i in range(3)}, [0], [2], [("conv2d", [0], 1, None), ("add", [1, 1], 2, None)])
    assert len(oc.fuse(g)) == 2
    g = _g({i: s for i in range(4)}, [0], [3],
           [("conv2d", [0], 1, None), ("conv2d", [0], 2, None), ("add", [1, 2], 3, None)])
    f = oc.fuse(g)
    assert len(f) == 2 and f[1].epilogue == [("add", 1)] and f[1].output == 3
    # the producer of the folded operand is not a convolution: stays standalone
    g = _g({0: s, 1: (1, 1, 4), 2: (1, 1, 4)}, [0], [2], [("global_avg_pool", [0], 1, None), ("activation", [1], 2, "relu")])
    assert len(oc.fuse(g)) == 2
    # two adds cannot both fold
    g = _g({i: s for i in range(4)}, [0], [3],
           [("conv2d", [0], 1, None), ("add", [0, 1], 2, None), ("add", [0, 2], 3, None)])
    f = oc.fuse(g)
    assert len(f) == 2 and f[1].kind == "add"


# ---------------------------------------------------------------------- identity removal (Section 3.1)
def _identity_graph(extra_output=False):
    """conv -> resize to the same size -> relu -> resize to the same size -> resize x2 -> output."""
    b = wl.GraphBuilder("identity_ops", 2, 21)
    x = b.input(6, 5, 8)
    c = b.conv2d(x, 12, 1)
    r1 = b.resize_bilinear(c, 6, 5, True)
    a = b.activation(r1, wl.ACT_RELU)
    r2 = b.resize_bilinear(a, 6, 5, False)
    r3 = b.resize_bilinear(r2, 12, 10, True)
    if extra_output:
        b.output(r2)
    b.output(r3)
    return b.finish(), (c, r1, a, r2, r3)


def test_identity_resize_is_removed_and_its_readers_read_its_input():
    g, (c, r1, a, r2, r3) = _identity_graph()
    f = oc.fuse(g)
    # the activation folds into the convolution THROUGH the removed resize; the real resize reads the conv's result
    assert [x.kind for x in f] == ["conv2d", "resize_bilinear"]
    assert f[0].epilogue == [("act", "relu")] and f[0].output == a and f[1].inputs == [a] and f[1].output == r3
    p = oc.plan_problem(g, f, convert_io=True)
    assert r1 not in p.size and r2 not in p.size
    # without fusion the identities are still removed
    assert [x.kind for x in oc.fuse(g, enable=False)] == ["conv2d", "activation", "resize_bilinear"]


def test_identity_resize_that_is_a_graph_output_stays():
    g, (c, r1, a, r2, r3) = _identity_graph(extra_output=True)
    f = oc.fuse(g)
    assert [x.kind for x in f] == ["conv2d", "resize_bilinear", "resize_bilinear"]
    assert f[1].output == r2 and f[1].inputs == [a] and f[2].inputs == [r2]
