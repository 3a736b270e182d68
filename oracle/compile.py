"""Oracle for the compile step: operator fusion, tensor lifetimes, sizes, memory planners
(naive, Algorithm 1, minimum-cost flow, greedy by size).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Every function follows its defining
text step by step with plain Python containers; nothing here is tuned.

A graph description is any object with the attributes of workloads.GraphSpec
(batch, shapes, inputs, outputs, ops[kind, inputs, output, act, ...]); this module
does not import it.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Set, Tuple

CONV_KINDS = ("conv2d", "depthwise_conv2d")


# --------------------------------------------------------------------------------------
# Fusion (Section 3.2, "Shader Program Optimization", first bullet: element-wise
# operators are fused with the expensive operator that precedes them)
# --------------------------------------------------------------------------------------
@dataclass
class FusedOp:
    kind: str                      # kind of the leading op; "pack"/"unpack" for layout conversions
    op_index: Optional[int]        # index of the leading op in the graph description
    inputs: List[int]              # tensors the leading op reads
    output: int                    # tensor the fused op finally writes
    epilogue: List[Tuple[str, object]] = field(default_factory=list)  # ("act", kind) | ("add", tensor)
    slot: int = 0                  # next free position in the pattern [act, add, act]

    def reads(self) -> List[int]:
        return list(self.inputs) + [t for k, t in self.epilogue if k == "add"]

    def take(self, what: str) -> bool:
        """Claim the next pattern position that can hold `what`; the pattern is act, add, act."""
        pattern = ("act", "add", "act")
        for pos in range(self.slot, 3):
            if pattern[pos] == what:
                self.slot = pos + 1
                return True
        return False

    def can_take(self, what: str) -> bool:
        pattern = ("act", "add", "act")
        return any(pattern[pos] == what for pos in range(self.slot, 3))


def fuse(g, enable: bool = True, fold_add: bool = True) -> List[FusedOp]:
    """Walk the ops in their (topological) order and fold element-wise ops into convolutions.

    An ACTIVATION or ADD op E is folded into the fused op F that produces its operand x iff
    F leads with a convolution (full or depthwise), E is the only use of x in the whole graph,
    x is not a graph output, and F's chain stays inside the pattern [act][add][act].  For ADD
    the other operand must be a different tensor of the same shape that exists before F runs
    (a graph input or the output of an earlier fused op); if both operands qualify the later
    fused op takes the add.  The folded op's output replaces x as F's output.

    First the graph is cleaned (Section 3.1, "Graph transformation"): a superfluous identity operator -
    a resize to the size its input already has, or an ADD / CONCAT with a single input - is removed and
    what read its output reads its input; it stays if its output is a graph output.
    """
    alias: Dict[int, int] = {}

    def src(t: int) -> int:
        return alias.get(t, t)

    dropped = set()
    uses: Dict[int, int] = {}
    for idx, op in enumerate(g.ops):
        identity = ((op.kind == "resize_bilinear" and tuple(g.shapes[op.output][:2]) == tuple(g.shapes[op.inputs[0]][:2]))
                    or (op.kind in ("add", "concat") and len(op.inputs) == 1))
        if identity and op.output not in set(g.outputs):
            alias[op.output] = src(op.inputs[0])
            dropped.add(idx)
            continue
        for t in op.inputs:
            uses[src(t)] = uses.get(src(t), 0) + 1
    graph_outputs = set(g.outputs)
    graph_inputs = set(g.inputs)
    fused: List[FusedOp] = []
    producer: Dict[int, int] = {}  # surviving tensor -> index of the fused op that writes it

    def foldable_into(x: int) -> Optional[int]:
        if x not in producer:
            return None
        i = producer[x]
        if fused[i].kind in CONV_KINDS and uses.get(x, 0) == 1 and x not in graph_outputs:
            return i
        return None

    for idx, op in enumerate(g.ops):
        if idx in dropped:
            continue
        ins = [src(t) for t in op.inputs]
        if enable and op.kind == "activation":
            i = foldable_into(ins[0])
            if i is not None and fused[i].can_take("act"):
                fused[i].take("act")
                fused[i].epilogue.append(("act", op.act))
                del producer[fused[i].output]
                fused[i].output = op.output
                producer[op.output] = i
                continue
        if enable and fold_add and op.kind == "add" and len(ins) == 2:
            a, b = ins
            if a != b and g.shapes[a] == g.shapes[b]:
                candidates = []
                for x, other in ((a, b), (b, a)):
                    i = foldable_into(x)
                    if i is None or not fused[i].can_take("add"):
                        continue
                    if other in graph_inputs or (other in producer and producer[other] < i):
                        candidates.append((i, x, other))
                if candidates:
                    i, x, other = max(candidates)
                    fused[i].take("add")
                    fused[i].epilogue.append(("add", other))
                    del producer[x]
                    fused[i].output = op.output
                    producer[op.output] = i
                    continue
        fused.append(FusedOp(kind=op.kind, op_index=idx, inputs=ins, output=op.output))
        producer[op.output] = len(fused) - 1
    return fused


# --------------------------------------------------------------------------------------
# Sizes and the planning problem
# --------------------------------------------------------------------------------------
def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def tensor_bytes(batch: int, shape: Tuple[int, int, int], elem_bytes: int = 2, align: int = 256) -> int:
    """Physical bytes of a PHWC4 tensor (Section 4): ceil(C/4) slices x batch planes of
    round_up(H*W*4, 8) elements, the total rounded up to `align`."""
    H, W, C = shape
    plane_elems = round_up(H * W * 4, 8)
    return round_up(batch * ((C + 3) // 4) * plane_elems * elem_bytes, align)


@dataclass
class PlanProblem:
    ops: List[Tuple[List[int], List[int]]]   # per executed op: (tensors read, tensors written)
    size: Dict[int, int]                     # bytes per tensor
    intermediate: Set[int]                   # tensors that live in the arena


EXTERNAL_BASE = 1 << 20  # ids of caller-owned NHWC buffers, outside the graph's tensor ids


def concat_views(g, fused: Sequence[FusedOp]) -> Dict[int, Tuple[int, int]]:
    """Concatenations that need no copy.  In the channel-sliced layout (Section 4) the slices of a tensor follow
    one another, so concat(a, b) with C(a) a multiple of 4 is `a`'s slices followed by `b`'s: if a and b are
    placed inside the result, their producers write the result directly.  Returns {a: (out, 0), b: (out, S(a))}
    over all eligible CONCAT ops, walked in execution order.  Eligible: two different inputs, C(a) % 4 == 0,
    none of a, b, out is a graph input or output, and neither a nor b is already placed inside another tensor
    or has tensors placed inside it."""
    views: Dict[int, Tuple[int, int]] = {}
    roots: Set[int] = set()
    io = set(g.inputs) | set(g.outputs)
    for f in fused:
        if f.kind != "concat" or len(f.inputs) != 2:
            continue
        a, b = f.inputs
        out = f.output
        if a == b or g.shapes[a][2] % 4 != 0 or {a, b, out} & io:
            continue
        if a in views or b in views or a in roots or b in roots:
            continue
        views[a] = (out, 0)
        views[b] = (out, g.shapes[a][2] // 4)
        roots.add(out)
    return views


def plan_problem(g, fused: Sequence[FusedOp], elem_bytes: int = 2, align: int = 256,
                 convert_io: bool = True, views: Optional[Dict[int, Tuple[int, int]]] = None) -> PlanProblem:
    """The executed op list and which tensors are intermediate (Section 5: neither a graph
    input nor a graph output, which the caller owns).  With convert_io, graph inputs and
    outputs are caller-owned NHWC buffers and a layout conversion op stands between each of
    them and the PHWC4 tensor the graph uses (Section 3, "Running Inference"), which makes
    every tensor of the graph an intermediate.  With `views` (see concat_views) a tensor placed inside
    another one is not planned: every use of it counts as a use of the tensor that holds it."""
    views = views or {}

    def root(t: int) -> int:
        return views[t][0] if t in views else t

    ops: List[Tuple[List[int], List[int]]] = []
    if convert_io:
        for k, t in enumerate(g.inputs):
            ops.append(([EXTERNAL_BASE + k], [t]))
    for f in fused:
        ops.append(([root(t) for t in f.reads()], [root(f.output)]))
    if convert_io:
        for k, t in enumerate(g.outputs):
            ops.append(([t], [EXTERNAL_BASE + len(g.inputs) + k]))
    live = set()
    for r, w in ops:
        live.update(r)
        live.update(w)
    size = {t: tensor_bytes(g.batch, g.shapes[t], elem_bytes, align) for t in live if t < EXTERNAL_BASE}
    if convert_io:
        intermediate = set(size)
    else:
        intermediate = set(size) - set(g.inputs) - set(g.outputs)
    return PlanProblem(ops=ops, size=size, intermediate=intermediate)


def lifetimes(p: PlanProblem) -> Dict[int, Tuple[int, int]]:
    """First and last executed op that touches each intermediate tensor, as input or output
    (Section 5, second paragraph)."""
    life: Dict[int, Tuple[int, int]] = {}
    for i, (reads, writes) in enumerate(p.ops):
        for t in list(reads) + list(writes):
            if t in p.intermediate:
                first, _ = life.get(t, (i, i))
                life[t] = (first, i)
    return life


def lower_bound(p: PlanProblem) -> int:
    """max over ops of the bytes of all intermediate tensors alive at that op."""
    life = lifetimes(p)
    best = 0
    for i in range(len(p.ops)):
        best = max(best, sum(p.size[t] for t, (a, b) in life.items() if a <= i <= b))
    return best


# --------------------------------------------------------------------------------------
# Planners.  Each returns (offset per intermediate tensor, total arena bytes).
# --------------------------------------------------------------------------------------
def plan_naive(p: PlanProblem) -> Tuple[Dict[int, int], int]:
    """Section 5 (a): every intermediate tensor gets memory of its own; offsets are the running
    sum in tensor-id order."""
    offsets, total = {}, 0
    for t in sorted(p.intermediate):
        offsets[t] = total
        total += p.size[t]
    return offsets, total


def plan_greedy_shared_objects(p: PlanProblem):
    """Algorithm 1 (Greedy Memory Management), in the paper's order: for each op, first give
    every intermediate output a shared object (a new one if the pool is empty, else the pooled
    object whose size is closest to the tensor's by absolute difference, grown if too small),
    then return to the pool the objects of the intermediate inputs this op uses last.

    Readings where the paper is silent: equally close objects -> the larger one, then the one
    created first; a tensor listed twice among an op's inputs releases its object once;
    an intermediate output that no op reads is never released (only inputs are inspected).
    One arena: objects are laid out in creation order, each at the sum of the final sizes of
    the objects created before it.

    Returns (offsets, total, object_of_tensor, object_sizes).
    """
    life = lifetimes(p)
    sizes: List[int] = []            # size of shared object k, creation order
    available: List[int] = []        # pool of object indices
    used: Set[int] = set()
    obj: Dict[int, int] = {}
    for i, (reads, writes) in enumerate(p.ops):
        for t in writes:
            if t not in p.intermediate or t in obj:  # (a tensor that several ops write - see plan_problem's views -
                continue                              # takes its object at the first of them)
            if not available:
                sizes.append(p.size[t])
                s = len(sizes) - 1
            else:
                s = min(available, key=lambda k: (abs(sizes[k] - p.size[t]), -sizes[k], k))
                available.remove(s)
                if p.size[t] > sizes[s]:
                    sizes[s] = p.size[t]
            obj[t] = s
            used.add(s)
        released = set()
        for t in reads:
            if t in p.intermediate and life[t][1] == i and t not in released:
                released.add(t)
                used.discard(obj[t])
                available.append(obj[t])
    starts, total = [], 0
    for s in sizes:
        starts.append(total)
        total += s
    offsets = {t: starts[k] for t, k in obj.items()}
    return offsets, total, obj, sizes


def plan_greedy_by_size(p: PlanProblem) -> Tuple[Dict[int, int], int]:
    """Greedy-by-size offsets into one buffer.  Lifetimes are inclusive at both ends.  Tensors
    are taken by decreasing size (ties: earlier first use, then smaller id).  For each, the
    already placed tensors whose lifetimes intersect its own are sorted by offset and the gaps
    between them, starting from offset 0, are scanned: the smallest gap that fits wins (ties:
    lowest offset); if no gap fits the tensor goes after the last of them."""
    life = lifetimes(p)
    order = sorted(p.intermediate, key=lambda t: (-p.size[t], life[t][0], t))
    offsets: Dict[int, int] = {}
    for t in order:
        a, b = life[t]
        placed = sorted((offsets[u], offsets[u] + p.size[u]) for u in offsets
                        if not (life[u][1] < a or b < life[u][0]))
        best_gap, best_off = None, None
        cursor = 0
        for lo, hi in placed:
            gap = lo - cursor
            if gap >= p.size[t] and (best_gap is None or gap < best_gap):
                best_gap, best_off = gap, cursor
            cursor = max(cursor, hi)
        offsets[t] = best_off if best_off is not None else cursor
    total = max((offsets[t] + p.size[t] for t in offsets), default=0)
    return offsets, total


def plan_min_cost_flow(p: PlanProblem):
    """The Minimum-Cost Flow Algorithm of Section 5, in the paper's steps and notation.

    Tensors x = 1..N are the intermediate tensors in execution order (first use, then id).
    Vertices: source s, sink t and two per tensor, l_x and r_x.  Edges, all of capacity 1:
      1. s -> r_x, cost size_x: tensor x gets a new shared object;
      2. l_x -> r_y, cost max(0, size_y - size_x), for every pair where the object of x can be
         re-used for y - x is dead before y is born (last use of x < first use of y; an op's output
         never shares with its input, as in Algorithm 1);
      3. s -> l_x, cost 0;   4. r_x -> t, cost 0.
    The minimum-cost flow (of value N) is found by successive shortest augmenting paths, each
    found with the Shortest Path Faster Algorithm (queue-based Bellman-Ford), as the paper
    names.  A saturated edge of type 1 creates a shared object for x; a saturated edge of type 2
    gives y the object of x.  The size of an object is the largest tensor assigned to it.

    Readings where the paper is silent: edges are inserted in the order 1, 2 (x ascending, then
    y ascending), 3, 4; the queue is first-in first-out and a distance is replaced only by a
    strictly smaller one; one arena, objects laid out in creation order (the order of the
    tensors that open them), as for Algorithm 1.

    Returns (offsets, total, object_of_tensor, object_sizes, flow_cost).
    """
    life = lifetimes(p)
    ts = sorted(p.intermediate, key=lambda t: (life[t][0], t))
    n = len(ts)
    s_v, t_v = 0, 2 * n + 1

    def l_v(i: int) -> int:
        return 1 + i

    def r_v(i: int) -> int:
        return 1 + n + i

    head: List[List[int]] = [[] for _ in range(2 * n + 2)]   # edge ids leaving each vertex
    to: List[int] = []
    cap: List[int] = []
    cost: List[int] = []

    def add_edge(u: int, v: int, c: int) -> None:  # edge 2k and its residual twin 2k+1
        head[u].append(len(to)); to.append(v); cap.append(1); cost.append(c)
        head[v].append(len(to)); to.append(u); cap.append(0); cost.append(-c)

    for i, x in enumerate(ts):                       # type 1
        add_edge(s_v, r_v(i), p.size[x])
    for i, x in enumerate(ts):                       # type 2
        for j, y in enumerate(ts):
            if life[x][1] < life[y][0]:
                add_edge(l_v(i), r_v(j), max(0, p.size[y] - p.size[x]))
    for i in range(n):                               # type 3
        add_edge(s_v, l_v(i), 0)
    for i in range(n):                               # type 4
        add_edge(r_v(i), t_v, 0)

    flow, flow_cost = 0, 0
    while True:
        dist: List[Optional[int]] = [None] * (2 * n + 2)
        via = [-1] * (2 * n + 2)
        queued = [False] * (2 * n + 2)
        dist[s_v] = 0
        queue = [s_v]
        while queue:
            u = queue.pop(0)
            queued[u] = False
            for e in head[u]:
                v = to[e]
                if cap[e] > 0 and (dist[v] is None or dist[u] + cost[e] < dist[v]):
                    dist[v] = dist[u] + cost[e]
                    via[v] = e
                    if not queued[v]:
                        queued[v] = True
                        queue.append(v)
        if dist[t_v] is None:
            break
        v = t_v
        while v != s_v:                              # push one unit along the shortest path
            e = via[v]
            cap[e] -= 1
            cap[e ^ 1] += 1
            v = to[e ^ 1]
        flow += 1
        flow_cost += dist[t_v]
    assert flow == n
    donor: Dict[int, int] = {}                       # y -> x for saturated edges of type 2
    for i in range(n):
        for e in head[l_v(i)]:
            if e % 2 == 0 and cap[e] == 0:
                donor[to[e] - 1 - n] = i
    obj: Dict[int, int] = {}
    sizes: List[int] = []
    for j, y in enumerate(ts):                       # a donor is dead before y is born: it comes earlier
        if j in donor:
            obj[y] = obj[ts[donor[j]]]
            sizes[obj[y]] = max(sizes[obj[y]], p.size[y])
        else:
            obj[y] = len(sizes)
            sizes.append(p.size[y])
    starts, total = [], 0
    for sz in sizes:
        starts.append(total)
        total += sz
    offsets = {t: starts[k] for t, k in obj.items()}
    return offsets, total, obj, sizes, flow_cost


def check_no_overlap(p: PlanProblem, offsets: Dict[int, int]) -> None:
    """Two tensors whose lifetimes intersect must not share a byte."""
    life = lifetimes(p)
    ts = sorted(offsets)
    for i, t in enumerate(ts):
        for u in ts[i + 1:]:
            if life[t][1] < life[u][0] or life[u][1] < life[t][0]:
                continue
            if offsets[t] < offsets[u] + p.size[u] and offsets[u] < offsets[t] + p.size[t]:
                raise AssertionError(f"tensors {t} and {u} overlap while both alive")
