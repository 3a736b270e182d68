"""Oracle for the compile step: operator fusion, tensor lifetimes, sizes, memory planners.

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
    """
    uses: Dict[int, int] = {}
    for op in g.ops:
        for t in op.inputs:
            uses[t] = uses.get(t, 0) + 1
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
        if enable and op.kind == "activation":
            i = foldable_into(op.inputs[0])
            if i is not None and fused[i].can_take("act"):
                fused[i].take("act")
                fused[i].epilogue.append(("act", op.act))
                del producer[fused[i].output]
                fused[i].output = op.output
                producer[op.output] = i
                continue
        if enable and fold_add and op.kind == "add":
            a, b = op.inputs
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
        fused.append(FusedOp(kind=op.kind, op_index=idx, inputs=list(op.inputs), output=op.output))
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


def plan_problem(g, fused: Sequence[FusedOp], elem_bytes: int = 2, align: int = 256,
                 convert_io: bool = True) -> PlanProblem:
    """The executed op list and which tensors are intermediate (Section 5: neither a graph
    input nor a graph output, which the caller owns).  With convert_io, graph inputs and
    outputs are caller-owned NHWC buffers and a layout conversion op stands between each of
    them and the PHWC4 tensor the graph uses (Section 3, "Running Inference"), which makes
    every tensor of the graph an intermediate."""
    ops: List[Tuple[List[int], List[int]]] = []
    if convert_io:
        for k, t in enumerate(g.inputs):
            ops.append(([EXTERNAL_BASE + k], [t]))
    for f in fused:
        ops.append((f.reads(), [f.output]))
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
            if t not in p.intermediate:
                continue
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
