// Compile step: operator fusion (Section 3.2), tensor lifetimes and the memory planners
// for intermediate tensors (Section 5), plus the query half of the C ABI.
#include <algorithm>
#include <cstring>
#include <deque>
#include <limits>
#include <map>
#include <new>
#include <set>

#include "gi_internal.h"

namespace gi {

static bool is_conv(int kind) { return kind == GI_OP_CONV2D || kind == GI_OP_DEPTHWISE_CONV2D; }
// ADD and CONCAT read inputs[1] unless it is -1 (a single-input ADD / CONCAT is the identity)
static bool two_inputs(const OpNode& op) { return (op.d.kind == GI_OP_ADD || op.d.kind == GI_OP_CONCAT) && op.d.inputs[1] >= 0; }

// The folded chain must be a sub-sequence of [activation][add][activation].
// `what`: 0 = activation, 1 = add.  Returns the pattern position it would occupy, or -1.
static int next_slot(int slot, int what) {
  static const int pattern[3] = {0, 1, 0};
  for (int p = slot; p < 3; ++p)
    if (pattern[p] == what) return p;
  return -1;
}

// Section 3.2, first bullet: element-wise operators are merged into the expensive operator
// before them so that fewer programs are queued.  An ACTIVATION or ADD is folded into the
// fused op that produces its operand when that op leads with a convolution, the operand has
// no other use and is not a graph output, and the chain stays inside [act][add][act]; the
// other operand of a folded ADD must already exist when the convolution runs.
//
// Before that, the graph is cleaned as in Section 3.1: a superfluous identity operator - a RESIZE whose
// output has the size of its input, an ADD or CONCAT with a single input - is dropped and its readers read
// its input instead (unless its output is a graph output, which has to exist as a tensor of its own).
gi_status fuse_graph(const gi_graph& g, bool enable, std::vector<FusedOp>* out) {
  const int nt = static_cast<int>(g.tensors.size());
  std::vector<int> alias(nt);  // tensor -> the tensor that holds its values
  for (int t = 0; t < nt; ++t) alias[t] = t;
  std::vector<char> dropped(g.ops.size(), 0);
  std::vector<int> uses(nt, 0);
  for (size_t idx = 0; idx < g.ops.size(); ++idx) {
    const OpNode& op = g.ops[idx];
    // insertion order must be topological: every input id is smaller than the output id
    for (int k = 0; k < 2; ++k) {
      const int t = op.d.inputs[k];
      if (k == 1 && !two_inputs(op)) continue;
      if (t < 0 || t >= op.output) return fail(GI_E_INVALID, "gi_compile: operator reads a tensor defined after it");
    }
    const int in0 = op.d.inputs[0];
    const bool same_size_resize = op.d.kind == GI_OP_RESIZE_BILINEAR && g.tensors[op.output].h == g.tensors[in0].h &&
                                  g.tensors[op.output].w == g.tensors[in0].w;
    const bool single_input = (op.d.kind == GI_OP_ADD || op.d.kind == GI_OP_CONCAT) && !two_inputs(op);
    if ((same_size_resize || single_input) && g.tensors[op.output].output_index < 0) {
      alias[op.output] = alias[in0];
      dropped[idx] = 1;
      continue;
    }
    ++uses[alias[in0]];
    if (two_inputs(op)) ++uses[alias[op.d.inputs[1]]];
  }
  std::vector<FusedOp>& fused = *out;
  fused.clear();
  std::vector<int> producer(nt, -1);  // fused-op index that currently writes the tensor

  auto foldable = [&](int x) -> int {
    const int i = producer[x];
    if (i < 0) return -1;
    if (!is_conv(fused[i].kind) || uses[x] != 1 || g.tensors[x].output_index >= 0) return -1;
    return i;
  };

  for (size_t idx = 0; idx < g.ops.size(); ++idx) {
    const OpNode& op = g.ops[idx];
    if (dropped[idx]) continue;
    const int in_a = alias[op.d.inputs[0]], in_b = two_inputs(op) ? alias[op.d.inputs[1]] : -1;
    if (enable && op.d.kind == GI_OP_ACTIVATION) {
      const int i = foldable(in_a);
      const int pos = i >= 0 ? next_slot(fused[i].slot, 0) : -1;
      if (pos >= 0) {
        FusedOp& f = fused[i];
        (pos == 0 ? f.act_pre : f.act_post) = op.d.act;
        f.slot = pos + 1;
        producer[f.out] = -1;
        f.out = op.output;
        producer[op.output] = i;
        continue;
      }
    }
    if (enable && op.d.kind == GI_OP_ADD && in_b >= 0) {
      const int a = in_a, b = in_b;
      if (a != b) {
        int best = -1, best_x = -1, best_other = -1;
        const int pair[2][2] = {{a, b}, {b, a}};
        for (const auto& xo : pair) {
          const int x = xo[0], other = xo[1];
          const int i = foldable(x);
          if (i < 0 || next_slot(fused[i].slot, 1) < 0) continue;
          const bool ready = g.tensors[other].input_index >= 0 || (producer[other] >= 0 && producer[other] < i);
          if (ready && i > best) {
            best = i;
            best_x = x;
            best_other = other;
          }
        }
        if (best >= 0) {
          FusedOp& f = fused[best];
          f.residual = best_other;
          f.slot = 2;
          producer[best_x] = -1;
          f.out = op.output;
          producer[op.output] = best;
          continue;
        }
      }
    }
    FusedOp f;
    f.kind = op.d.kind;
    f.graph_op = static_cast<int>(idx);
    f.in0 = in_a;
    f.in1 = in_b;
    f.out = op.output;
    fused.push_back(f);
    producer[op.output] = static_cast<int>(fused.size()) - 1;
  }
  return GI_OK;
}

// ------------------------------------------------------------------------------ planning
static void reads_of(const FusedOp& f, int r[3]) {
  r[0] = f.in0;
  r[1] = f.in1;
  r[2] = f.residual;
}

// Section 5: for each intermediate tensor the first and the last executed op that uses it,
// as input or output.
static void compute_lifetimes(gi_exec* e) {
  for (size_t i = 0; i < e->ops.size(); ++i) {
    int r[3];
    reads_of(e->ops[i], r);
    const int touched[4] = {r[0], r[1], r[2], e->ops[i].out};
    for (int t : touched) {
      if (t < 0) continue;
      TensorPlan& p = e->plan[t];
      p.alive = 1;
      if (p.first < 0) p.first = static_cast<int>(i);
      p.last = static_cast<int>(i);
    }
  }
}

// Section 5 (a): no sharing; running sum in tensor-id order.
static uint64_t plan_naive(gi_exec* e) {
  uint64_t total = 0;
  for (TensorPlan& p : e->plan)
    if (p.intermediate) {
      p.offset = total;
      total += p.bytes;
    }
  return total;
}

// Algorithm 1 (Greedy Memory Management).  Per op: every intermediate output takes a shared
// object - a fresh one if the pool is empty, otherwise the pooled object closest in size
// (absolute difference; ties: larger, then older), grown when too small - and only afterwards
// the objects of intermediate inputs whose last consumer is this op go back to the pool.
// Objects are then laid out one after another in creation order.
static uint64_t plan_shared_objects(gi_exec* e) {
  struct Obj {
    uint64_t size;
  };
  std::vector<Obj> objs;
  std::vector<int> pool;
  std::vector<int> obj_of(e->plan.size(), -1);
  // a tensor placed inside another one (the input of a CONCAT that needs no copy) stands for that tensor,
  // which takes its object at the first op that writes any part of it
  auto holder = [&](int t) { return t >= 0 && e->plan[t].view_of >= 0 ? e->plan[t].view_of : t; };
  for (size_t i = 0; i < e->ops.size(); ++i) {
    const FusedOp& f = e->ops[i];
    const int out = holder(f.out);
    if (out >= 0 && e->plan[out].intermediate && obj_of[out] < 0) {
      const uint64_t need = e->plan[out].bytes;
      int s;
      if (pool.empty()) {
        objs.push_back({need});
        s = static_cast<int>(objs.size()) - 1;
      } else {
        size_t pick = 0;
        for (size_t k = 1; k < pool.size(); ++k) {
          const uint64_t dk = objs[pool[k]].size > need ? objs[pool[k]].size - need : need - objs[pool[k]].size;
          const uint64_t dp = objs[pool[pick]].size > need ? objs[pool[pick]].size - need : need - objs[pool[pick]].size;
          if (dk < dp || (dk == dp && (objs[pool[k]].size > objs[pool[pick]].size ||
                                       (objs[pool[k]].size == objs[pool[pick]].size && pool[k] < pool[pick]))))
            pick = k;
        }
        s = pool[pick];
        pool.erase(pool.begin() + static_cast<long>(pick));
        if (need > objs[s].size) objs[s].size = need;
      }
      obj_of[out] = s;
    }
    int r[3];
    reads_of(f, r);
    for (int k = 0; k < 3; ++k) r[k] = holder(r[k]);
    for (int k = 0; k < 3; ++k) {
      const int t = r[k];
      if (t < 0 || !e->plan[t].intermediate || e->plan[t].last != static_cast<int>(i)) continue;
      bool seen = false;
      for (int j = 0; j < k; ++j) seen = seen || r[j] == t;
      if (!seen) pool.push_back(obj_of[t]);
    }
  }
  std::vector<uint64_t> start(objs.size(), 0);
  uint64_t total = 0;
  for (size_t k = 0; k < objs.size(); ++k) {
    start[k] = total;
    total += objs[k].size;
  }
  for (size_t t = 0; t < e->plan.size(); ++t)
    if (obj_of[t] >= 0) e->plan[t].offset = start[obj_of[t]];
  return total;
}

// The Minimum-Cost Flow Algorithm (Section 5).  Intermediate tensors in execution order (first use, then
// id) are x = 1..N; the network has a source, a sink and vertices l_x, r_x; unit-capacity edges
//   1. s -> r_x, cost size_x (x opens a shared object),
//   2. l_x -> r_y, cost max(0, size_y - size_x), where x is dead before y is born (y takes over x's object),
//   3. s -> l_x and 4. r_x -> t, cost 0.
// The flow of value N and minimum cost is built one augmenting path at a time, each a shortest path found
// by the queue-based Bellman-Ford the paper names (SPFA): first-in first-out queue, edges in the order they
// were added (1, 2 by x then y, 3, 4), a distance replaced only by a strictly smaller one.  A saturated edge
// of type 2 hands x's object to y; an object is as large as its largest tensor; objects are laid out in the
// order their first tensors appear.
static uint64_t plan_min_cost_flow(gi_exec* e) {
  std::vector<int> ts;
  for (size_t t = 0; t < e->plan.size(); ++t)
    if (e->plan[t].intermediate) ts.push_back(static_cast<int>(t));
  std::stable_sort(ts.begin(), ts.end(), [&](int a, int b) { return e->plan[a].first < e->plan[b].first; });
  const int n = static_cast<int>(ts.size());
  const int src = 0, sink = 2 * n + 1, nv = 2 * n + 2;
  struct Edge {
    int to, cap;
    long long cost;
  };
  std::vector<Edge> edges;                  // edge 2k and its reverse 2k + 1
  std::vector<std::vector<int>> out(static_cast<size_t>(nv));
  auto add_edge = [&](int u, int v, long long c) {
    out[static_cast<size_t>(u)].push_back(static_cast<int>(edges.size()));
    edges.push_back({v, 1, c});
    out[static_cast<size_t>(v)].push_back(static_cast<int>(edges.size()));
    edges.push_back({u, 0, -c});
  };
  auto size_of = [&](int i) { return static_cast<long long>(e->plan[ts[static_cast<size_t>(i)]].bytes); };
  for (int i = 0; i < n; ++i) add_edge(src, 1 + n + i, size_of(i));
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j)
      if (e->plan[ts[static_cast<size_t>(i)]].last < e->plan[ts[static_cast<size_t>(j)]].first)
        add_edge(1 + i, 1 + n + j, std::max<long long>(0, size_of(j) - size_of(i)));
  for (int i = 0; i < n; ++i) add_edge(src, 1 + i, 0);
  for (int i = 0; i < n; ++i) add_edge(1 + n + i, sink, 0);
  const long long kInf = std::numeric_limits<long long>::max();
  std::vector<long long> dist(static_cast<size_t>(nv));
  std::vector<int> via(static_cast<size_t>(nv));
  std::vector<char> queued(static_cast<size_t>(nv));
  for (;;) {
    std::fill(dist.begin(), dist.end(), kInf);
    std::fill(via.begin(), via.end(), -1);
    std::fill(queued.begin(), queued.end(), 0);
    std::deque<int> queue;
    dist[src] = 0;
    queue.push_back(src);
    while (!queue.empty()) {
      const int u = queue.front();
      queue.pop_front();
      queued[static_cast<size_t>(u)] = 0;
      for (int id : out[static_cast<size_t>(u)]) {
        const Edge& ed = edges[static_cast<size_t>(id)];
        if (ed.cap > 0 && dist[static_cast<size_t>(u)] + ed.cost < dist[static_cast<size_t>(ed.to)]) {
          dist[static_cast<size_t>(ed.to)] = dist[static_cast<size_t>(u)] + ed.cost;
          via[static_cast<size_t>(ed.to)] = id;
          if (!queued[static_cast<size_t>(ed.to)]) {
            queued[static_cast<size_t>(ed.to)] = 1;
            queue.push_back(ed.to);
          }
        }
      }
    }
    if (dist[static_cast<size_t>(sink)] == kInf) break;
    for (int v = sink; v != src;) {
      const int id = via[static_cast<size_t>(v)];
      edges[static_cast<size_t>(id)].cap -= 1;
      edges[static_cast<size_t>(id ^ 1)].cap += 1;
      v = edges[static_cast<size_t>(id ^ 1)].to;
    }
  }
  std::vector<int> donor(static_cast<size_t>(n), -1);
  for (int i = 0; i < n; ++i)
    for (int id : out[static_cast<size_t>(1 + i)])
      if (id % 2 == 0 && edges[static_cast<size_t>(id)].cap == 0) donor[static_cast<size_t>(edges[static_cast<size_t>(id)].to - 1 - n)] = i;
  std::vector<int> obj(static_cast<size_t>(n), -1);
  std::vector<uint64_t> sizes;
  for (int j = 0; j < n; ++j) {  // a donor is dead before its heir is born: it comes earlier in the order
    const uint64_t need = e->plan[ts[static_cast<size_t>(j)]].bytes;
    if (donor[static_cast<size_t>(j)] >= 0) {
      obj[static_cast<size_t>(j)] = obj[static_cast<size_t>(donor[static_cast<size_t>(j)])];
      uint64_t& sz = sizes[static_cast<size_t>(obj[static_cast<size_t>(j)])];
      if (need > sz) sz = need;
    } else {
      obj[static_cast<size_t>(j)] = static_cast<int>(sizes.size());
      sizes.push_back(need);
    }
  }
  std::vector<uint64_t> start(sizes.size(), 0);
  uint64_t total = 0;
  for (size_t k = 0; k < sizes.size(); ++k) {
    start[k] = total;
    total += sizes[k];
  }
  for (int j = 0; j < n; ++j) e->plan[ts[static_cast<size_t>(j)]].offset = start[static_cast<size_t>(obj[static_cast<size_t>(j)])];
  return total;
}

// Greedy by size: largest tensor first (ties: earlier first use, smaller id).  Among the
// tensors already placed whose lifetime intersects, scan the free gaps from offset 0 upward
// and take the smallest that fits (ties: lowest offset); otherwise append after them.
static uint64_t plan_by_size(gi_exec* e) {
  std::vector<int> order;
  for (size_t t = 0; t < e->plan.size(); ++t)
    if (e->plan[t].intermediate) order.push_back(static_cast<int>(t));
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    const TensorPlan &pa = e->plan[a], &pb = e->plan[b];
    if (pa.bytes != pb.bytes) return pa.bytes > pb.bytes;
    if (pa.first != pb.first) return pa.first < pb.first;
    return a < b;
  });
  std::vector<int> placed;
  uint64_t total = 0;
  for (int t : order) {
    TensorPlan& p = e->plan[t];
    std::vector<std::pair<uint64_t, uint64_t>> busy;
    for (int u : placed) {
      const TensorPlan& q = e->plan[u];
      if (q.last < p.first || p.last < q.first) continue;
      busy.emplace_back(q.offset, q.offset + q.bytes);
    }
    std::sort(busy.begin(), busy.end());
    uint64_t cursor = 0, best_gap = 0, best_off = 0;
    bool found = false;
    for (const auto& iv : busy) {
      if (iv.first > cursor) {
        const uint64_t gap = iv.first - cursor;
        if (gap >= p.bytes && (!found || gap < best_gap)) {
          found = true;
          best_gap = gap;
          best_off = cursor;
        }
      }
      cursor = std::max(cursor, iv.second);
    }
    p.offset = found ? best_off : cursor;
    total = std::max(total, p.offset + p.bytes);
    placed.push_back(t);
  }
  return total;
}

// Concatenations that need no copy.  The slices of a tensor follow one another in memory (Section 4), so
// concat(a, b) with C(a) a multiple of 4 is a's slices followed by b's: a and b are placed inside the result
// and their producers write the result directly; the CONCAT itself launches nothing.  Eligible (walked in
// execution order): two different inputs, C(a) % 4 == 0, none of a, b, out is a graph input or output, and
// neither a nor b is already placed inside another tensor or holds tensors itself.
static void find_concat_views(gi_exec* e) {
  std::vector<char> is_root(e->tensors.size(), 0);
  auto io = [&](int t) { return e->tensors[t].input_index >= 0 || e->tensors[t].output_index >= 0; };
  for (const FusedOp& f : e->ops) {
    if (f.kind != GI_OP_CONCAT || f.in1 < 0) continue;
    const int a = f.in0, b = f.in1, out = f.out;
    if (a == b || e->tensors[a].c % 4 != 0 || io(a) || io(b) || io(out)) continue;
    if (e->plan[a].view_of >= 0 || e->plan[b].view_of >= 0 || is_root[a] || is_root[b]) continue;
    e->plan[a].view_of = out;
    e->plan[a].view_slice = 0;
    e->plan[b].view_of = out;
    e->plan[b].view_slice = e->tensors[a].c / 4;
    is_root[out] = 1;
  }
}

gi_status plan_memory(gi_exec* e) {
  const uint64_t align = static_cast<uint64_t>(e->opt.align);
  for (size_t t = 0; t < e->tensors.size(); ++t) {
    const TensorDesc& d = e->tensors[t];
    e->plan[t].bytes = gi_tensor_bytes(e->batch, d.h, d.w, d.c, e->storage, static_cast<int32_t>(align));
  }
  if (e->opt.fuse) find_concat_views(e);
  compute_lifetimes(e);
  // a tensor that holds others is in use whenever one of them is
  for (size_t t = 0; t < e->tensors.size(); ++t) {
    const TensorPlan& v = e->plan[t];
    if (v.view_of < 0 || !v.alive) continue;
    TensorPlan& r = e->plan[v.view_of];
    r.first = std::min(r.first, v.first);
    r.last = std::max(r.last, v.last);
  }
  for (size_t t = 0; t < e->tensors.size(); ++t) {
    const TensorDesc& d = e->tensors[t];
    TensorPlan& p = e->plan[t];
    // caller-owned PHWC4 inputs / outputs are not planned, nor is a tensor placed inside another one;
    // everything else that is alive is
    const bool callers = (d.input_index >= 0 && d.input_layout == GI_PHWC4) ||
                         (d.output_index >= 0 && d.output_layout == GI_PHWC4);
    p.intermediate = p.alive && !callers && p.view_of < 0;
  }
  e->naive_bytes = 0;
  for (const TensorPlan& p : e->plan)
    if (p.intermediate) e->naive_bytes += p.bytes;
  e->lower_bound = 0;
  for (size_t i = 0; i < e->ops.size(); ++i) {
    uint64_t live = 0;
    for (const TensorPlan& p : e->plan)
      if (p.intermediate && p.first <= static_cast<int>(i) && static_cast<int>(i) <= p.last) live += p.bytes;
    e->lower_bound = std::max(e->lower_bound, live);
  }
  switch (e->opt.planner) {
    case GI_PLAN_NAIVE: e->arena_bytes = plan_naive(e); break;
    case GI_PLAN_GREEDY_SHARED_OBJECTS: e->arena_bytes = plan_shared_objects(e); break;
    case GI_PLAN_GREEDY_BY_SIZE: e->arena_bytes = plan_by_size(e); break;
    case GI_PLAN_MIN_COST_FLOW: e->arena_bytes = plan_min_cost_flow(e); break;
    default: return fail(GI_E_INVALID, "gi_compile: unknown planner");
  }
  // tensors placed inside another one: their slices start `view_slice` slices into it
  for (size_t t = 0; t < e->tensors.size(); ++t) {
    TensorPlan& v = e->plan[t];
    if (v.view_of < 0 || !v.alive) continue;
    const TensorDesc& d = e->tensors[t];
    const uint64_t slice_bytes = static_cast<uint64_t>(e->batch) * plane_pixels(d.h, d.w) * 4 * elem_bytes(e->storage);
    v.offset = e->plan[v.view_of].offset + static_cast<uint64_t>(v.view_slice) * slice_bytes;
    v.intermediate = 2;
  }
  return GI_OK;
}

}  // namespace gi

using namespace gi;

extern "C" {

gi_status gi_compile(const gi_graph* g, const gi_compile_options* opt, gi_exec** out) {
  if (!g || !out) return fail(GI_E_INVALID, "gi_compile: null argument");
  *out = nullptr;
  if (g->inputs.empty() || g->outputs.empty()) return fail(GI_E_INVALID, "gi_compile: graph needs an input and an output");
  gi_compile_options o{};
  o.planner = GI_PLAN_GREEDY_BY_SIZE;
  o.fuse = 1;
  o.align = 256;
  o.pointwise = GI_PW_AUTO;
  o.cross_op = GI_XOP_AUTO;
  if (opt) {
    o = *opt;
    if (o.align == 0) o.align = 256;
  }
  if (o.align < 256 || (o.align & (o.align - 1))) return fail(GI_E_INVALID, "gi_compile: align must be a power of two >= 256");
  if (o.pointwise < GI_PW_AUTO || o.pointwise > GI_PW_RULE) return fail(GI_E_INVALID, "gi_compile: unknown pointwise option");
  if (o.cross_op < GI_XOP_AUTO || o.cross_op > GI_XOP_CHAIN) return fail(GI_E_INVALID, "gi_compile: unknown cross_op option");
  gi_exec* e = nullptr;
  try {
    e = new gi_exec();
    e->batch = g->batch;
    e->storage = g->storage;
    e->opt = o;
    e->tensors = g->tensors;
    e->plan.assign(g->tensors.size(), TensorPlan());
    e->n_inputs = static_cast<int>(g->inputs.size());
    e->n_outputs = static_cast<int>(g->outputs.size());
    std::vector<FusedOp> fused;
    gi_status s = fuse_graph(*g, o.fuse != 0, &fused);
    if (s != GI_OK) {
      delete e;
      return s;
    }
    // a tensor that no op produces and that is not a graph input cannot be read
    e->n_fused = static_cast<int>(fused.size());
    // executed ops: layout conversions for NHWC inputs, the fused ops, conversions for NHWC outputs
    for (int k = 0; k < e->n_inputs; ++k) {
      const int t = g->inputs[k];
      if (g->tensors[t].input_layout != GI_NHWC) continue;
      FusedOp p;
      p.kind = GI_EXEC_PACK;
      p.out = t;
      p.io_index = k;
      e->ops.push_back(p);
    }
    e->ops.insert(e->ops.end(), fused.begin(), fused.end());
    for (int k = 0; k < e->n_outputs; ++k) {
      const int t = g->outputs[k];
      if (g->tensors[t].output_layout != GI_NHWC) continue;
      FusedOp p;
      p.kind = GI_EXEC_UNPACK;
      p.in0 = t;
      p.io_index = k;
      e->ops.push_back(p);
    }
    s = plan_memory(e);
    if (s == GI_OK) s = lower(*g, e);
    if (s != GI_OK) {
      delete e;
      return s;
    }
  } catch (const std::bad_alloc&) {
    delete e;
    return fail(GI_E_NOMEM, "gi_compile: out of host memory");
  }
  *out = e;
  return GI_OK;
}

void gi_exec_destroy(gi_exec* e) {
  if (!e) return;
  release_run_state(e);
  delete e;
}

gi_status gi_exec_query(const gi_exec* e, gi_exec_info* info) {
  if (!e || !info) return fail(GI_E_INVALID, "gi_exec_query: null argument");
  std::memset(info, 0, sizeof *info);
  info->n_ops = static_cast<int32_t>(e->ops.size());
  info->n_fused_ops = e->n_fused;
  info->n_tensors = static_cast<int32_t>(e->tensors.size());
  info->batch = e->batch;
  info->storage = e->storage;
  info->arena_bytes = e->arena_bytes;
  info->naive_bytes = e->naive_bytes;
  info->lower_bound_bytes = e->lower_bound;
  info->weight_bytes = e->weight_blob.size();
  return GI_OK;
}

gi_status gi_exec_tensor(const gi_exec* e, gi_tensor t, gi_tensor_info* info) {
  if (!e || !info) return fail(GI_E_INVALID, "gi_exec_tensor: null argument");
  if (t < 0 || t >= static_cast<int>(e->tensors.size())) return fail(GI_E_INVALID, "gi_exec_tensor: unknown tensor");
  std::memset(info, 0, sizeof *info);
  const TensorDesc& d = e->tensors[t];
  const TensorPlan& p = e->plan[t];
  info->h = d.h;
  info->w = d.w;
  info->c = d.c;
  info->alive = p.alive;
  info->intermediate = p.intermediate;
  info->first_op = p.alive ? p.first : -1;
  info->last_op = p.alive ? p.last : -1;
  info->bytes = p.bytes;
  info->offset = p.intermediate ? p.offset : 0;
  return GI_OK;
}

gi_status gi_exec_op(const gi_exec* e, int32_t index, gi_op_info* info) {
  if (!e || !info) return fail(GI_E_INVALID, "gi_exec_op: null argument");
  if (index < 0 || index >= static_cast<int>(e->op_info.size())) return fail(GI_E_INVALID, "gi_exec_op: index out of range");
  *info = e->op_info[index];
  return GI_OK;
}

}  // extern "C"
