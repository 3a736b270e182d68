// Lowering: choose a kernel per executed op, pack its weights into the kernel's operand
// layout (fp16 storage: weights rounded to fp16 once, biases stay fp32) and record the
// launch geometry.  Host work only.
#include <cstdlib>
#include <cstring>

#include "gi_internal.h"
#include "kernels.h"

namespace gi {

static float as_storage(float v, int storage) {
  if (storage == GI_F32) return v;
  // value the weight has after being stored as fp16
  const uint16_t h = f32_to_f16_rne(v);
  const uint32_t s = (h & 0x8000u) << 16, e = (h >> 10) & 0x1fu, m = h & 0x3ffu;
  uint32_t u;
  float r;
  if (e == 0) {
    r = static_cast<float>(m) * (1.0f / 16777216.0f);
    std::memcpy(&u, &r, 4);
  } else if (e == 31) {
    u = 0x7f800000u | (m << 13);
  } else {
    u = ((e + 112u) << 23) | (m << 13);
  }
  u |= s;
  std::memcpy(&r, &u, 4);
  return r;
}

static uint64_t blob_reserve(std::vector<uint8_t>* blob, uint64_t bytes) {
  const uint64_t off = round_up_u64(blob->size(), 256);
  blob->resize(off + bytes, 0);
  return off;
}

static Loc loc_of(const gi_exec* e, int t) {
  Loc l;
  if (t < 0) return l;
  const TensorDesc& d = e->tensors[t];
  if (d.input_index >= 0 && d.input_layout == GI_PHWC4) {
    l.where = W_INPUT;
    l.index = d.input_index;
  } else if (d.output_index >= 0 && d.output_layout == GI_PHWC4) {
    l.where = W_OUTPUT;
    l.index = d.output_index;
  } else {
    l.where = W_ARENA;
    l.offset = e->plan[t].offset;
  }
  return l;
}

// Weights of the CUDA-core convolution kernel: float W[group][tap][in_slice][OS*4 co][4 ci],
// a group being OS consecutive output slices; entries beyond Cin / Cout are zero.
static void pack_conv_simt(const OpNode& op, int cin, int storage, int os, std::vector<uint8_t>* blob, LaunchRec* r) {
  const int taps = op.d.kh * op.d.kw, sin = slices(cin), sout = slices(op.d.cout);
  const int groups = (sout + os - 1) / os, jn = os * 4;
  const uint64_t nw = static_cast<uint64_t>(groups) * taps * sin * jn * 4;
  const uint64_t woff = blob_reserve(blob, nw * sizeof(float));
  const uint64_t boff = blob_reserve(blob, static_cast<uint64_t>(groups) * jn * sizeof(float));
  float* w = reinterpret_cast<float*>(blob->data() + woff);
  float* b = reinterpret_cast<float*>(blob->data() + boff);
  for (int g = 0; g < groups; ++g)
    for (int j = 0; j < jn; ++j) {
      const int co = g * jn + j;
      if (co >= op.d.cout) continue;
      b[g * jn + j] = op.bias[co];
      for (int tap = 0; tap < taps; ++tap)
        for (int ci = 0; ci < cin; ++ci) {
          const float v = op.weights[(static_cast<size_t>(co) * taps + tap) * cin + ci];
          w[(((static_cast<size_t>(g) * taps + tap) * sin + ci / 4) * jn + j) * 4 + ci % 4] = as_storage(v, storage);
        }
    }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = nw * sizeof(float);
}

// Depthwise: float W[tap][C4], bias[C4].
static void pack_depthwise(const OpNode& op, int c, int storage, std::vector<uint8_t>* blob, LaunchRec* r) {
  const int taps = op.d.kh * op.d.kw, c4 = slices(c) * 4;
  const uint64_t woff = blob_reserve(blob, static_cast<uint64_t>(taps) * c4 * sizeof(float));
  const uint64_t boff = blob_reserve(blob, static_cast<uint64_t>(c4) * sizeof(float));
  float* w = reinterpret_cast<float*>(blob->data() + woff);
  float* b = reinterpret_cast<float*>(blob->data() + boff);
  for (int ch = 0; ch < c; ++ch) {
    b[ch] = op.bias[ch];
    for (int tap = 0; tap < taps; ++tap) w[tap * c4 + ch] = as_storage(op.weights[static_cast<size_t>(tap) * c + ch], storage);
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = static_cast<uint64_t>(taps) * c4 * sizeof(float);
}

// The executed op after depthwise op `i` is a 1x1 convolution that is the only reader of the depthwise
// output, that output is an arena tensor, and the pair's input and output do not share memory: the pair
// may run as one kernel.
static bool pointwise_follows(const gi_graph& g, const gi_exec* e, size_t i) {
  if (i + 1 >= e->ops.size()) return false;
  const FusedOp& f = e->ops[i];
  const FusedOp& n = e->ops[i + 1];
  if (f.kind != GI_OP_DEPTHWISE_CONV2D || n.kind != GI_OP_CONV2D) return false;
  if (f.residual >= 0 || f.act_post != GI_ACT_NONE || f.out < 0) return false;
  if (n.in0 != f.out || n.in1 == f.out || n.residual == f.out) return false;
  const TensorPlan& tp = e->plan[f.out];
  if (!tp.intermediate || tp.first != static_cast<int>(i) || tp.last != static_cast<int>(i + 1)) return false;
  if (e->tensors[f.out].output_index >= 0) return false;
  // One kernel reads the depthwise input while it writes the 1x1 convolution's output.  As separate ops their
  // lifetimes do not meet, so the planner may have given them the same arena bytes: then the pair stays two kernels.
  const TensorPlan& pin = e->plan[f.in0];
  const TensorPlan& pout = e->plan[n.out];
  if (loc_of(e, f.in0).where == W_ARENA && loc_of(e, n.out).where == W_ARENA && pin.offset < pout.offset + pout.bytes &&
      pout.offset < pin.offset + pin.bytes)
    return false;
  const gi_op_desc& d = g.ops[n.graph_op].d;
  return d.kh == 1 && d.kw == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_t == 0 && d.pad_l == 0 && d.pad_b == 0 &&
         d.pad_r == 0;
}

// Launch table: the fastest 1x1 kernel per shape as measured on the device (generated; the analogue of the paper's
// table of optimal work-group sizes, Section 4).  Consulted before the rule below; shapes that are not in it - any
// network other than the benchmark ones - take the rule.
struct LaunchChoice {
  long long px;
  int cin, cout, kernel;
  float ms_pair, ms_lane, ms_wide;
};
static const LaunchChoice kLaunchTable[] = {
    {0, 0, 0, 0, 0.f, 0.f, 0.f},  // keeps the array non-empty when the table has not been generated
#include "launch_table.inc"
};
static const LaunchChoice* launch_table_lookup(long long px, int cin, int cout) {
  for (const LaunchChoice& c : kLaunchTable)
    if (c.px == px && c.cin == cin && c.cout == cout && c.kernel != 0) return &c;
  return nullptr;
}

// The same for the staged depthwise stencil: how large a staging buffer may be and how much shared memory a CTA takes
// (which together decide planes per work item, buffers in flight and CTAs per SM), per depthwise shape of the
// benchmark networks, as measured by the tuner.  Shapes that are not in the table run with the kernel's defaults.
struct DwChoice {
  int batch, h, w, c, stride, buf_kb, cta_kb;
  float ms_default, ms_best;
};
static const DwChoice kDwTable[] = {
    {0, 0, 0, 0, 0, 0, 0, 0.f, 0.f},  // keeps the array non-empty when the table has not been generated
#include "dw_table.inc"
};
static const DwChoice* dw_table_lookup(int batch, int h, int w, int c, int stride) {
  for (const DwChoice& d : kDwTable)
    if (d.batch == batch && d.h == h && d.w == w && d.c == c && d.stride == stride && d.batch != 0) return &d;
  return nullptr;
}

// pixels of a 1x1 convolution's input as the kernels count them: batch x stored plane
static long long m_px_all_for_mm(const gi_exec* e, const TensorDesc* t) {
  return static_cast<long long>(e->batch) * plane_pixels(t->h, t->w);
}

static bool is_plain_pointwise(const gi_op_desc& d) {
  return d.kh == 1 && d.kw == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_t == 0 && d.pad_l == 0 && d.pad_b == 0 && d.pad_r == 0;
}

// A tensor written by executed op `i`, read by op `i + 1` and by nothing else, living in the arena: one that a kernel
// running both ops never has to store.
static bool private_between(const gi_exec* e, int t, size_t i) {
  if (t < 0) return false;
  const TensorPlan& tp = e->plan[t];
  return tp.intermediate == 1 && tp.first == static_cast<int>(i) && tp.last == static_cast<int>(i + 1) &&
         e->tensors[t].output_index < 0 && e->tensors[t].input_index < 0;
}

// Executed ops i, i + 1, i + 2 are the three convolutions of an inverted-residual block - 1x1 expansion, depthwise
// 3x3, 1x1 projection (with or without the residual sum) - and the two tensors between them have no other reader, so
// that one kernel may run all three and keep those tensors on chip.
static bool block_follows(const gi_graph& g, const gi_exec* e, size_t i) {
  if (i + 2 >= e->ops.size()) return false;
  const FusedOp& a = e->ops[i];
  const FusedOp& b = e->ops[i + 1];
  const FusedOp& c = e->ops[i + 2];
  if (a.kind != GI_OP_CONV2D || b.kind != GI_OP_DEPTHWISE_CONV2D || c.kind != GI_OP_CONV2D) return false;
  if (a.residual >= 0 || a.act_post != GI_ACT_NONE || b.residual >= 0 || b.act_post != GI_ACT_NONE) return false;
  if (b.in0 != a.out || c.in0 != b.out || c.residual == a.out || c.residual == b.out) return false;
  if (!private_between(e, a.out, i) || !private_between(e, b.out, i + 1)) return false;
  if (!is_plain_pointwise(g.ops[a.graph_op].d) || !is_plain_pointwise(g.ops[c.graph_op].d)) return false;
  const gi_op_desc& d = g.ops[b.graph_op].d;
  if (d.stride_h != d.stride_w || d.dilation_h != 1 || d.dilation_w != 1) return false;
  // One kernel reads the block's input while it writes the block's output.  Without a residual the two never live
  // at the same op, so the planner may have given them the same arena bytes: then the block stays three kernels.
  const TensorPlan& pin = e->plan[a.in0];
  const TensorPlan& pout = e->plan[c.out];
  if (loc_of(e, a.in0).where == W_ARENA && loc_of(e, c.out).where == W_ARENA && pin.offset < pout.offset + pout.bytes &&
      pout.offset < pin.offset + pin.bytes)
    return false;
  return true;
}

// Two tensors that both live in the arena and share at least one byte.
static bool arena_overlap(const gi_exec* e, int t1, int t2) {
  if (t1 < 0 || t2 < 0) return false;
  const Loc a = loc_of(e, t1), b = loc_of(e, t2);
  if (a.where != W_ARENA || b.where != W_ARENA) return false;
  return a.offset < b.offset + e->plan[t2].bytes && b.offset < a.offset + e->plan[t1].bytes;
}

// Executed ops i and i + 1 are plain 1x1 convolutions, the second reads the first one's output and has neither a
// residual nor a second activation: one kernel may run both, storing both outputs (the first output may have any
// number of other readers).  As separate ops the first op's input and residual may die before the second op's output is
// born, so the planner may have put that output on their bytes; one kernel reads them while it writes it - such a
// pair stays two kernels.
static bool chain_follows(const gi_graph& g, const gi_exec* e, size_t i) {
  if (i + 1 >= e->ops.size()) return false;
  const FusedOp& a = e->ops[i];
  const FusedOp& b = e->ops[i + 1];
  if (a.kind != GI_OP_CONV2D || b.kind != GI_OP_CONV2D || a.out < 0 || b.out < 0) return false;
  if (b.in0 != a.out || b.residual >= 0 || b.act_post != GI_ACT_NONE) return false;
  if (!is_plain_pointwise(g.ops[a.graph_op].d) || !is_plain_pointwise(g.ops[b.graph_op].d)) return false;
  if (arena_overlap(e, a.in0, b.out) || arena_overlap(e, a.residual, b.out)) return false;
  return true;
}

// The executed op that converts graph input `t` from NHWC, if executed op `reader` is the only op that reads
// the converted tensor (and it is not also a graph output); else -1.
static int nhwc_pack_feeding_only(const gi_exec* e, int t, size_t reader) {
  if (t < 0) return -1;
  const TensorDesc& d = e->tensors[t];
  if (d.input_index < 0 || d.input_layout != GI_NHWC || d.output_index >= 0) return -1;
  int pack = -1;
  for (size_t j = 0; j < e->ops.size(); ++j) {
    const FusedOp& o = e->ops[j];
    if (o.kind == GI_EXEC_PACK && o.out == t) pack = static_cast<int>(j);
    if (j != reader && (o.in0 == t || o.in1 == t || o.residual == t)) return -1;
  }
  const FusedOp& r = e->ops[reader];
  if (r.in1 == t || r.residual == t) return -1;
  return pack;
}

gi_status lower(const gi_graph& g, gi_exec* e) {
  const int eb = elem_bytes(e->storage);
  const uint64_t B = static_cast<uint64_t>(e->batch);
  int absorbed = 0;  // this many following ops run inside the kernel of an op already lowered
  for (size_t i = 0; i < e->ops.size(); ++i) {
    const FusedOp& f = e->ops[i];
    LaunchRec r;
    gi_op_info info{};
    info.kind = f.kind;
    info.graph_op = f.graph_op;
    info.inputs[0] = f.in0;
    info.inputs[1] = f.in1;
    info.residual = f.residual;
    info.output = f.out;
    info.act_pre = f.act_pre;
    info.act_post = f.act_post;
    r.B = e->batch;
    r.ep.act_pre = f.act_pre;
    r.ep.has_res = f.residual >= 0;
    r.ep.act_post = f.act_post;
    const TensorDesc* din = f.in0 >= 0 ? &e->tensors[f.in0] : nullptr;
    const TensorDesc* dout = f.out >= 0 ? &e->tensors[f.out] : nullptr;
    if (din) {
      r.H = din->h;
      r.W = din->w;
      r.C = din->c;
    }
    if (dout) {
      r.Ho = dout->h;
      r.Wo = dout->w;
      r.Co = dout->c;
    }
    if (f.in0 >= 0 && f.in0 != f.in1 && f.in0 != f.residual)
      r.in0_dead = e->plan[f.in0].last == static_cast<int>(i) && e->tensors[f.in0].output_index < 0;
    r.in0 = loc_of(e, f.in0);
    r.in1 = loc_of(e, f.in1);
    r.res = loc_of(e, f.residual);
    r.out = loc_of(e, f.out);
    const uint64_t in_px = din ? B * din->h * din->w : 0, out_px = dout ? B * dout->h * dout->w : 0;
    const uint64_t in_c4 = din ? slices(din->c) * 4 : 0, out_c4 = dout ? slices(dout->c) * 4 : 0;
    switch (f.kind) {
      case GI_EXEC_PACK: {
        r.kernel = GI_KERNEL_PACK;
        r.in0 = Loc{W_INPUT, f.io_index, 0};
        r.H = dout->h;
        r.W = dout->w;
        r.C = dout->c;
        info.bytes = out_px * dout->c * eb + out_px * out_c4 * eb;
        break;
      }
      case GI_EXEC_UNPACK: {
        r.kernel = GI_KERNEL_UNPACK;
        r.out = Loc{W_OUTPUT, f.io_index, 0};
        info.bytes = in_px * in_c4 * eb + in_px * din->c * eb;
        break;
      }
      case GI_OP_CONV2D:
      case GI_OP_DEPTHWISE_CONV2D: {
        const OpNode& op = g.ops[f.graph_op];
        r.kh = op.d.kh;
        r.kw = op.d.kw;
        r.sh = op.d.stride_h;
        r.sw = op.d.stride_w;
        r.dh = op.d.dilation_h;
        r.dw = op.d.dilation_w;
        r.pt = op.d.pad_t;
        r.pl = op.d.pad_l;
        const uint64_t taps = static_cast<uint64_t>(op.d.kh) * op.d.kw;
        info.bytes = (in_px * in_c4 + out_px * out_c4 * (r.ep.has_res ? 2 : 1)) * eb;
        if (absorbed > 0) {
          // an earlier op's kernel computes this convolution too; its bytes and flops are counted there
          --absorbed;
          r.kernel = GI_KERNEL_NONE;
          info.bytes = 0;
        } else if (f.kind == GI_OP_DEPTHWISE_CONV2D) {
          r.kernel = GI_KERNEL_DEPTHWISE;
          r.C = din->c;
          if (op.d.dilation_h == 1 && op.d.stride_h == op.d.stride_w) {
            // (GI_DW_BUF_KB / GI_DW_CTA_KB in the environment of gi_compile override the table: the tuner's hook)
            const char* ebuf = getenv("GI_DW_BUF_KB");
            const char* ecta = getenv("GI_DW_CTA_KB");
            if (ebuf || ecta) {
              r.dw_buf_kb = ebuf ? atoi(ebuf) : 0;
              r.dw_cta_kb = ecta ? atoi(ecta) : 0;
            } else if (const DwChoice* dc = dw_table_lookup(e->batch, din->h, din->w, din->c, op.d.stride_h)) {
              r.dw_buf_kb = dc->buf_kb;
              r.dw_cta_kb = dc->cta_kb;
            }
          }
          r.dw_staged = e->storage == GI_F16 && depthwise_f16_supported(r);
          if (!r.dw_staged && (r.dw_buf_kb || r.dw_cta_kb)) {
            // not with these sizes: the kernel's own
            r.dw_buf_kb = r.dw_cta_kb = 0;
            r.dw_staged = e->storage == GI_F16 && depthwise_f16_supported(r);
          }
          if (!r.dw_staged && e->batch > 65535)
            return fail(GI_E_UNSUPPORTED, "gi_compile: depthwise convolution: batch above 65535 with a shape only the plain kernel runs");
          pack_depthwise(op, din->c, e->storage, &e->weight_blob, &r);
          info.bytes += taps * din->c * eb;
          info.flops = 2 * taps * out_px * din->c;
          if (e->storage == GI_F16 && e->opt.cross_op == GI_XOP_ON && pointwise_follows(g, e, i) &&
              depthwise_pointwise_supported(r, g.ops[e->ops[i + 1].graph_op].d.cout, nullptr, nullptr)) {
            // (GI_XOP_AUTO never takes this path yet: on every depthwise -> projection pair of MobileNetV2 at
            // batch 256 the single kernel measured between 4 % faster and 30 % slower than the two kernels; its
            // stencil half is bound by instruction issue, which the two-kernel path spreads over more warps)
            // one kernel for both: reads the depthwise input, writes the 1x1 convolution's output
            const FusedOp& n = e->ops[i + 1];
            const OpNode& pw = g.ops[n.graph_op];
            const TensorDesc& d2 = e->tensors[n.out];
            r.kernel = GI_KERNEL_DEPTHWISE_POINTWISE;
            depthwise_pointwise_pack(pw.weights.data(), pw.bias.data(), din->c, pw.d.cout, din->w, &e->weight_blob, &r);
            r.Co2 = pw.d.cout;
            r.ep2.act_pre = n.act_pre;
            r.ep2.has_res = n.residual >= 0;
            r.ep2.act_post = n.act_post;
            r.out = loc_of(e, n.out);
            r.res = loc_of(e, n.residual);
            const uint64_t px2 = B * d2.h * d2.w, c42 = slices(d2.c) * 4;
            info.bytes = (in_px * in_c4 + px2 * c42 * (r.ep2.has_res ? 2 : 1) + taps * din->c +
                          static_cast<uint64_t>(din->c) * pw.d.cout) * eb;
            info.flops += 2 * px2 * din->c * pw.d.cout;
            absorbed = 1;
          }
        } else {
          const bool pointwise = op.d.kh == 1 && op.d.stride_h == 1 && op.d.stride_w == 1 && op.d.pad_t == 0 &&
                                 op.d.pad_l == 0 && op.d.pad_b == 0 && op.d.pad_r == 0;
          const bool tc = e->storage == GI_F16 && e->opt.pointwise != GI_PW_SIMT;
          // Which tensor-core kernel: a rule distilled from measurements of the kernels on every 1x1 shape of
          // the benchmark networks (single launches whose input was written just before, as a producing kernel
          // leaves it, and confirmed inside the networks).  The lane-per-pixel kernel (dense weights, activations
          // through tensor memory) wins for 24 <= Cin < 960 with at least 96 output channels - the expansion layers
          // 24 -> 144, 32 -> 192 and 96 -> 576 included: with their input cold the pixel-pair kernel measured 8 % ahead
          // there, inside MobileNetV2, where the projection before them has just written it, the lane kernel is
          // 1.8 % of the whole step faster (1.450 -> 1.424 ms at batch 256); the pixel-pair kernel (both operands by
          // TMA, 4x expanded weights) wins elsewhere: few input or output channels, where its tiles are small,
          // and very deep inputs, where the lane kernel's weights no longer stay resident.
          // Launches whose pixels all fit one wave of 128-pixel tiles are latency-bound and take the lane
          // kernel (shorter fill; MobileNetV2 batch 1 0.296 -> 0.276 ms) - up to 64 tiles always, up to one
          // tile per SM unless the input is 960 channels deep or more.
          // Whole inverted-residual block as one kernel: only on request (GI_XOP_ON).  The library's own choice
          // (GI_XOP_AUTO) follows A/Bs of MobileNetV2 at batch 256 on one B200.  With the 14x14 blocks as one kernel each
          // the step is 2.5 % slower (alone, L2 flushed, a 14x14 block takes 55-88 us as one kernel against 48-65 us as
          // three).  The two 7x7 blocks that qualify were a tie (1.549 against 1.552 ms) until the 1x1 kernels around
          // them got faster - the CTA-pair kernel on 960 -> 160, the lane-per-pixel kernel's drain on 160 -> 960; now
          // three kernels per block win: 1.450 ms against 1.469 ms with the blocks fused (55 us each, bound by their own
          // instruction stream).
          long long ir_units = 0;
          if (pointwise && tc && e->opt.fuse && e->opt.cross_op != GI_XOP_OFF && block_follows(g, e, i)) {
            const FusedOp& fd = e->ops[i + 1];
            const FusedOp& fp = e->ops[i + 2];
            const OpNode& dwn = g.ops[fd.graph_op];
            const OpNode& pwn = g.ops[fp.graph_op];
            const TensorDesc& dd = e->tensors[fd.out];
            if (inverted_residual_supported(e->batch, din->h, din->w, dd.h, dd.w, dwn.d.stride_h, dwn.d.dilation_h, dwn.d.pad_t,
                                            dwn.d.pad_l, din->c, op.d.cout, pwn.d.cout, &ir_units) &&
                e->opt.cross_op == GI_XOP_ON) {
              const TensorDesc& d2 = e->tensors[fp.out];
              r.kernel = GI_KERNEL_INVERTED_RESIDUAL;
              r.Ho = dd.h;
              r.Wo = dd.w;
              r.sh = r.sw = dwn.d.stride_h;
              r.pt = dwn.d.pad_t;
              r.pl = dwn.d.pad_l;
              r.kh = r.kw = 3;
              r.Cmid = op.d.cout;
              r.Co2 = pwn.d.cout;
              r.ep_mid.act_pre = fd.act_pre;
              r.ep2.act_pre = fp.act_pre;
              r.ep2.has_res = fp.residual >= 0;
              r.ep2.act_post = fp.act_post;
              r.out = loc_of(e, fp.out);
              r.res = loc_of(e, fp.residual);
              inverted_residual_pack(op.weights.data(), op.bias.data(), dwn.weights.data(), dwn.bias.data(), pwn.weights.data(),
                                     pwn.bias.data(), din->c, op.d.cout, pwn.d.cout, &e->weight_blob, &r);
              const uint64_t px2 = B * d2.h * d2.w, c42 = slices(d2.c) * 4;
              info.bytes = (in_px * in_c4 + px2 * c42 * (r.ep2.has_res ? 2 : 1) + static_cast<uint64_t>(din->c) * op.d.cout +
                            9ull * op.d.cout + static_cast<uint64_t>(op.d.cout) * pwn.d.cout) * eb;
              info.flops = 2 * out_px * din->c * op.d.cout + 2 * 9 * px2 * op.d.cout + 2 * px2 * op.d.cout * pwn.d.cout;
              absorbed = 2;
              info.kernel = r.kernel;
              e->launches.push_back(r);
              e->op_info.push_back(info);
              continue;
            }
          }
          // Projection + the next block's expansion as one kernel (the expansion must not be the start of a block that
          // runs as one kernel itself).
          // GI_XOP_AUTO takes it where it measured faster inside MobileNetV2 at batch 256 than the two kernels: 14x14
          // planes with at most 64 channels in the middle and at least two tiles per SM.
          const long long pc_tiles = (m_px_all_for_mm(e, din) + 127) / 128;
          const bool chain_auto = din->h * din->w > 64 && din->h * din->w <= 256 && op.d.cout <= 64 && din->c >= 192 && pc_tiles >= 2 * 148;
          if (pointwise && tc && e->opt.fuse && (e->opt.cross_op == GI_XOP_CHAIN || (e->opt.cross_op == GI_XOP_AUTO && chain_auto)) &&
              chain_follows(g, e, i) &&
              pointwise_chain_supported(din->c, op.d.cout, g.ops[e->ops[i + 1].graph_op].d.cout, f.residual >= 0)) {
            const FusedOp& fb = e->ops[i + 1];
            const OpNode& nb = g.ops[fb.graph_op];
            const TensorDesc& d2 = e->tensors[fb.out];
            r.kernel = GI_KERNEL_POINTWISE_CHAIN;
            r.Cmid = op.d.cout;
            r.Co2 = nb.d.cout;
            r.ep2.act_pre = fb.act_pre;
            r.out2 = loc_of(e, fb.out);
            pointwise_chain_pack(op.weights.data(), op.bias.data(), nb.weights.data(), nb.bias.data(), din->c, op.d.cout, nb.d.cout,
                                 &e->weight_blob, &r);
            const uint64_t c42 = slices(d2.c) * 4;
            info.bytes = (in_px * in_c4 + out_px * out_c4 * (r.ep.has_res ? 2 : 1) + out_px * c42 +
                          static_cast<uint64_t>(din->c) * op.d.cout + static_cast<uint64_t>(op.d.cout) * nb.d.cout) * eb;
            info.flops = 2 * out_px * din->c * op.d.cout + 2 * out_px * op.d.cout * nb.d.cout;
            absorbed = 1;
            info.kernel = r.kernel;
            e->launches.push_back(r);
            e->op_info.push_back(info);
            continue;
          }
          const long long m_px_all = static_cast<long long>(e->batch) * din->h * din->w;
          const bool one_wave = m_px_all <= 64LL * 128 || (m_px_all <= 148LL * 128 && din->c < 960);
          const bool lane_rule = op.d.cout >= 96 && din->c >= 24 && din->c < 960;
          const bool lane_auto = one_wave || lane_rule;
          const bool lane_kernel = e->opt.pointwise == GI_PW_TC_LANE || ((e->opt.pointwise == GI_PW_AUTO || e->opt.pointwise == GI_PW_RULE) && lane_auto);
          // The wide-tile kernel (a CTA pair per tile of 256 pixels x up to 256 output channels) is for the layers with many
          // input channels: at least 512.  Measured against the better of the other two kernels at batch 256 (time wide /
          // time other): 7x7 1024->1024 0.56, 14x14 512->512 0.76, 7x7 512->1024 0.80, 960->160 0.82, 960->320 0.95,
          // 576->160 0.93; batch 64: 14x14 512->512 0.90, 576->96 0.88, 7x7 1024->1024 0.72.  It loses where a launch has
          // too few tiles to fill the 74 pairs' pipelines (batch 64 7x7 960->160, 13 tiles: 1.14) and where many tiles
          // meet a narrow output (batch 256 14x14 576->96, 196 tiles: 1.09 - an MMA takes the same 128 cycles for 96
          // output channels as for 256).  With fewer input channels it wins or loses by a few per cent (28x28 256->256
          // 4 % ahead, 14x14 256->512 15 % behind the lane kernel): the table decides.
          const long long mm_units = ((m_px_all_for_mm(e, din) + 255) / 256) * ((slices(op.d.cout) * 4 + 255) / 256);
          const bool mm_auto = mm_units >= 40 && din->c >= 512 && (op.d.cout >= 160 || mm_units <= 74);
          bool wide_kernel = e->opt.pointwise == GI_PW_TC_WIDE || ((e->opt.pointwise == GI_PW_AUTO || e->opt.pointwise == GI_PW_RULE) && mm_auto);
          bool lane_tab = false, pair_tab = false;
          if (e->opt.pointwise == GI_PW_AUTO && pointwise && tc) {
            if (const LaunchChoice* lc = launch_table_lookup(m_px_all_for_mm(e, din), din->c, op.d.cout)) {
              wide_kernel = lc->kernel == GI_KERNEL_POINTWISE_MM;
              lane_tab = lc->kernel == GI_KERNEL_POINTWISE_TS;
              pair_tab = lc->kernel == GI_KERNEL_POINTWISE_TC;
            }
          }
          if (pointwise && tc && wide_kernel && pointwise_mm_supported(din->c, op.d.cout)) {
            r.kernel = GI_KERNEL_POINTWISE_MM;
            pointwise_mm_pack(op.weights.data(), op.bias.data(), din->c, op.d.cout, &e->weight_blob, &r);
          } else if (pointwise && tc && (lane_tab || (lane_kernel && !pair_tab)) && pointwise_ts_supported(din->c, op.d.cout)) {
            r.kernel = GI_KERNEL_POINTWISE_TS;
            pointwise_ts_pack(op.weights.data(), op.bias.data(), din->c, op.d.cout, &e->weight_blob, &r);
          } else if (pointwise && tc && pointwise_tc_supported(din->c, op.d.cout)) {
            r.kernel = GI_KERNEL_POINTWISE_TC;
            pointwise_tc_pack(op.weights.data(), op.bias.data(), din->c, op.d.cout, &e->weight_blob, &r);
          } else if (tc && conv3x3_tc_supported(din->c, op.d.cout, op.d.kh, op.d.kw, op.d.stride_h, op.d.stride_w,
                                          op.d.dilation_h, op.d.dilation_w)) {
            r.kernel = GI_KERNEL_CONV3X3_TC;
            // Section 3.2 folds cheap operators into the expensive one next to them; the layout conversion in
            // front of the stem is such an operator: where the kernel can read the caller's NHWC tensor itself
            // (and nothing else reads the converted tensor) the conversion launches nothing
            const int pack_op = nhwc_pack_feeding_only(e, f.in0, i);
            if (e->opt.fuse && pack_op >= 0 &&
                conv3x3_tc_reads_nhwc(din->c, din->h, din->w, op.d.stride_h, op.d.dilation_h, op.d.pad_t, op.d.pad_l)) {
              r.nhwc_in = 1;
              r.in0 = Loc{W_INPUT, din->input_index, 0};
              e->launches[pack_op].kernel = GI_KERNEL_NONE;
              e->op_info[pack_op].kernel = GI_KERNEL_NONE;
              e->op_info[pack_op].bytes = 0;
              info.bytes = (in_px * din->c + out_px * out_c4 * (r.ep.has_res ? 2 : 1)) * eb;
            }
            conv3x3_tc_pack(op.weights.data(), op.bias.data(), din->c, op.d.cout, &e->weight_blob, &r);
          } else if (tc && conv_kxk_tc_supported(din->c, op.d.cout, op.d.kh, op.d.kw, op.d.stride_h, op.d.stride_w,
                                                  op.d.dilation_h, op.d.dilation_w)) {
            // any other 1x1 (strided or padded), 2x2 or 3x3 convolution whose weights fit shared memory
            r.kernel = GI_KERNEL_CONV_TC;
            conv_kxk_tc_pack(op.weights.data(), op.bias.data(), din->c, op.d.cout, op.d.kh, &e->weight_blob, &r);
          } else {
            r.kernel = GI_KERNEL_CONV_SIMT;
            const int sout = slices(op.d.cout);
            const int os = sout >= 8 ? 8 : sout >= 4 ? 4 : sout >= 2 ? 2 : 1;
            r.tc_nt = os;
            pack_conv_simt(op, din->c, e->storage, os, &e->weight_blob, &r);
          }
          info.bytes += taps * din->c * op.d.cout * eb;
          info.flops = 2 * taps * out_px * din->c * op.d.cout;
        }
        break;
      }
      case GI_OP_CONCAT:
        if (f.in1 >= 0 && e->plan[f.in0].view_of == f.out && e->plan[f.in1].view_of == f.out) {
          // both inputs were placed inside the output: their producers have already written it
          r.kernel = GI_KERNEL_NONE;
          info.bytes = 0;
          break;
        }
        if (f.in1 >= 0) {
          r.kernel = GI_KERNEL_CONCAT;
          info.bytes = (in_px * (in_c4 + slices(e->tensors[f.in1].c) * 4) + out_px * out_c4) * eb;
          break;
        }
        // a single-input CONCAT that survived the clean-up (its output is a graph output) is a copy
        [[fallthrough]];
      case GI_OP_ADD:
      case GI_OP_ACTIVATION: {
        r.kernel = GI_KERNEL_ELTWISE;
        const OpNode& op = g.ops[f.graph_op];
        if (f.kind == GI_OP_ACTIVATION) r.ep.act_pre = op.d.act;
        info.act_pre = r.ep.act_pre;
        const bool sum = f.kind == GI_OP_ADD && f.in1 >= 0;
        r.ep.has_res = sum;
        info.bytes = (in_px * in_c4 * (sum ? 2 : 1) + out_px * out_c4) * eb;
        info.flops = f.kind == GI_OP_CONCAT || (f.kind == GI_OP_ADD && !sum) ? 0 : out_px * dout->c;
        break;
      }
      case GI_OP_GLOBAL_AVG_POOL:
        r.kernel = GI_KERNEL_POOL;
        info.bytes = (in_px * in_c4 + out_px * out_c4) * eb;
        info.flops = in_px * din->c;
        break;
      case GI_OP_RESIZE_BILINEAR: {
        r.kernel = GI_KERNEL_RESIZE;
        r.align_corners = g.ops[f.graph_op].d.align_corners;
        info.bytes = (in_px * in_c4 + out_px * out_c4) * eb;
        info.flops = 8 * out_px * dout->c;
        break;
      }
      default:
        return fail(GI_E_INVALID, "gi_compile: unknown executed-op kind");
    }
    info.kernel = r.kernel;
    e->launches.push_back(r);
    e->op_info.push_back(info);
  }
  // keep the blob a whole number of 256-byte units so any tail read stays inside it
  e->weight_blob.resize(round_up_u64(e->weight_blob.size() + 1, 256), 0);
  return GI_OK;
}

}  // namespace gi
