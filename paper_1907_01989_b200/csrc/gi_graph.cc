// Graph construction half of the C ABI: validation and shape inference at gi_add_op.
#include <cstring>
#include <new>

#include "gi_internal.h"

namespace gi {

static thread_local std::string g_last_error;

void set_error(const std::string& msg) { g_last_error = msg; }

gi_status fail(gi_status s, const std::string& msg) {
  g_last_error = msg;
  return s;
}

// fp32 -> fp16 bits, round to nearest even, done on the integer representation.
uint16_t f32_to_f16_rne(float f) {
  uint32_t x;
  std::memcpy(&x, &f, sizeof x);
  const uint16_t sign = static_cast<uint16_t>((x >> 16) & 0x8000u);
  x &= 0x7fffffffu;
  if (x > 0x7f800000u) return static_cast<uint16_t>(sign | 0x7e00u | ((x >> 13) & 0x1ffu));  // NaN
  if (x >= 0x47800000u) return static_cast<uint16_t>(sign | 0x7c00u);  // >= 65536 (or inf): infinity
  if (x < 0x33000000u) return sign;                                    // < 2^-25: zero
  uint32_t mant, shift;
  if (x < 0x38800000u) {
    // result is subnormal: express the value as an integer count of 2^-24
    shift = 126u - (x >> 23);  // between 14 and 24
    mant = (x & 0x7fffffu) | 0x800000u;
    const uint32_t q = mant >> shift;
    const uint32_t rest = mant - (q << shift);
    const uint32_t halfway = 1u << (shift - 1);
    const uint32_t up = (rest > halfway) || (rest == halfway && (q & 1u));
    return static_cast<uint16_t>(sign | (q + up));
  }
  // normal: rebias the exponent (127 -> 15) and drop 13 mantissa bits with RNE; a carry out of
  // the mantissa moves into the exponent, which is the correctly rounded result (up to infinity)
  const uint32_t rebased = x - 0x38000000u;
  const uint32_t q = rebased >> 13;
  const uint32_t rest = rebased & 0x1fffu;
  const uint32_t up = (rest > 0x1000u) || (rest == 0x1000u && (q & 1u));
  return static_cast<uint16_t>(sign | (q + up));
}

static int conv_out(int in, int k, int stride, int dil, int p0, int p1) {
  const int span = (k - 1) * dil + 1;
  const int padded = in + p0 + p1;
  if (padded < span) return 0;
  return (padded - span) / stride + 1;
}

}  // namespace gi

using namespace gi;

extern "C" {

const char* gi_status_str(gi_status s) {
  switch (s) {
    case GI_OK: return "GI_OK";
    case GI_E_INVALID: return "GI_E_INVALID";
    case GI_E_UNSUPPORTED: return "GI_E_UNSUPPORTED";
    case GI_E_NOMEM: return "GI_E_NOMEM";
    case GI_E_CUDA: return "GI_E_CUDA";
    case GI_E_STATE: return "GI_E_STATE";
    case GI_E_ARENA: return "GI_E_ARENA";
    default: return "GI_E_UNKNOWN";
  }
}

const char* gi_last_error(void) { return g_last_error.c_str(); }

void gi_f32_to_f16(const float* src, uint16_t* dst, size_t n) {
  if (!src || !dst) return;
  for (size_t i = 0; i < n; ++i) dst[i] = f32_to_f16_rne(src[i]);
}

uint64_t gi_tensor_bytes(int32_t batch, int32_t H, int32_t W, int32_t C, int32_t storage, int32_t align) {
  if (batch <= 0 || H <= 0 || W <= 0 || C <= 0) return 0;
  const uint64_t a = align > 0 ? static_cast<uint64_t>(align) : 256u;
  const uint64_t raw = static_cast<uint64_t>(batch) * slices(C) * plane_pixels(H, W) * 4u * elem_bytes(storage);
  return round_up_u64(raw, a);
}

gi_status gi_graph_create(gi_graph** out, int32_t batch, int32_t storage) {
  if (!out) return fail(GI_E_INVALID, "gi_graph_create: out is null");
  *out = nullptr;
  if (batch <= 0) return fail(GI_E_INVALID, "gi_graph_create: batch must be positive");
  if (storage != GI_F16 && storage != GI_F32) return fail(GI_E_INVALID, "gi_graph_create: unknown storage type");
  gi_graph* g = new (std::nothrow) gi_graph();
  if (!g) return fail(GI_E_NOMEM, "gi_graph_create: out of host memory");
  g->batch = batch;
  g->storage = storage;
  *out = g;
  return GI_OK;
}

void gi_graph_destroy(gi_graph* g) { delete g; }

gi_status gi_graph_input(gi_graph* g, int32_t H, int32_t W, int32_t C, int32_t layout, gi_tensor* out) {
  if (!g || !out) return fail(GI_E_INVALID, "gi_graph_input: null argument");
  if (H <= 0 || W <= 0 || C <= 0) return fail(GI_E_INVALID, "gi_graph_input: extents must be positive");
  if (layout != GI_NHWC && layout != GI_PHWC4) return fail(GI_E_INVALID, "gi_graph_input: unknown layout");
  if (static_cast<uint64_t>(H) * W > (1u << 28)) return fail(GI_E_UNSUPPORTED, "gi_graph_input: plane too large");
  TensorDesc t;
  t.h = H;
  t.w = W;
  t.c = C;
  t.input_index = static_cast<int>(g->inputs.size());
  t.input_layout = layout;
  const size_t nt = g->tensors.size();
  try {
    g->tensors.push_back(t);
    g->inputs.push_back(static_cast<int>(nt));
  } catch (const std::bad_alloc&) {
    g->tensors.resize(nt);
    return fail(GI_E_NOMEM, "gi_graph_input: out of host memory");
  }
  *out = g->inputs.back();
  return GI_OK;
}

gi_status gi_graph_output(gi_graph* g, gi_tensor t, int32_t layout) {
  if (!g) return fail(GI_E_INVALID, "gi_graph_output: null graph");
  if (t < 0 || t >= static_cast<int>(g->tensors.size())) return fail(GI_E_INVALID, "gi_graph_output: unknown tensor");
  if (layout != GI_NHWC && layout != GI_PHWC4) return fail(GI_E_INVALID, "gi_graph_output: unknown layout");
  TensorDesc& d = g->tensors[t];
  if (d.input_index >= 0) return fail(GI_E_INVALID, "gi_graph_output: a graph input cannot be an output");
  if (d.output_index >= 0) return fail(GI_E_INVALID, "gi_graph_output: tensor is already an output");
  try {
    g->outputs.push_back(t);
  } catch (const std::bad_alloc&) {
    return fail(GI_E_NOMEM, "gi_graph_output: out of host memory");
  }
  d.output_index = static_cast<int>(g->outputs.size()) - 1;
  d.output_layout = layout;
  return GI_OK;
}

// gi_add_op proper; may throw std::bad_alloc (the exported wrapper below turns that into GI_E_NOMEM)
static gi_status add_op_checked(gi_graph* g, const gi_op_desc* desc, gi_tensor* out) {
  const int nt = static_cast<int>(g->tensors.size());
  auto known = [&](int t) { return t >= 0 && t < nt; };
  if (!known(desc->inputs[0])) return fail(GI_E_INVALID, "gi_add_op: inputs[0] is not a tensor of this graph");
  const TensorDesc in = g->tensors[desc->inputs[0]];
  OpNode node;
  node.d = *desc;
  node.d.weights = nullptr;
  node.d.bias = nullptr;
  TensorDesc o;
  switch (desc->kind) {
    case GI_OP_CONV2D:
    case GI_OP_DEPTHWISE_CONV2D: {
      const bool dwise = desc->kind == GI_OP_DEPTHWISE_CONV2D;
      if (desc->kh != desc->kw || desc->kh < 1 || desc->kh > 3 || (dwise && desc->kh != 3))
        return fail(GI_E_UNSUPPORTED, "gi_add_op: kernel must be 1x1, 2x2 or 3x3 (depthwise: 3x3)");
      if (desc->stride_h < 1 || desc->stride_w < 1 || desc->dilation_h < 1 || desc->dilation_w < 1)
        return fail(GI_E_INVALID, "gi_add_op: stride and dilation must be >= 1");
      if (desc->stride_h > (dwise ? 2 : 3) || desc->stride_w > (dwise ? 2 : 3))
        return fail(GI_E_UNSUPPORTED, "gi_add_op: stride above 3 (depthwise: above 2) is not supported");
      if (desc->pad_t < 0 || desc->pad_l < 0 || desc->pad_b < 0 || desc->pad_r < 0)
        return fail(GI_E_INVALID, "gi_add_op: negative padding");
      if (!desc->weights) return fail(GI_E_INVALID, "gi_add_op: convolution without weights");
      if (desc->weight_dtype != GI_F32 && desc->weight_dtype != GI_F16)
        return fail(GI_E_INVALID, "gi_add_op: weight_dtype must be GI_F32 or GI_F16");
      const int cout = dwise ? in.c : desc->cout;
      if (cout <= 0) return fail(GI_E_INVALID, "gi_add_op: cout must be positive");
      o.h = conv_out(in.h, desc->kh, desc->stride_h, desc->dilation_h, desc->pad_t, desc->pad_b);
      o.w = conv_out(in.w, desc->kw, desc->stride_w, desc->dilation_w, desc->pad_l, desc->pad_r);
      o.c = cout;
      if (o.h <= 0 || o.w <= 0) return fail(GI_E_INVALID, "gi_add_op: kernel window larger than the padded input");
      node.d.cout = cout;
      const size_t nw = static_cast<size_t>(dwise ? 1 : cout) * desc->kh * desc->kw * in.c;
      node.weights.resize(nw);
      if (desc->weight_dtype == GI_F32) {
        std::memcpy(node.weights.data(), desc->weights, nw * sizeof(float));
      } else {
        const uint16_t* h = static_cast<const uint16_t*>(desc->weights);
        for (size_t i = 0; i < nw; ++i) {
          // widen fp16 bits to fp32 exactly
          const uint32_t s = (h[i] & 0x8000u) << 16, e = (h[i] >> 10) & 0x1fu, m = h[i] & 0x3ffu;
          float v;
          if (e == 0) {
            v = static_cast<float>(m) * (1.0f / 16777216.0f);
          } else if (e == 31) {
            const uint32_t u = 0x7f800000u | (m << 13);
            std::memcpy(&v, &u, 4);
          } else {
            const uint32_t u = ((e + 112u) << 23) | (m << 13);
            std::memcpy(&v, &u, 4);
          }
          uint32_t u;
          std::memcpy(&u, &v, 4);
          u |= s;
          std::memcpy(&node.weights[i], &u, 4);
        }
      }
      node.bias.assign(cout, 0.0f);
      if (desc->bias) std::memcpy(node.bias.data(), desc->bias, cout * sizeof(float));
      break;
    }
    case GI_OP_ADD: {
      o.h = in.h;
      o.w = in.w;
      o.c = in.c;
      if (desc->inputs[1] == -1) break;  // single input: the identity
      if (!known(desc->inputs[1])) return fail(GI_E_INVALID, "gi_add_op: ADD: inputs[1] is neither a tensor of this graph nor -1");
      const TensorDesc& b = g->tensors[desc->inputs[1]];
      if (b.h != in.h || b.w != in.w || b.c != in.c) return fail(GI_E_INVALID, "gi_add_op: ADD operands differ in shape");
      break;
    }
    case GI_OP_CONCAT: {
      o.h = in.h;
      o.w = in.w;
      o.c = in.c;
      if (desc->inputs[1] == -1) break;  // single input: the identity
      if (!known(desc->inputs[1])) return fail(GI_E_INVALID, "gi_add_op: CONCAT: inputs[1] is neither a tensor of this graph nor -1");
      const TensorDesc& b = g->tensors[desc->inputs[1]];
      if (b.h != in.h || b.w != in.w) return fail(GI_E_INVALID, "gi_add_op: CONCAT operands differ in height or width");
      if (static_cast<int64_t>(in.c) + b.c > (1 << 20)) return fail(GI_E_UNSUPPORTED, "gi_add_op: CONCAT: too many channels");
      o.c = in.c + b.c;
      break;
    }
    case GI_OP_ACTIVATION:
      if (desc->act != GI_ACT_RELU && desc->act != GI_ACT_RELU6)
        return fail(GI_E_INVALID, "gi_add_op: ACTIVATION needs GI_ACT_RELU or GI_ACT_RELU6");
      o.h = in.h;
      o.w = in.w;
      o.c = in.c;
      break;
    case GI_OP_GLOBAL_AVG_POOL:
      o.h = 1;
      o.w = 1;
      o.c = in.c;
      break;
    case GI_OP_RESIZE_BILINEAR:
      if (desc->out_h <= 0 || desc->out_w <= 0) return fail(GI_E_INVALID, "gi_add_op: RESIZE needs positive out_h, out_w");
      o.h = desc->out_h;
      o.w = desc->out_w;
      o.c = in.c;
      break;
    default:
      return fail(GI_E_INVALID, "gi_add_op: unknown operator kind");
  }
  if (desc->kind != GI_OP_ADD && desc->kind != GI_OP_CONCAT) node.d.inputs[1] = -1;
  if (static_cast<uint64_t>(o.h) * o.w > (1u << 28)) return fail(GI_E_UNSUPPORTED, "gi_add_op: output plane too large");
  g->tensors.push_back(o);
  node.output = static_cast<int>(g->tensors.size()) - 1;
  g->ops.push_back(std::move(node));
  *out = g->ops.back().output;
  return GI_OK;
}

gi_status gi_add_op(gi_graph* g, const gi_op_desc* desc, gi_tensor* out) {
  if (!g || !desc || !out) return fail(GI_E_INVALID, "gi_add_op: null argument");
  // no exception may cross the C boundary: whatever the copies of weights and bias or the growth of the
  // graph's vectors throw, the graph is left as it was before the call
  const size_t n_tensors = g->tensors.size(), n_ops = g->ops.size();
  try {
    return add_op_checked(g, desc, out);
  } catch (const std::bad_alloc&) {
    g->tensors.resize(n_tensors);
    g->ops.resize(n_ops);
    return fail(GI_E_NOMEM, "gi_add_op: out of host memory");
  } catch (...) {
    g->tensors.resize(n_tensors);
    g->ops.resize(n_ops);
    return fail(GI_E_NOMEM, "gi_add_op: unexpected host failure");
  }
}

}  // extern "C"
