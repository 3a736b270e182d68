// Internal structures shared by the host compile step and the CUDA launchers.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "gi.h"

namespace gi {

// ---------------------------------------------------------------- graph (host)
struct TensorDesc {
  int h = 0, w = 0, c = 0;
  int input_index = -1, input_layout = GI_NHWC;    // >= 0 if declared with gi_graph_input
  int output_index = -1, output_layout = GI_NHWC;  // >= 0 if marked with gi_graph_output
};

struct OpNode {
  gi_op_desc d{};             // weights/bias pointers are cleared; the data lives below
  std::vector<float> weights; // fp32 copy, [cout][kh][kw][cin] (depthwise [kh][kw][c])
  std::vector<float> bias;    // cout floats, zeros if none was given
  int output = -1;
};

}  // namespace gi

struct gi_graph {
  int batch = 1, storage = GI_F16;
  std::vector<gi::TensorDesc> tensors;
  std::vector<gi::OpNode> ops;
  std::vector<int> inputs, outputs;
};

namespace gi {

// ---------------------------------------------------------------- executable
// Where a tensor's bytes are at run time.
enum Where : int { W_NONE = 0, W_ARENA = 1, W_INPUT = 2, W_OUTPUT = 3, W_WEIGHTS = 4 };
struct Loc {
  int where = W_NONE;
  int index = 0;        // input / output number
  uint64_t offset = 0;  // byte offset inside the arena or the weight blob
};

struct Epilogue {
  int act_pre = GI_ACT_NONE;
  int has_res = 0;
  int act_post = GI_ACT_NONE;
};

// Parameters of one kernel launch; pointers are resolved by gi_run from the Locs.
struct LaunchRec {
  int kernel = 0;  // GI_KERNEL_*
  Loc in0, in1, res, out, wts, bias;
  // geometry (pixels per stored plane are h*w rounded up to even)
  int B = 1, H = 0, W = 0, C = 0;  // input logical shape
  int Ho = 0, Wo = 0, Co = 0;      // output logical shape
  int kh = 1, kw = 1, sh = 1, sw = 1, dh = 1, dw = 1, pt = 0, pl = 0;
  int align_corners = 1;
  int io_layout = GI_NHWC;
  Epilogue ep;
  // pointwise tensor-core kernel: tiling chosen at compile time
  int tc_nt = 0;       // output channels per CTA tile
  int tc_kc = 0;       // input slices per pipeline stage
  int tc_stages = 0;
  uint64_t wts_bytes = 0;
  // no executed op reads the first input after this one (and it is not a graph output): it is read
  // with the "evict first" L2 policy, which keeps this op's output - the next op's input - resident
  // instead (MobileNetV2 at batch 256: 1.756 -> 1.728 ms, measured in one run on one GPU)
  int in0_dead = 0;
  // depthwise: 1 = the shared-memory staged fp16 stencil runs this op, 0 = the plain one-thread-per-pixel kernel
  int dw_staged = 0;
  // staged stencil: size limit of one staging buffer and shared memory of one CTA in KB, from the measured table of
  // staging choices (0 = the kernel's defaults, 64 and 110)
  int dw_buf_kb = 0, dw_cta_kb = 0;
  // the stem convolution reads the caller's NHWC input itself; the layout conversion in front of it launches nothing
  int nhwc_in = 0;
  // depthwise + pointwise as one kernel: the 1x1 convolution's weights, bias, output channels and epilogue
  // (`out` and `res` are then the 1x1 convolution's; `ep` stays the depthwise op's)
  Loc wts2, bias2;
  int Co2 = 0;
  Epilogue ep2;
  // a whole inverted-residual block as one kernel: `ep` is the expansion's epilogue, `ep_mid` the depthwise op's,
  // `ep2` the projection's; Cmid the hidden channels; the stride / pads are the depthwise op's, (Ho, Wo) its output
  int Cmid = 0;
  Epilogue ep_mid;
  // two consecutive 1x1 convolutions as one kernel: `out` / `res` / `ep` / `wts` are the first one's (Cmid its output
  // channels), `out2` / `ep2` / `wts2` / Co2 the second one's; `bias` holds both bias vectors
  Loc out2;
};

struct FusedOp {
  int kind = 0;       // GI_OP_* | GI_EXEC_PACK | GI_EXEC_UNPACK
  int graph_op = -1;
  int in0 = -1, in1 = -1, residual = -1, out = -1;
  int act_pre = GI_ACT_NONE, act_post = GI_ACT_NONE;
  int slot = 0;       // next free position in the pattern [act][add][act]
  int io_index = -1;  // pack: input number, unpack: output number
};

struct TensorPlan {
  int alive = 0, intermediate = 0, first = -1, last = -1;  // intermediate: 1 planned, 2 placed inside `view_of`
  uint64_t bytes = 0, offset = 0;
  int view_of = -1;    // the tensor whose memory holds this one (an input of a CONCAT that needs no copy), or -1
  int view_slice = 0;  // first slice of `view_of` that this tensor occupies
};

}  // namespace gi

struct gi_exec {
  int batch = 1, storage = GI_F16;
  gi_compile_options opt{};
  std::vector<gi::TensorDesc> tensors;
  std::vector<gi::TensorPlan> plan;
  std::vector<gi::FusedOp> ops;       // executed ops in order
  std::vector<gi_op_info> op_info;
  std::vector<gi::LaunchRec> launches;
  std::vector<uint8_t> weight_blob;   // host staging copy of all packed weights
  int n_inputs = 0, n_outputs = 0, n_fused = 0;
  uint64_t arena_bytes = 0, naive_bytes = 0, lower_bound = 0;
  void* dev_weights = nullptr;        // set by gi_exec_bind
  void* tc_state = nullptr;           // tensor-map cache owned by the run module
};

namespace gi {

void set_error(const std::string& msg);
gi_status fail(gi_status s, const std::string& msg);

inline uint64_t round_up_u64(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }
inline int plane_pixels(int h, int w) { return (h * w + 1) / 2 * 2; }
inline int slices(int c) { return (c + 3) / 4; }
inline int elem_bytes(int storage) { return storage == GI_F32 ? 4 : 2; }

uint16_t f32_to_f16_rne(float f);

// compile-step pieces (gi_compile.cc)
gi_status fuse_graph(const gi_graph& g, bool enable, std::vector<FusedOp>* out);
gi_status plan_memory(gi_exec* e);

// weight packing + launch records (gi_lower.cc)
gi_status lower(const gi_graph& g, gi_exec* e);

// run module (gi_run.cu)
void release_run_state(gi_exec* e);

}  // namespace gi
