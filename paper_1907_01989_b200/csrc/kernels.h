// Launchers of the CUDA kernels.  Each takes resolved device pointers, enqueues on `stream`
// and returns the cudaError_t of the launch (as int, so host-only files need no CUDA headers).
#pragma once

#include <cstdint>
#include <vector>

#include "gi_internal.h"

namespace gi {

// Launch-side facts that belong to a device, not to the process (a process may drive several
// GPUs): SM count and "shared-memory attribute already raised" flags, indexed by the current device.
constexpr int kMaxDevices = 64;
int current_device_slot();  // cudaGetDevice() folded into [0, kMaxDevices)
int device_sm_count();      // of the current device (cached); 148 if the query fails

struct Ptrs {
  const void* in0 = nullptr;
  const void* in1 = nullptr;
  const void* res = nullptr;
  void* out = nullptr;
  const void* wts = nullptr;
  const void* bias = nullptr;
  const void* wts2 = nullptr;   // second operator of a two-operator kernel
  const void* bias2 = nullptr;
  void* out2 = nullptr;         // second output of a kernel that stores two tensors
};

int launch_pack(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_unpack(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_conv_simt(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_depthwise(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
// fp16 storage, equal strides / dilations on both axes: shared-memory staged stencil
int launch_depthwise_f16(const LaunchRec& r, const Ptrs& p, void* stream);
bool depthwise_f16_supported(const LaunchRec& r);  // host-only check, used when the op is lowered
unsigned int depthwise_error_word(int* cuda_err);
int launch_eltwise(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_concat(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_pool(const LaunchRec& r, const Ptrs& p, int storage, void* stream);
int launch_resize(const LaunchRec& r, const Ptrs& p, int storage, void* stream);

// Tensor-core pointwise convolution (fp16 storage only).
bool pointwise_tc_supported(int cin, int cout);
void pointwise_tc_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r);
// tensor maps depend on device addresses; `state` caches them per executable
int launch_pointwise_tc(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream);
void pointwise_tc_release(void* state);
unsigned int pointwise_tc_error_word(int* cuda_err);


// Full 3x3 convolution with one input slice (<= 4 channels) on the tensor cores (fp16 storage).
bool conv3x3_tc_supported(int cin, int cout, int kh, int kw, int sh, int sw, int dh, int dw);
bool conv3x3_tc_reads_nhwc(int cin, int H, int W, int stride, int dil, int pt, int pl);
void conv3x3_tc_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r);
int launch_conv3x3_tc(const LaunchRec& r, const Ptrs& p, void* stream);
unsigned int conv3x3_tc_error_word(int* cuda_err);

// k x k convolution (k = 1..3) of any number of input channels on the tensor cores (conv_tc.cu)
bool conv_kxk_tc_supported(int cin, int cout, int kh, int kw, int sh, int sw, int dh, int dw);
void conv_kxk_tc_pack(const float* w, const float* bias, int cin, int cout, int k, std::vector<uint8_t>* blob, LaunchRec* r);
int launch_conv_kxk_tc(const LaunchRec& r, const Ptrs& p, void* stream);
unsigned int conv_kxk_tc_error_word(int* cuda_err);

// Pointwise convolution with the activation operand in tensor memory (fp16 storage).
bool pointwise_ts_supported(int cin, int cout);
void pointwise_ts_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r);
int launch_pointwise_ts(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream);
unsigned int pointwise_ts_error_word(int* cuda_err);

// Depthwise 3x3 followed by a pointwise convolution, as one kernel (fp16 storage): the depthwise
// output stays on chip.  `dw` is the depthwise op's record; `tiles` receives the kernel's parallelism,
// `lanes` how many of an MMA's 128 rows a pixel tile fills.
bool depthwise_pointwise_supported(const LaunchRec& dw, int cout, long long* tiles, int* lanes);
void depthwise_pointwise_pack(const float* w, const float* bias, int cin, int cout, int width, std::vector<uint8_t>* blob,
                              LaunchRec* r);
int launch_depthwise_pointwise(const LaunchRec& r, const Ptrs& p, void* stream);
unsigned int depthwise_pointwise_error_word(int* cuda_err);

// Pointwise convolution for tensor-bound shapes (many input and output channels): 256 x 256 CTA tiles, both operands
// streamed (pointwise_mm.cu; fp16 storage)
bool pointwise_mm_supported(int cin, int cout);
void pointwise_mm_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r);
void pointwise_mm_blob_layout(int cin, int cout, uint64_t* bias_off, uint64_t* total);
int launch_pointwise_mm(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream);
int launch_pointwise_mm_slice8(const void* in, void* out, const void* wts, const float* bias, unsigned m_total, int cin, int cout,
                               int act, void* stream);
unsigned int pointwise_mm_error_word(int* cuda_err);

// Two consecutive 1x1 convolutions (a block's projection and the next block's expansion) as one kernel (fp16 storage):
// both outputs are stored, the tensor between them is not read back (pointwise_chain.cu)
bool pointwise_chain_supported(int cin, int cmid, int cout, bool has_res);
void pointwise_chain_pack(const float* w1, const float* b1, const float* w2, const float* b2, int cin, int cmid, int cout,
                          std::vector<uint8_t>* blob, LaunchRec* r);
int launch_pointwise_chain(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream);
unsigned int pointwise_chain_error_word(int* cuda_err);

// One inverted-residual block (1x1 expansion -> depthwise 3x3 -> 1x1 projection, + residual) as one kernel (fp16
// storage, planes of at most 256 pixels): neither hidden tensor leaves the SM.  `units` receives the kernel's parallelism.
bool inverted_residual_supported(int B, int H, int W, int Ho, int Wo, int stride, int dil, int pt, int pl, int cin, int chid,
                                 int cout, long long* units);
void inverted_residual_pack(const float* we, const float* be, const float* wd, const float* bd, const float* wp, const float* bp,
                            int cin, int chid, int cout, std::vector<uint8_t>* blob, LaunchRec* r);
int launch_inverted_residual(const LaunchRec& r, const Ptrs& p, void* stream);
unsigned int inverted_residual_error_word(int* cuda_err);

}  // namespace gi
