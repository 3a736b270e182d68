// Run half of the C ABI: weight upload and the launch loop.  gi_run only enqueues work on
// the caller's stream; it never synchronises and never allocates device memory.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "gi_internal.h"
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace gi {

int current_device_slot() {
  int dev = 0;
  cudaGetDevice(&dev);
  return dev < 0 ? 0 : dev % kMaxDevices;
}

int device_sm_count() {
  static int sms[kMaxDevices] = {};
  const int slot = current_device_slot();
  if (sms[slot] == 0) {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    sms[slot] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
  }
  return sms[slot];
}


void release_run_state(gi_exec* e) {
  if (e->tc_state) {
    pointwise_tc_release(e->tc_state);
    e->tc_state = nullptr;
  }
}

static bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

}  // namespace gi

using namespace gi;

extern "C" {

gi_status gi_exec_bind(gi_exec* e, void* dev_weights, size_t weight_bytes, void* stream) {
  if (!e || !dev_weights) return fail(GI_E_INVALID, "gi_exec_bind: null argument");
  if (!aligned256(dev_weights)) return fail(GI_E_ARENA, "gi_exec_bind: dev_weights must be 256-byte aligned");
  if (weight_bytes < e->weight_blob.size()) return fail(GI_E_ARENA, "gi_exec_bind: weight buffer too small");
  const cudaError_t err = cudaMemcpyAsync(dev_weights, e->weight_blob.data(), e->weight_blob.size(), cudaMemcpyHostToDevice,
                                          static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return fail(GI_E_CUDA, std::string("gi_exec_bind: ") + cudaGetErrorString(err));
  if (e->dev_weights != dev_weights) release_run_state(e);  // cached tensor maps point at the old buffer
  e->dev_weights = dev_weights;
  return GI_OK;
}

static gi_status run_impl(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* dev_arena,
                          size_t arena_bytes, void* stream, cudaEvent_t* events) {
  if (!e || !dev_inputs || !dev_outputs) return fail(GI_E_INVALID, "gi_run: null argument");
  if (!e->dev_weights) return fail(GI_E_STATE, "gi_run: gi_exec_bind has not been called");
  if (e->arena_bytes > 0) {
    if (!dev_arena) return fail(GI_E_ARENA, "gi_run: null arena");
    if (!aligned256(dev_arena)) return fail(GI_E_ARENA, "gi_run: arena must be 256-byte aligned");
    if (arena_bytes < e->arena_bytes) return fail(GI_E_ARENA, "gi_run: arena smaller than gi_exec_info.arena_bytes");
  }
  for (int i = 0; i < e->n_inputs; ++i)
    if (!dev_inputs[i] || !aligned256(dev_inputs[i])) return fail(GI_E_INVALID, "gi_run: input pointer null or not 256-byte aligned");
  for (int i = 0; i < e->n_outputs; ++i)
    if (!dev_outputs[i] || !aligned256(dev_outputs[i])) return fail(GI_E_INVALID, "gi_run: output pointer null or not 256-byte aligned");

  auto resolve = [&](const Loc& l) -> void* {
    switch (l.where) {
      case W_ARENA: return static_cast<char*>(dev_arena) + l.offset;
      case W_INPUT: return const_cast<void*>(dev_inputs[l.index]);
      case W_OUTPUT: return dev_outputs[l.index];
      case W_WEIGHTS: return static_cast<char*>(e->dev_weights) + l.offset;
      default: return nullptr;
    }
  };

  for (size_t i = 0; i < e->launches.size(); ++i) {
    const LaunchRec& r = e->launches[i];
    if (events) cudaEventRecord(events[i], static_cast<cudaStream_t>(stream));
    Ptrs p;
    p.in0 = resolve(r.in0);
    p.in1 = resolve(r.in1);
    p.res = resolve(r.res);
    p.out = resolve(r.out);
    p.wts = resolve(r.wts);
    p.bias = resolve(r.bias);
    p.wts2 = resolve(r.wts2);
    p.bias2 = resolve(r.bias2);
    p.out2 = resolve(r.out2);
    int err = 0;
    switch (r.kernel) {
      case GI_KERNEL_PACK: err = launch_pack(r, p, e->storage, stream); break;
      case GI_KERNEL_UNPACK: err = launch_unpack(r, p, e->storage, stream); break;
      case GI_KERNEL_CONV_SIMT: err = launch_conv_simt(r, p, e->storage, stream); break;
      case GI_KERNEL_POINTWISE_TC: err = launch_pointwise_tc(r, p, &e->tc_state, static_cast<int>(i), stream); break;
      case GI_KERNEL_CONV3X3_TC: err = launch_conv3x3_tc(r, p, stream); break;
      case GI_KERNEL_POINTWISE_TS: err = launch_pointwise_ts(r, p, &e->tc_state, static_cast<int>(i), stream); break;
      case GI_KERNEL_DEPTHWISE: err = launch_depthwise(r, p, e->storage, stream); break;
      case GI_KERNEL_DEPTHWISE_POINTWISE: err = launch_depthwise_pointwise(r, p, stream); break;
      case GI_KERNEL_INVERTED_RESIDUAL: err = launch_inverted_residual(r, p, stream); break;
      case GI_KERNEL_POINTWISE_MM: err = launch_pointwise_mm(r, p, &e->tc_state, static_cast<int>(i), stream); break;
      case GI_KERNEL_POINTWISE_CHAIN: err = launch_pointwise_chain(r, p, &e->tc_state, static_cast<int>(i), stream); break;
      case GI_KERNEL_NONE: break;  // computed by the previous launch
      case GI_KERNEL_ELTWISE:
        if (r.ep.has_res && !p.in1) p.in1 = p.res;
        err = launch_eltwise(r, p, e->storage, stream);
        break;
      case GI_KERNEL_CONV_TC: err = launch_conv_kxk_tc(r, p, stream); break;
      case GI_KERNEL_CONCAT: err = launch_concat(r, p, e->storage, stream); break;
      case GI_KERNEL_POOL: err = launch_pool(r, p, e->storage, stream); break;
      case GI_KERNEL_RESIZE: err = launch_resize(r, p, e->storage, stream); break;
      default: return fail(GI_E_INVALID, "gi_run: corrupt launch table");
    }
    if (err != 0) {
      return fail(GI_E_CUDA, "gi_run: launch " + std::to_string(i) + " failed: " +
                                 cudaGetErrorString(static_cast<cudaError_t>(err)));
    }
  }
  if (events) cudaEventRecord(events[e->launches.size()], static_cast<cudaStream_t>(stream));
  return GI_OK;
}

gi_status gi_device_status(uint32_t* flags) {
  if (!flags) return fail(GI_E_INVALID, "gi_device_status: null argument");
  int err = 0;
  *flags = pointwise_tc_error_word(&err);
  if (err == 0) *flags |= depthwise_error_word(&err) << 16;
  if (err == 0) *flags |= conv3x3_tc_error_word(&err) << 20;
  if (err == 0) *flags |= conv_kxk_tc_error_word(&err) << 20;
  if (err == 0) *flags |= pointwise_ts_error_word(&err) << 24;
  if (err == 0) *flags |= depthwise_pointwise_error_word(&err) << 28;
  if (err == 0) *flags |= inverted_residual_error_word(&err) << 4;
  if (err == 0) *flags |= pointwise_mm_error_word(&err) << 8;
  if (err == 0) *flags |= pointwise_chain_error_word(&err) << 12;
  if (err != 0) return fail(GI_E_CUDA, std::string("gi_device_status: ") + cudaGetErrorString(static_cast<cudaError_t>(err)));
  return GI_OK;
}

gi_status gi_run(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* dev_arena, size_t arena_bytes,
                 void* stream) {
  return run_impl(e, dev_inputs, dev_outputs, dev_arena, arena_bytes, stream, nullptr);
}

// ---------------------------------------------------------------- fixed arena (no allocation)
// The arena of gi_run_static.  In host code this name is only a handle for the symbol: the
// address kernels can use is obtained with cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_arena[GI_STATIC_ARENA_BYTES];
static std::mutex g_static_mu;
static void* g_static_ptr[64] = {};

gi_status gi_run_static(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* stream) {
  if (!e) return fail(GI_E_INVALID, "gi_run_static: null executable");
  if (e->arena_bytes > GI_STATIC_ARENA_BYTES)
    return fail(GI_E_ARENA, "gi_run_static: executable needs " + std::to_string(e->arena_bytes) +
                                " arena bytes, the built-in arena holds " + std::to_string(GI_STATIC_ARENA_BYTES));
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return fail(GI_E_CUDA, std::string("gi_run_static: ") + cudaGetErrorString(err));
  if (dev < 0 || dev >= 64) return fail(GI_E_UNSUPPORTED, "gi_run_static: device ordinal above 63");
  void* arena = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
      void* ptr = nullptr;
      err = cudaGetSymbolAddress(&ptr, g_static_arena);
      if (err != cudaSuccess || !ptr)
        return fail(GI_E_CUDA, std::string("gi_run_static: cudaGetSymbolAddress: ") + cudaGetErrorString(err));
      g_static_ptr[dev] = ptr;
    }
    arena = g_static_ptr[dev];
  }
  return run_impl(e, dev_inputs, dev_outputs, arena, GI_STATIC_ARENA_BYTES, stream, nullptr);
}

// ---------------------------------------------------------------- self-test of the bounded wait
namespace {
__device__ unsigned int g_selftest_error = 0;
__global__ void bounded_wait_selftest_kernel(unsigned timeout_ns, unsigned long long* result) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ unsigned abort_flag;
  if (threadIdx.x == 0) {
    gi::ptx::mbar_init(gi::ptx::smem_u32(&bar), 1);  // one arrival expected; nobody arrives
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const unsigned long long t0 = gi::ptx::global_timer_ns();
  // the whole warp waits, as the drain warps of the tensor-core kernels do; one lane's limit ends it for all
  const bool ok = gi::ptx::mbar_wait_warp(gi::ptx::smem_u32(&bar), 0u, &abort_flag, timeout_ns, &g_selftest_error, 1u);
  const unsigned long long t1 = gi::ptx::global_timer_ns();
  if (threadIdx.x == 0) {
    result[0] = t1 - t0;
    result[1] = ok ? 0ull : 1ull;
    result[2] = abort_flag;
    result[3] = g_selftest_error;
  }
}
}  // namespace

gi_status gi_selftest_bounded_wait(uint32_t limit_us, uint32_t* waited_us, int32_t* gave_up, void* stream) {
  if (!waited_us || !gave_up) return fail(GI_E_INVALID, "gi_selftest_bounded_wait: null argument");
  if (limit_us < 1 || limit_us > 100000) return fail(GI_E_INVALID, "gi_selftest_bounded_wait: limit_us must be 1 .. 100000");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // pinned, device-visible host memory for the four result words: the library allocates no device memory
  unsigned long long* host = nullptr;
  cudaError_t err = cudaHostAlloc(reinterpret_cast<void**>(&host), 4 * sizeof(unsigned long long), cudaHostAllocMapped);
  if (err != cudaSuccess) return fail(GI_E_CUDA, std::string("gi_selftest_bounded_wait: ") + cudaGetErrorString(err));
  for (int i = 0; i < 4; ++i) host[i] = ~0ull;
  unsigned long long* dev = nullptr;
  err = cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev), host, 0);
  if (err == cudaSuccess) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(limit_us * 1000u, dev);
    err = cudaGetLastError();
  }
  if (err == cudaSuccess) err = cudaStreamSynchronize(st);
  gi_status status = GI_OK;
  if (err != cudaSuccess) {
    status = fail(GI_E_CUDA, std::string("gi_selftest_bounded_wait: ") + cudaGetErrorString(err));
  } else {
    *waited_us = static_cast<uint32_t>(host[0] / 1000ull);
    *gave_up = (host[1] == 1ull && host[2] == 1ull && (host[3] & 1ull)) ? 1 : 0;
  }
  cudaFreeHost(host);
  return status;
}

gi_status gi_run_timed(gi_exec* e, const void* const* dev_inputs, void* const* dev_outputs, void* dev_arena,
                       size_t arena_bytes, void* stream, float* op_ms, int32_t n_op_ms) {
  if (!e || !op_ms) return fail(GI_E_INVALID, "gi_run_timed: null argument");
  const size_t n = e->launches.size();
  if (n_op_ms < 0 || static_cast<size_t>(n_op_ms) < n) return fail(GI_E_INVALID, "gi_run_timed: op_ms too short");
  std::vector<cudaEvent_t> ev(n + 1, nullptr);
  gi_status st = GI_OK;
  for (size_t i = 0; i <= n && st == GI_OK; ++i)
    if (cudaEventCreate(&ev[i]) != cudaSuccess) st = fail(GI_E_CUDA, "gi_run_timed: cudaEventCreate failed");
  if (st == GI_OK) st = run_impl(e, dev_inputs, dev_outputs, dev_arena, arena_bytes, stream, ev.data());
  if (st == GI_OK) {
    const cudaError_t err = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) st = fail(GI_E_CUDA, std::string("gi_run_timed: ") + cudaGetErrorString(err));
  }
  if (st == GI_OK)
    for (size_t i = 0; i < n; ++i)
      if (cudaEventElapsedTime(&op_ms[i], ev[i], ev[i + 1]) != cudaSuccess) op_ms[i] = -1.0f;
  for (cudaEvent_t x : ev)
    if (x) cudaEventDestroy(x);
  return st;
}

// ---- layout experiment: 1x1 convolution on tensors in slices of eight channels
uint64_t gi_slice8_tensor_bytes(int32_t batch, int32_t H, int32_t W, int32_t C) {
  if (batch <= 0 || H <= 0 || W <= 0 || C <= 0) return 0;
  return static_cast<uint64_t>((C + 7) / 8) * batch * plane_pixels(H, W) * 16u;
}

namespace {
gi_status slice8_shape(const char* who, int32_t cin, int32_t cout) {
  if (cin <= 0 || cout <= 0) return fail(GI_E_INVALID, std::string(who) + ": cin and cout must be positive");
  if (!pointwise_mm_supported(cin, cout)) return fail(GI_E_UNSUPPORTED, std::string(who) + ": shape not supported by the wide-tile kernel");
  return GI_OK;
}
}  // namespace

// the blob: packed weights at offset 0, bias behind them (256-byte aligned), exactly as pointwise_mm_pack lays them out
gi_status gi_slice8_pointwise_blob_bytes(int32_t cin, int32_t cout, uint64_t* bytes) {
  if (!bytes) return fail(GI_E_INVALID, "gi_slice8_pointwise_blob_bytes: null argument");
  const gi_status st = slice8_shape("gi_slice8_pointwise_blob_bytes", cin, cout);
  if (st != GI_OK) return st;
  uint64_t boff = 0;
  pointwise_mm_blob_layout(cin, cout, &boff, bytes);
  return GI_OK;
}

gi_status gi_slice8_pointwise_pack(const float* w, const float* bias, int32_t cin, int32_t cout, void* host_blob, uint64_t blob_bytes) {
  if (!w || !bias || !host_blob) return fail(GI_E_INVALID, "gi_slice8_pointwise_pack: null argument");
  const gi_status st = slice8_shape("gi_slice8_pointwise_pack", cin, cout);
  if (st != GI_OK) return st;
  try {
    std::vector<uint8_t> blob;
    LaunchRec r{};
    pointwise_mm_pack(w, bias, cin, cout, &blob, &r);
    if (blob_bytes < blob.size()) return fail(GI_E_INVALID, "gi_slice8_pointwise_pack: host_blob too small");
    std::memcpy(host_blob, blob.data(), blob.size());
    return GI_OK;
  } catch (const std::bad_alloc&) {
    return fail(GI_E_NOMEM, "gi_slice8_pointwise_pack: out of memory");
  }
}

gi_status gi_slice8_pointwise_run(const void* dev_in, void* dev_out, const void* dev_blob, int32_t batch, int32_t H, int32_t W,
                                  int32_t cin, int32_t cout, int32_t act, void* stream) {
  if (!dev_in || !dev_out || !dev_blob) return fail(GI_E_INVALID, "gi_slice8_pointwise_run: null argument");
  if (batch <= 0 || H <= 0 || W <= 0 || cin <= 0 || cout <= 0) return fail(GI_E_INVALID, "gi_slice8_pointwise_run: sizes must be positive");
  if (act != GI_ACT_NONE && act != GI_ACT_RELU && act != GI_ACT_RELU6) return fail(GI_E_INVALID, "gi_slice8_pointwise_run: unknown activation");
  if ((reinterpret_cast<uintptr_t>(dev_in) | reinterpret_cast<uintptr_t>(dev_out)) & 15u)
    return fail(GI_E_INVALID, "gi_slice8_pointwise_run: tensors must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(dev_blob) & 255u) return fail(GI_E_INVALID, "gi_slice8_pointwise_run: the blob must be 256-byte aligned");
  if (!pointwise_mm_supported(cin, cout)) return fail(GI_E_UNSUPPORTED, "gi_slice8_pointwise_run: shape not supported by the wide-tile kernel");
  const uint64_t m_total = static_cast<uint64_t>(batch) * plane_pixels(H, W);
  if (m_total >= (1ull << 31)) return fail(GI_E_UNSUPPORTED, "gi_slice8_pointwise_run: tensor too large");
  uint64_t boff = 0, total = 0;
  pointwise_mm_blob_layout(cin, cout, &boff, &total);
  const unsigned char* blob = static_cast<const unsigned char*>(dev_blob);
  const int err = launch_pointwise_mm_slice8(dev_in, dev_out, blob, reinterpret_cast<const float*>(blob + boff),
                                             static_cast<unsigned>(m_total), cin, cout, act, stream);
  if (err != 0) return fail(GI_E_CUDA, std::string("gi_slice8_pointwise_run: ") + cudaGetErrorString(static_cast<cudaError_t>(err)));
  return GI_OK;
}

}  // extern "C"

#ifdef GI_TRACE
namespace gi {
int pointwise_ts_trace(unsigned long long* dst, int n);
int depthwise_pointwise_trace(unsigned long long* dst, int n);
int inverted_residual_trace(unsigned long long* dst, int n);
int pointwise_chain_trace(unsigned long long* dst, int n);
}
// debug builds only: copy the timeline table of the lane-per-pixel kernel's last launch
extern "C" GI_API int gi_debug_trace(int which, unsigned long long* dst, int n) {
  return which == 3 ? gi::pointwise_chain_trace(dst, n) : which == 2 ? gi::inverted_residual_trace(dst, n) : which == 1 ? gi::depthwise_pointwise_trace(dst, n) : gi::pointwise_ts_trace(dst, n);
}
#endif
