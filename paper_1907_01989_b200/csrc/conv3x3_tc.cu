// Full 3x3 convolution of a tensor with at most 4 channels (one input slice; the stem of the
// MobileNets) as an implicit GEMM on the tensor cores (Section 4, "For a 2D Convolution": each
// output iterates over the window and the input channels under it - here the window is unrolled
// into the K axis).
//
//   D[pixel][co] = sum_k A[pixel][k] * B[co][k],   k = tap * 4 + ci  (36 values, padded to 48)
//
// A tile of 128 output pixels is one TMEM lane per pixel.  The 128 gather threads read the nine
// 8-byte taps of their pixel from the channel-sliced input (zero outside the image) and write
// them, two taps per 16-byte unit, straight into the canonical K-major shared-memory operand
// layout; the weights sit in shared memory for the whole kernel.  Three tcgen05.mma (K = 16 each)
// produce the tile; the same 128 threads then read their lane from tensor memory, add the bias,
// apply the fused element-wise tail and store 8 bytes per output slice (256 contiguous bytes per
// warp).  Operand tiles and accumulators are double-buffered: the gather of tile i+1 runs while
// the MMAs of tile i are in flight.  Waits are bounded like in the pointwise kernel.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kRows = 128;            // output pixels per tile
constexpr int kKCores = 6;            // 48 / 8: 16-byte K units per row
constexpr int kABytes = kKCores * kRows * 16;
constexpr int kGatherThreads = 128;
constexpr int kThreads = kGatherThreads + 32;
constexpr int kMaxN = 256;

__device__ unsigned int g_conv_tc_error = 0;

struct StemParams {
  const __half* in;
  const __half* res;
  __half* out;
  const unsigned char* wts;  // [6][n_pad][8] fp16
  const float* bias;         // [n_pad]
  int B, H, W, Pin, Ho, Wo, Pout;
  int stride, dil, pt, pl;
  int s_out, n_pad;          // output slices; Cout rounded up to a multiple of 16
  int tiles;                 // ceil(B * Pout / 128)
  int act_pre, has_res, act_post;
  unsigned tmem_cols;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long a_full[2];
  unsigned long long acc_full[2];
  unsigned tmem_addr;
  unsigned abort_flag;
};

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

__global__ void __launch_bounds__(kThreads, 2) conv3x3_tc_kernel(const StemParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  unsigned char* a_tiles = smem + 1024;                 // 2 x kABytes
  unsigned char* b_tile = a_tiles + 2 * kABytes;        // 6 * n_pad * 16
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kGatherThreads);
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) tmem_alloc(smem_u32(&hdr->tmem_addr), p.tmem_cols);
  // weights: plain copy into shared memory, then made visible to the tensor core's proxy
  for (int i = threadIdx.x; i < kKCores * p.n_pad; i += kThreads)
    reinterpret_cast<uint4*>(b_tile)[i] = __ldg(reinterpret_cast<const uint4*>(p.wts) + i);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // everything above touched only weights and on-chip state; the activations come after the wait
  pdl_launch_dependents();
  pdl_wait();
  const unsigned tmem_base = hdr->tmem_addr;
  const unsigned n_cols = static_cast<unsigned>(p.n_pad);
  const long long m_total = static_cast<long long>(p.B) * p.Pout;

  if (warp < 4) {
    const int t = threadIdx.x;  // row of the tile = TMEM lane
    // ---- gather of one tile into operand buffer `buf`
    auto gather = [&](int tile, int buf) {
      const long long gp = static_cast<long long>(tile) * kRows + t;
      uint2 tap[10];
#pragma unroll
      for (int k = 0; k < 10; ++k) tap[k] = make_uint2(0u, 0u);
      if (gp < m_total) {
        const int b = static_cast<int>(gp / p.Pout), q = static_cast<int>(gp - static_cast<long long>(b) * p.Pout);
        if (q < p.Ho * p.Wo) {
          const int oy = q / p.Wo, ox = q - oy * p.Wo;
          const __half* plane = p.in + static_cast<size_t>(b) * p.Pin * 4;
#pragma unroll
          for (int ky = 0; ky < 3; ++ky) {
            const int iy = oy * p.stride - p.pt + ky * p.dil;
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
              const int ix = ox * p.stride - p.pl + kx * p.dil;
              if (iy >= 0 && iy < p.H && ix >= 0 && ix < p.W)
                tap[ky * 3 + kx] = __ldg(reinterpret_cast<const uint2*>(plane + (static_cast<size_t>(iy) * p.W + ix) * 4));
            }
          }
        }
      }
      uint4* dst = reinterpret_cast<uint4*>(a_tiles + buf * kABytes) + t;
#pragma unroll
      for (int j = 0; j < 5; ++j) dst[j * kRows] = make_uint4(tap[2 * j].x, tap[2 * j].y, tap[2 * j + 1].x, tap[2 * j + 1].y);
      dst[5 * kRows] = make_uint4(0u, 0u, 0u, 0u);
      // generic-proxy writes above must be visible to the MMA (async proxy) before the arrival
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&hdr->a_full[buf]));
    };
    // ---- epilogue of one tile from accumulator `buf`
    auto epilogue = [&](int tile, int buf, unsigned phase) -> bool {
      if (!mbar_wait(smem_u32(&hdr->acc_full[buf]), phase, abort_flag, p.timeout_ns, &g_conv_tc_error, 4u)) return false;
      tc_fence_after();
      const long long gp = static_cast<long long>(tile) * kRows + t;
      const bool in_tensor = gp < m_total;
      bool real = false;
      if (in_tensor) {
        const int b = static_cast<int>(gp / p.Pout);
        real = static_cast<int>(gp - static_cast<long long>(b) * p.Pout) < p.Ho * p.Wo;
      }
      const unsigned t_addr = tmem_base + buf * n_cols + (static_cast<unsigned>(warp * 32) << 16);
      for (unsigned c0 = 0; c0 < n_cols; c0 += 16) {
        unsigned r[16];
        tmem_ld16(t_addr + c0, r);
        tmem_ld_wait16(r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int so = static_cast<int>(c0 / 4) + j;
          if (so >= p.s_out || !in_tensor) continue;
          const size_t off = (static_cast<size_t>(so) * m_total + gp) * 4;  // in halves
          uint2 o = make_uint2(0u, 0u);  // the padding pixel of an odd plane stays zero
          if (real) {
            const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias) + so);
            float v[4] = {__uint_as_float(r[4 * j]) + bv.x, __uint_as_float(r[4 * j + 1]) + bv.y,
                          __uint_as_float(r[4 * j + 2]) + bv.z, __uint_as_float(r[4 * j + 3]) + bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = act1(v[e], p.act_pre);
            if (p.has_res) {
              const uint2 q = __ldg(reinterpret_cast<const uint2*>(p.res + off));
              const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
              const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
              v[0] += r0.x;
              v[1] += r0.y;
              v[2] += r1.x;
              v[3] += r1.y;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = act1(v[e], p.act_post);
            const __half2 lo = __floats2half2_rn(v[0], v[1]), hi = __floats2half2_rn(v[2], v[3]);
            o.x = *reinterpret_cast<const unsigned*>(&lo);
            o.y = *reinterpret_cast<const unsigned*>(&hi);
          }
          *reinterpret_cast<uint2*>(p.out + off) = o;
        }
      }
      tc_fence_before();
      return true;
    };

    // software pipeline over this CTA's tiles: gather(i+1) is issued before epilogue(i)
    int n = 0;
    int prev_tile = -1;
    for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++n) {
      // operand buffer n&1 was read by the MMAs of tile n-2, whose accumulator the epilogue of
      // tile n-2 has already waited for, so the buffer is free
      gather(tile, n & 1);
      if (prev_tile >= 0 && !epilogue(prev_tile, (n - 1) & 1, ((n - 1) >> 1) & 1)) {
        prev_tile = -1;
        break;
      }
      prev_tile = tile;
    }
    if (prev_tile >= 0) epilogue(prev_tile, (n - 1) & 1, ((n - 1) >> 1) & 1);
  } else if (lane == 0) {
    // ---- MMA issuer
    // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = n_pad
    const unsigned idesc = (1u << 4) | ((n_cols >> 3) << 17) | ((kRows >> 4) << 24);
    const unsigned b_base = smem_u32(b_tile), b_lbo = n_cols * 16u;
    int n = 0;
    for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++n) {
      const int buf = n & 1;
      // the accumulator buffer was drained by the epilogue of tile n-2 before the gather threads
      // arrived for tile n (they run gather(n) after epilogue(n-2)), so waiting for the operands
      // also orders the accumulator reuse
      if (!mbar_wait(smem_u32(&hdr->a_full[buf]), (n >> 1) & 1, abort_flag, p.timeout_ns, &g_conv_tc_error, 2u)) break;
      tc_fence_after();
      const unsigned a_base = smem_u32(a_tiles + buf * kABytes);
#pragma unroll
      for (int ks = 0; ks < 3; ++ks) {
        const unsigned long long ad = smem_desc(a_base + ks * 2 * kRows * 16, kRows * 16, 128);
        const unsigned long long bd = smem_desc(b_base + ks * 2 * b_lbo, b_lbo, 128);
        umma_f16(tmem_base + buf * n_cols, ad, bd, idesc, ks > 0 ? 1u : 0u);
      }
      umma_commit(smem_u32(&hdr->acc_full[buf]));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace

bool conv3x3_tc_supported(int cin, int cout, int kh, int kw, int sh, int sw, int dh, int dw) {
  return kh == 3 && kw == 3 && cin <= 4 && cout >= 1 && cout <= kMaxN && sh == sw && dh == dw;
}

// Weights as the B operand: [6 K units][n_pad rows][8 halves], k = unit * 8 + e = tap * 4 + ci.
void conv3x3_tc_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const int n_pad = (cout + 15) / 16 * 16;
  const size_t wbytes = static_cast<size_t>(kKCores) * n_pad * 16;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(n_pad) * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) {
    bp[co] = bias[co];
    for (int tap = 0; tap < 9; ++tap)
      for (int ci = 0; ci < cin; ++ci) {
        const int k = tap * 4 + ci;
        wp[(static_cast<size_t>(k / 8) * n_pad + co) * 8 + k % 8] = f32_to_f16_rne(w[(static_cast<size_t>(co) * 9 + tap) * cin + ci]);
      }
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = n_pad;
}

int launch_conv3x3_tc(const LaunchRec& r, const Ptrs& p, void* stream) {
  StemParams k;
  k.in = static_cast<const __half*>(p.in0);
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.bias = static_cast<const float*>(p.bias);
  k.B = r.B;
  k.H = r.H;
  k.W = r.W;
  k.Pin = plane_pixels(r.H, r.W);
  k.Ho = r.Ho;
  k.Wo = r.Wo;
  k.Pout = plane_pixels(r.Ho, r.Wo);
  k.stride = r.sh;
  k.dil = r.dh;
  k.pt = r.pt;
  k.pl = r.pl;
  k.s_out = slices(r.Co);
  k.n_pad = r.tc_nt;
  const long long m_total = static_cast<long long>(r.B) * k.Pout;
  const long long tiles = (m_total + kRows - 1) / kRows;
  if (tiles > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  k.tiles = static_cast<int>(tiles);
  k.act_pre = r.ep.act_pre;
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  unsigned cols = 32;
  while (cols < static_cast<unsigned>(2 * k.n_pad)) cols <<= 1;
  k.tmem_cols = cols;
  k.timeout_ns = 1000000000u;
  static int sms = 0;
  static bool attr_set = false;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const size_t smem = 1024 + 2 * kABytes + static_cast<size_t>(kKCores) * k.n_pad * 16;
  if (!attr_set) {
    const cudaError_t e = cudaFuncSetAttribute(conv3x3_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               1024 + 2 * kABytes + kKCores * kMaxN * 16);
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  // a few CTAs per SM: one CTA's gather latency hides behind another's epilogue; tensor memory
  // allows 512 / tmem_cols of them
  int per_sm = static_cast<int>(512u / cols);
  if (per_sm > 8) per_sm = 8;
  if (per_sm < 1) per_sm = 1;
  long long grid = static_cast<long long>(sms) * per_sm;
  if (grid > tiles) grid = tiles;
  launch_pdl(conv3x3_tc_kernel, static_cast<unsigned>(grid), kThreads, smem, static_cast<cudaStream_t>(stream), k);
  return static_cast<int>(cudaGetLastError());
}

unsigned int conv3x3_tc_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_conv_tc_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
