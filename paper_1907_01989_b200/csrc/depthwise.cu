// Depthwise 3x3 convolution for fp16 storage: a bandwidth-bound stencil.
//
// A CTA owns a band of output rows in a few planes (plane = one 4-channel slice of one image;
// the planes of one slice are adjacent in memory, so they share the slice's 36 weights).  The
// input rows the band needs - its halo included - are one contiguous run per plane and are staged
// into shared memory by bulk asynchronous copies (16-byte aligned, one mbarrier).  Each thread then
// walks down one output column, keeping a sliding window of input rows in registers, so every
// input pixel-slice is read from HBM once, from shared memory three times, and is converted to
// fp32 once per use; stores are 8 bytes per lane, contiguous across the warp.  Zero padding is
// applied by predicates while the rows are fetched from shared memory.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"

namespace gi {
namespace {

__device__ unsigned int g_dw_error = 0;  // sticky: set if the staging copy did not arrive in time

struct DwGeom {
  int B, H, W, Pin, Ho, Wo, Pout, S;
  int stride, dil, pt, pl;
  int nb;       // planes per CTA
  int sub;      // sub-bands per CTA band (thread groups walking different rows of one plane)
  int tr;       // output rows walked by one thread
  int bands;    // CTA bands per plane
  int bchunks;  // ceil(B / nb)
  int plane_stride_px;  // pixels reserved per plane in shared memory (even)
  unsigned timeout_ns;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ float4 ld_px(const __half* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

__device__ __forceinline__ void fma4(float4& acc, const float4& x, const float4& w) {
  acc.x = fmaf(x.x, w.x, acc.x);
  acc.y = fmaf(x.y, w.y, acc.y);
  acc.z = fmaf(x.z, w.z, acc.z);
  acc.w = fmaf(x.w, w.w, acc.w);
}

struct Row {
  float4 v[3];
};

// MODE 0: stride 1, dilation 1 (one new input row per output row)
// MODE 1: stride 2, dilation 1 (two new input rows per output row)
// MODE 2: anything else (three rows fetched per output row)
template <int MODE>
__global__ void __launch_bounds__(512) depthwise_f16_kernel(const __half* __restrict__ in, const float* __restrict__ w,
                                                             const float* __restrict__ bias, const __half* __restrict__ res,
                                                             __half* __restrict__ out, const DwGeom g, const Epilogue ep) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bar;
  __half* tile = reinterpret_cast<__half*>(smem_raw);

  const int band = blockIdx.x % g.bands;
  const int bc = (blockIdx.x / g.bands) % g.bchunks;
  const int s = blockIdx.x / (g.bands * g.bchunks);
  const int b0 = bc * g.nb;
  const int nbk = min(g.nb, g.B - b0);
  const int th = g.sub * g.tr;
  const int oy0 = band * th, oy1 = min(g.Ho, oy0 + th);
  const int in_y0 = max(0, oy0 * g.stride - g.pt);
  const int in_y1 = min(g.H, (oy1 - 1) * g.stride - g.pt + 2 * g.dil + 1);
  int start_px = in_y0 * g.W;
  start_px -= start_px & 1;  // copies start on a 16-byte boundary: at most one pixel early
  const int end_px = min((in_y1 * g.W + 1) & ~1, g.Pin);
  const unsigned copy_bytes = static_cast<unsigned>(end_px - start_px) * 8u;
  const unsigned bar_addr = smem_u32(&bar);

  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(copy_bytes * nbk) : "memory");
    for (int pi = 0; pi < nbk; ++pi) {
      const __half* src = in + ((static_cast<size_t>(s) * g.B + b0 + pi) * g.Pin + start_px) * 4;
      const unsigned dst = smem_u32(tile + static_cast<size_t>(pi) * g.plane_stride_px * 4);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                   "r"(copy_bytes), "r"(bar_addr)
                   : "memory");
    }
  }
  // weights of this slice: 9 taps x 4 channels, kept in registers
  float4 wt[9];
  const int C4 = g.S * 4;
#pragma unroll
  for (int t = 0; t < 9; ++t) wt[t] = __ldg(reinterpret_cast<const float4*>(w + t * C4 + s * 4));
  const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + s * 4));
  __syncthreads();  // the barrier is initialised before anyone polls it

  {  // bounded wait for the staged rows
    unsigned ok = 0;
    unsigned long long t0 = 0;
    for (unsigned spin = 0; !ok; ++spin) {
      asm volatile(
          "{\n\t.reg .pred p;\n\t"
          "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(ok)
          : "r"(bar_addr)
          : "memory");
      if (!ok && (spin & 255u) == 255u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (t0 == 0) {
          t0 = now;
        } else if (now - t0 > g.timeout_ns) {
          atomicOr(&g_dw_error, 1u);
          return;
        }
      }
    }
  }

  const int cols = nbk * g.sub * g.Wo;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const int x = c % g.Wo, vp = c / g.Wo;
    const int sb = vp % g.sub, pi = vp / g.sub;
    const int ya = oy0 + sb * g.tr, yb = min(oy1, ya + g.tr);
    if (ya >= yb) continue;
    const int base_px = pi * g.plane_stride_px - start_px;  // pixel (iy, ix) is staged at base_px + iy*W + ix
    // column offsets and validity of the three taps
    int ix[3];
    bool vx[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      ix[k] = x * g.stride - g.pl + k * g.dil;
      vx[k] = ix[k] >= 0 && ix[k] < g.W;
    }
    auto fetch = [&](int iy) {
      Row r;
      const bool vy = iy >= 0 && iy < g.H;
      const int row_px = base_px + iy * g.W;
#pragma unroll
      for (int k = 0; k < 3; ++k) r.v[k] = (vy && vx[k]) ? ld_px(tile + (row_px + ix[k]) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      return r;
    };
    const size_t out_plane = (static_cast<size_t>(s) * g.B + b0 + pi) * g.Pout;
    auto emit = [&](int oy, const Row& r0, const Row& r1, const Row& r2) {
      float4 acc = bv;
#pragma unroll
      for (int k = 0; k < 3; ++k) fma4(acc, r0.v[k], wt[k]);
#pragma unroll
      for (int k = 0; k < 3; ++k) fma4(acc, r1.v[k], wt[3 + k]);
#pragma unroll
      for (int k = 0; k < 3; ++k) fma4(acc, r2.v[k], wt[6 + k]);
      acc = make_float4(act1(acc.x, ep.act_pre), act1(acc.y, ep.act_pre), act1(acc.z, ep.act_pre), act1(acc.w, ep.act_pre));
      const size_t off = (out_plane + static_cast<size_t>(oy) * g.Wo + x) * 4;
      if (ep.has_res) {
        const float4 r = ld_px(res + off);
        acc.x += r.x;
        acc.y += r.y;
        acc.z += r.z;
        acc.w += r.w;
      }
      acc = make_float4(act1(acc.x, ep.act_post), act1(acc.y, ep.act_post), act1(acc.z, ep.act_post), act1(acc.w, ep.act_post));
      const __half2 lo = __floats2half2_rn(acc.x, acc.y), hi = __floats2half2_rn(acc.z, acc.w);
      uint2 u;
      u.x = *reinterpret_cast<const unsigned*>(&lo);
      u.y = *reinterpret_cast<const unsigned*>(&hi);
      *reinterpret_cast<uint2*>(out + off) = u;
    };
    if (MODE == 0) {
      Row r0 = fetch(ya - g.pt), r1 = fetch(ya - g.pt + 1);
      for (int oy = ya; oy < yb; ++oy) {
        const Row r2 = fetch(oy - g.pt + 2);
        emit(oy, r0, r1, r2);
        r0 = r1;
        r1 = r2;
      }
    } else if (MODE == 1) {
      Row r0 = fetch(ya * 2 - g.pt);
      for (int oy = ya; oy < yb; ++oy) {
        const Row r1 = fetch(oy * 2 - g.pt + 1), r2 = fetch(oy * 2 - g.pt + 2);
        emit(oy, r0, r1, r2);
        r0 = r2;
      }
    } else {
      for (int oy = ya; oy < yb; ++oy) {
        const int iy = oy * g.stride - g.pt;
        emit(oy, fetch(iy), fetch(iy + g.dil), fetch(iy + 2 * g.dil));
      }
    }
  }
  // an odd plane carries one extra pixel: keep it zero
  if (band == g.bands - 1 && g.Pout > g.Ho * g.Wo && threadIdx.x < nbk) {
    const size_t off = ((static_cast<size_t>(s) * g.B + b0 + threadIdx.x) * g.Pout + g.Ho * g.Wo) * 4;
    *reinterpret_cast<uint2*>(out + off) = make_uint2(0u, 0u);
  }
}

constexpr int kMaxSmem = 160 * 1024;

}  // namespace

int launch_depthwise_f16(const LaunchRec& r, const Ptrs& p, void* stream) {
  DwGeom g;
  g.B = r.B;
  g.H = r.H;
  g.W = r.W;
  g.Pin = plane_pixels(r.H, r.W);
  g.Ho = r.Ho;
  g.Wo = r.Wo;
  g.Pout = plane_pixels(r.Ho, r.Wo);
  g.S = slices(r.C);
  g.stride = r.sh;
  g.dil = r.dh;
  g.pt = r.pt;
  g.pl = r.pl;
  g.timeout_ns = 1000000000u;
  // thread groups: as many "virtual planes" (plane x sub-band) as fit in ~256 threads
  int vp = 256 / g.Wo;
  if (vp < 1) vp = 1;
  g.nb = vp < g.B ? vp : g.B;
  g.sub = vp / g.nb;
  if (g.sub < 1) g.sub = 1;
  const int tr_target = g.stride == 1 ? 16 : 8;
  int total_sub = (g.Ho + tr_target - 1) / tr_target;
  if (total_sub < g.sub) g.sub = total_sub;
  g.tr = (g.Ho + total_sub - 1) / total_sub;
  g.bands = (total_sub + g.sub - 1) / g.sub;
  auto smem_for = [&](const DwGeom& q) {
    const int th = q.sub * q.tr;
    const int rows_in = (th - 1) * q.stride + 2 * q.dil + 1;
    int px = (rows_in < q.H ? rows_in : q.H) * q.W + 2;
    if (px > q.Pin) px = q.Pin;
    return (px + 1) & ~1;
  };
  g.plane_stride_px = smem_for(g);
  // shrink until the staging buffer fits
  while (static_cast<long long>(g.plane_stride_px) * 8 * g.nb > kMaxSmem && (g.nb > 1 || g.sub > 1 || g.tr > 1)) {
    if (g.nb > 1) {
      g.nb = (g.nb + 1) / 2;
    } else if (g.sub > 1) {
      g.sub = (g.sub + 1) / 2;
    } else {
      g.tr = (g.tr + 1) / 2;
    }
    total_sub = (g.Ho + g.tr - 1) / g.tr;
    g.bands = (total_sub + g.sub - 1) / g.sub;
    g.plane_stride_px = smem_for(g);
  }
  const size_t smem = static_cast<size_t>(g.plane_stride_px) * 8 * g.nb;
  if (smem > static_cast<size_t>(kMaxSmem)) return static_cast<int>(cudaErrorInvalidConfiguration);
  g.bchunks = (g.B + g.nb - 1) / g.nb;
  const long long blocks = static_cast<long long>(g.S) * g.bchunks * g.bands;
  if (blocks > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  int threads = (g.nb * g.sub * g.Wo + 31) / 32 * 32;
  if (threads > 512) threads = 512;
  if (threads < 32) threads = 32;
  const int mode = (g.stride == 1 && g.dil == 1 && r.sw == 1 && r.dw == 1) ? 0
                   : (g.stride == 2 && g.dil == 1 && r.sw == 2 && r.dw == 1) ? 1 : 2;
  static bool attr_done[3] = {false, false, false};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* in = static_cast<const __half*>(p.in0);
  const float* w = static_cast<const float*>(p.wts);
  const float* b = static_cast<const float*>(p.bias);
  const __half* res = static_cast<const __half*>(p.res);
  __half* out = static_cast<__half*>(p.out);
#define GI_DW_LAUNCH(M)                                                                                                \
  do {                                                                                                                 \
    if (!attr_done[M]) {                                                                                               \
      const cudaError_t e = cudaFuncSetAttribute(depthwise_f16_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem); \
      if (e != cudaSuccess) return static_cast<int>(e);                                                                \
      attr_done[M] = true;                                                                                             \
    }                                                                                                                  \
    depthwise_f16_kernel<M><<<static_cast<unsigned>(blocks), threads, smem, st>>>(in, w, b, res, out, g, r.ep);        \
  } while (0)
  if (mode == 0) {
    GI_DW_LAUNCH(0);
  } else if (mode == 1) {
    GI_DW_LAUNCH(1);
  } else {
    GI_DW_LAUNCH(2);
  }
#undef GI_DW_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

unsigned int depthwise_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_dw_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
