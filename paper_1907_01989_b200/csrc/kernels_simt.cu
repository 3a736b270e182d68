// CUDA-core kernels: layout conversion, depthwise 3x3, direct convolution, element-wise, channel
// concatenation, global average pool, bilinear resize.  All work on the channel-sliced layout
//   element (b,h,w,c) -> ((c/4 * B + b) * P + h*W + w) * 4 + c%4,   P = H*W rounded up to even,
// and move one pixel-slice (4 channels: 8 bytes fp16, 16 bytes fp32) per vector access, so a
// warp touches 32 consecutive pixels of one plane = one contiguous 256 / 512-byte run.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"

namespace gi {
namespace {

template <typename T>
struct Px;  // one pixel-slice in storage type T

template <>
struct Px<__half> {
  static __device__ __forceinline__ float4 load(const __half* p) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
  static __device__ __forceinline__ void store(__half* p, float4 v) {
    const __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<const unsigned*>(&a);
    u.y = *reinterpret_cast<const unsigned*>(&b);
    *reinterpret_cast<uint2*>(p) = u;
  }
  static __device__ __forceinline__ float get(const __half* p) { return __half2float(*p); }
  static __device__ __forceinline__ void put(__half* p, float v) { *p = __float2half_rn(v); }
};

template <>
struct Px<float> {
  static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
  static __device__ __forceinline__ void store(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
  static __device__ __forceinline__ float get(const float* p) { return *p; }
  static __device__ __forceinline__ void put(float* p, float v) { *p = v; }
};

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}
__device__ __forceinline__ float4 act4(float4 v, int kind) {
  return make_float4(act1(v.x, kind), act1(v.y, kind), act1(v.z, kind), act1(v.w, kind));
}

// bias is already in v: activation, residual add, activation, in graph order
template <typename T>
__device__ __forceinline__ float4 epilogue(float4 v, const Epilogue& ep, const T* res, size_t idx) {
  v = act4(v, ep.act_pre);
  if (ep.has_res) {
    const float4 r = Px<T>::load(res + idx);
    v.x += r.x;
    v.y += r.y;
    v.z += r.z;
    v.w += r.w;
  }
  return act4(v, ep.act_post);
}

// ------------------------------------------------------------------ layout conversion
// grid: x over the pixels of a plane (padding pixel included), y strides over planes (slice * B + image; a grid
// dimension holds at most 65535, deep tensors at large batch have more planes than that)
template <typename T>
__global__ void pack_kernel(const T* __restrict__ nhwc, T* __restrict__ out, int B, int HW, int C, int P, int S) {
  pdl_launch_dependents();
  pdl_wait();
  const int pix = blockIdx.x * blockDim.x + threadIdx.x;
  if (pix >= P) return;
  for (int plane = blockIdx.y; plane < S * B; plane += gridDim.y) {
    const int s = plane / B, b = plane - s * B;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (pix < HW) {
      const T* src = nhwc + (static_cast<size_t>(b) * HW + pix) * C + s * 4;
      const int n = min(4, C - s * 4);
      float t[4] = {0.f, 0.f, 0.f, 0.f};
      for (int j = 0; j < n; ++j) t[j] = Px<T>::get(src + j);
      v = make_float4(t[0], t[1], t[2], t[3]);
    }
    Px<T>::store(out + (static_cast<size_t>(plane) * P + pix) * 4, v);
  }
}

// fp16 images with 3 channels (the usual network input) whose pixel count is a multiple of 4:
// a thread turns 4 pixels (24 contiguous bytes, three 8-byte loads) into 4 pixel-slices (two
// 16-byte stores).  grid: x over quads of an image, y over images.
__global__ void pack3_f16_kernel(const uint2* __restrict__ nhwc, uint4* __restrict__ out, int quads) {
  pdl_launch_dependents();
  pdl_wait();
  const int q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= quads) return;
  const size_t at = static_cast<size_t>(blockIdx.y) * quads + q;
  const uint2 a = __ldg(nhwc + at * 3), c = __ldg(nhwc + at * 3 + 1), d = __ldg(nhwc + at * 3 + 2);
  // halves h0..h11 = a.x, a.y, c.x, c.y, d.x, d.y (two per word); pixel i takes h[3i .. 3i+2] and a zero
  uint4 lo, hi;
  lo.x = a.x;
  lo.y = a.y & 0xffffu;
  lo.z = (a.y >> 16) | (c.x << 16);
  lo.w = c.x >> 16;
  hi.x = c.y;
  hi.y = d.x & 0xffffu;
  hi.z = (d.x >> 16) | (d.y << 16);
  hi.w = d.y >> 16;
  out[at * 2] = lo;
  out[at * 2 + 1] = hi;
}

template <typename T>
__global__ void unpack_kernel(const T* __restrict__ in, T* __restrict__ nhwc, int B, int HW, int C, int P, int S) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t total = static_cast<size_t>(B) * HW * S;
  if (idx >= total) return;
  const int s = static_cast<int>(idx % S);
  const int pix = static_cast<int>((idx / S) % HW);
  const int b = static_cast<int>(idx / (static_cast<size_t>(S) * HW));
  const float4 v = Px<T>::load(in + ((static_cast<size_t>(s) * B + b) * P + pix) * 4);
  const float t[4] = {v.x, v.y, v.z, v.w};
  T* dst = nhwc + (static_cast<size_t>(b) * HW + pix) * C + s * 4;
  const int n = min(4, C - s * 4);
  for (int j = 0; j < n; ++j) Px<T>::put(dst + j, t[j]);
}

// fp16, any channel count: a block turns 128 consecutive pixels of one image into one contiguous
// run of 128 * C halves.  The pixel-slices are read coalesced (8 bytes per lane and slice) into
// shared memory in NHWC order; the run is then written with 4-byte stores (plus a 2-byte store at
// a misaligned head / tail) instead of one 2-byte store per element.  grid: x over 128-pixel
// chunks of an image, y over images; dynamic shared memory: 128 * C halves.
__global__ void __launch_bounds__(128) unpack_f16_kernel(const __half* __restrict__ in, __half* __restrict__ nhwc, int B, int HW, int C,
                                                         int P, int S) {
  extern __shared__ __align__(16) unsigned char unpack_smem[];
  unsigned short* tile = reinterpret_cast<unsigned short*>(unpack_smem);
  pdl_launch_dependents();
  pdl_wait();
  const int pix0 = blockIdx.x * 128, b = blockIdx.y;
  const int npx = min(128, HW - pix0);
  const int t = threadIdx.x;
  if (t < npx) {
    const uint2* src = reinterpret_cast<const uint2*>(in) + static_cast<size_t>(b) * P + pix0 + t;
    const size_t step = static_cast<size_t>(B) * P;
    unsigned short* dst = tile + t * C;
    for (int s = 0; s < S; ++s, src += step) {
      const uint2 u = __ldg(src);
      const unsigned short h[4] = {static_cast<unsigned short>(u.x & 0xffffu), static_cast<unsigned short>(u.x >> 16),
                                   static_cast<unsigned short>(u.y & 0xffffu), static_cast<unsigned short>(u.y >> 16)};
      const int n = min(4, C - s * 4);
      for (int j = 0; j < n; ++j) dst[s * 4 + j] = h[j];
    }
  }
  __syncthreads();
  const size_t first = (static_cast<size_t>(b) * HW + pix0) * C;  // in halves
  const int total = npx * C;
  unsigned short* out = reinterpret_cast<unsigned short*>(nhwc) + first;
  const int head = static_cast<int>(first & 1);  // halves before the first 4-byte boundary
  if (t == 0 && head) out[0] = tile[0];
  const int words = (total - head) / 2;
  unsigned* out32 = reinterpret_cast<unsigned*>(out + head);
  for (int w = t; w < words; w += 128) {
    const int i = head + 2 * w;
    out32[w] = static_cast<unsigned>(tile[i]) | (static_cast<unsigned>(tile[i + 1]) << 16);
  }
  if (t == 0 && ((total - head) & 1)) out[total - 1] = tile[total - 1];
}

// ------------------------------------------------------------------ direct convolution
struct ConvGeom {
  int B, H, W, Sin, Pin, Ho, Wo, Sout, Pout;
  int kh, kw, sh, sw, dh, dw, pt, pl;
};

// One thread = one output pixel x OS output slices.  Weights W[group][tap][in_slice][OS*4][4]
// are read with warp-uniform addresses (one broadcast L1 transaction per float4).
template <typename T, int OS>
__global__ void __launch_bounds__(128) conv_simt_kernel(const T* __restrict__ in, const float4* __restrict__ w,
                                                        const float* __restrict__ bias, const T* __restrict__ res,
                                                        T* __restrict__ out, ConvGeom g, Epilogue ep) {
  pdl_launch_dependents();
  pdl_wait();
  const int pix = blockIdx.x * 128 + threadIdx.x;
  const int grp = blockIdx.y, b = blockIdx.z;
  if (pix >= g.Pout) return;
  constexpr int JN = OS * 4;
  float acc[JN];
#pragma unroll
  for (int j = 0; j < JN; ++j) acc[j] = 0.f;
  const bool real = pix < g.Ho * g.Wo;
  if (real) {
    const int oy = pix / g.Wo, ox = pix - oy * g.Wo;
    const float4* wg = w + static_cast<size_t>(grp) * g.kh * g.kw * g.Sin * JN;
    for (int ky = 0; ky < g.kh; ++ky) {
      const int iy = oy * g.sh - g.pt + ky * g.dh;
      if (iy < 0 || iy >= g.H) continue;
      for (int kx = 0; kx < g.kw; ++kx) {
        const int ix = ox * g.sw - g.pl + kx * g.dw;
        if (ix < 0 || ix >= g.W) continue;
        const float4* wt = wg + static_cast<size_t>(ky * g.kw + kx) * g.Sin * JN;
        const T* ip = in + (static_cast<size_t>(b) * g.Pin + iy * g.W + ix) * 4;
        for (int s = 0; s < g.Sin; ++s) {
          const float4 x = Px<T>::load(ip + static_cast<size_t>(s) * g.B * g.Pin * 4);
          const float4* ws = wt + s * JN;
#pragma unroll
          for (int j = 0; j < JN; ++j) {
            const float4 wv = __ldg(ws + j);
            acc[j] = fmaf(x.x, wv.x, acc[j]);
            acc[j] = fmaf(x.y, wv.y, acc[j]);
            acc[j] = fmaf(x.z, wv.z, acc[j]);
            acc[j] = fmaf(x.w, wv.w, acc[j]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 0; o < OS; ++o) {
    const int so = grp * OS + o;
    if (so >= g.Sout) break;
    const size_t idx = ((static_cast<size_t>(so) * g.B + b) * g.Pout + pix) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (real) {
      const float4 bv = *reinterpret_cast<const float4*>(bias + (grp * OS + o) * 4);
      v = make_float4(acc[o * 4] + bv.x, acc[o * 4 + 1] + bv.y, acc[o * 4 + 2] + bv.z, acc[o * 4 + 3] + bv.w);
      v = epilogue<T>(v, ep, res, idx);
    }
    Px<T>::store(out + idx, v);
  }
}

// ------------------------------------------------------------------ depthwise 3x3
template <typename T>
__global__ void __launch_bounds__(128) depthwise_kernel(const T* __restrict__ in, const float* __restrict__ w,
                                                        const float* __restrict__ bias, const T* __restrict__ res,
                                                        T* __restrict__ out, ConvGeom g, Epilogue ep) {
  pdl_launch_dependents();
  pdl_wait();
  const int pix = blockIdx.x * 128 + threadIdx.x;
  const int s = blockIdx.y, b = blockIdx.z;
  if (pix >= g.Pout) return;
  const size_t idx = ((static_cast<size_t>(s) * g.B + b) * g.Pout + pix) * 4;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (pix < g.Ho * g.Wo) {
    const int oy = pix / g.Wo, ox = pix - oy * g.Wo;
    const int C4 = g.Sin * 4;
    v = *reinterpret_cast<const float4*>(bias + s * 4);
    const T* plane = in + (static_cast<size_t>(s) * g.B + b) * g.Pin * 4;
#pragma unroll
    for (int ky = 0; ky < 3; ++ky) {
      const int iy = oy * g.sh - g.pt + ky * g.dh;
      if (iy < 0 || iy >= g.H) continue;
#pragma unroll
      for (int kx = 0; kx < 3; ++kx) {
        const int ix = ox * g.sw - g.pl + kx * g.dw;
        if (ix < 0 || ix >= g.W) continue;
        const float4 x = Px<T>::load(plane + (static_cast<size_t>(iy) * g.W + ix) * 4);
        const float4 wv = __ldg(reinterpret_cast<const float4*>(w + (ky * 3 + kx) * C4 + s * 4));
        v.x = fmaf(x.x, wv.x, v.x);
        v.y = fmaf(x.y, wv.y, v.y);
        v.z = fmaf(x.z, wv.z, v.z);
        v.w = fmaf(x.w, wv.w, v.w);
      }
    }
    v = epilogue<T>(v, ep, res, idx);
  }
  Px<T>::store(out + idx, v);
}

// ------------------------------------------------------------------ element-wise
template <typename T>
__global__ void eltwise_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, size_t n_px,
                               Epilogue ep) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  if (i >= n_px) return;
  const float4 v = epilogue<T>(Px<T>::load(a + i * 4), ep, b, i * 4);
  Px<T>::store(out + i * 4, v);
}

// ------------------------------------------------------------------ channel concatenation
// grid: x over the pixels of all planes of one output slice (B * P), y over output slices.  Output channel c
// is channel c of `a` for c < Ca and channel c - Ca of `b` after that; lanes beyond Ca + Cb and the padding
// pixel of a plane are written as zeros.  With Ca a multiple of 4 every output slice is one whole input
// slice (one vector load); otherwise each lane is fetched from the slice that holds it.
template <typename T>
__global__ void concat_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, size_t n_px, int P, int HW,
                              int Ca, int Cb) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  if (i >= n_px) return;
  const int so = blockIdx.y, c0 = so * 4;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (static_cast<int>(i % P) < HW) {
    if ((Ca & 3) == 0) {
      const bool from_a = c0 < Ca;
      const T* src = from_a ? a + (static_cast<size_t>(so) * n_px + i) * 4 : b + (static_cast<size_t>(so - Ca / 4) * n_px + i) * 4;
      v = Px<T>::load(src);
      const int valid = (from_a ? Ca : Ca + Cb) - c0;  // channels of this slice that exist
      if (valid < 4) v.w = 0.f;
      if (valid < 3) v.z = 0.f;
      if (valid < 2) v.y = 0.f;
    } else {
      float lane[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + j;
        lane[j] = 0.f;
        if (c < Ca) lane[j] = Px<T>::get(a + (static_cast<size_t>(c >> 2) * n_px + i) * 4 + (c & 3));
        else if (c < Ca + Cb) lane[j] = Px<T>::get(b + (static_cast<size_t>((c - Ca) >> 2) * n_px + i) * 4 + ((c - Ca) & 3));
      }
      v = make_float4(lane[0], lane[1], lane[2], lane[3]);
    }
  }
  Px<T>::store(out + (static_cast<size_t>(so) * n_px + i) * 4, v);
}

// ------------------------------------------------------------------ global average pool
// eight lanes per (slice, image), four planes per warp: a lane strides over the pixels with all its
// loads independent (many small planes are latency-bound otherwise), then a shuffle reduction over
// the eight lanes in a fixed order
template <typename T>
__global__ void pool_kernel(const T* __restrict__ in, T* __restrict__ out, int planes, int HW, int Pin, int Pout) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, sub = lane & 7;
  const int plane_id = ((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 4 + (lane >> 3);
  const bool live = plane_id < planes;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (live) {
    const T* plane = in + static_cast<size_t>(plane_id) * Pin * 4;
    int p = sub;
    for (; p + 24 < HW; p += 32) {  // four loads in flight
      const float4 x0 = Px<T>::load(plane + static_cast<size_t>(p) * 4), x1 = Px<T>::load(plane + static_cast<size_t>(p + 8) * 4);
      const float4 x2 = Px<T>::load(plane + static_cast<size_t>(p + 16) * 4), x3 = Px<T>::load(plane + static_cast<size_t>(p + 24) * 4);
      s.x += (x0.x + x1.x) + (x2.x + x3.x);
      s.y += (x0.y + x1.y) + (x2.y + x3.y);
      s.z += (x0.z + x1.z) + (x2.z + x3.z);
      s.w += (x0.w + x1.w) + (x2.w + x3.w);
    }
    for (; p < HW; p += 8) {
      const float4 x = Px<T>::load(plane + static_cast<size_t>(p) * 4);
      s.x += x.x;
      s.y += x.y;
      s.z += x.z;
      s.w += x.w;
    }
  }
  for (int d = 4; d > 0; d >>= 1) {
    s.x += __shfl_down_sync(0xffffffffu, s.x, d, 8);
    s.y += __shfl_down_sync(0xffffffffu, s.y, d, 8);
    s.z += __shfl_down_sync(0xffffffffu, s.z, d, 8);
    s.w += __shfl_down_sync(0xffffffffu, s.w, d, 8);
  }
  if (live && sub < Pout) {
    const float inv = 1.0f / static_cast<float>(HW);
    const float4 v = sub == 0 ? make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv) : make_float4(0.f, 0.f, 0.f, 0.f);
    Px<T>::store(out + (static_cast<size_t>(plane_id) * Pout + sub) * 4, v);
  }
}

// ------------------------------------------------------------------ bilinear resize
// source coordinate as an exact fraction num/den so that floor() never depends on rounding.
// grid: x over the columns of a row, y = SOURCE row y0, z = image.  All output rows whose upper
// source row is y0 share the four source pixels of a column, so a thread interpolates along x once
// per slice (top, bottom - top) and then emits every such output row with one FMA per channel;
// the row weights are block-uniform and live in shared memory.  I is the integer type of the
// coordinate products (32 bits whenever OH*ny and OW*nx fit: 64-bit divisions are emulated).
constexpr int kResizeRows = 32;
template <typename T, typename I>
__global__ void __launch_bounds__(128) resize_kernel(const T* __restrict__ in, T* __restrict__ out, int B, int S, int H, int W,
                                                     int Pin, int OH, int OW, int Pout, int ny, int dy, int nx, int dx) {
  __shared__ float wy_s[kResizeRows];
  pdl_launch_dependents();
  pdl_wait();
  const int ox = blockIdx.x * 128 + threadIdx.x, y0 = blockIdx.y;
  const bool active = ox < OW;
  // output rows oy with floor(oy * ny / dy) == y0
  int oy_lo, oy_hi;
  if (ny == 0) {
    oy_lo = 0;
    oy_hi = y0 == 0 ? OH : 0;
  } else {
    oy_lo = static_cast<int>((static_cast<I>(y0) * static_cast<I>(dy) + static_cast<I>(ny - 1)) / static_cast<I>(ny));
    const I hi = (static_cast<I>(y0 + 1) * static_cast<I>(dy) + static_cast<I>(ny - 1)) / static_cast<I>(ny);
    oy_hi = hi > static_cast<I>(OH) ? OH : static_cast<int>(hi);
  }
  const int y1 = min(y0 + 1, H - 1);
  // column: source pixel pair and weight
  int x0 = 0, x1 = 0;
  float wx = 0.f;
  if (active) {
    const I qx = static_cast<I>(ox) * static_cast<I>(nx);
    x0 = static_cast<int>(qx / static_cast<I>(dx));
    wx = static_cast<float>(qx - static_cast<I>(x0) * static_cast<I>(dx)) / static_cast<float>(dx);
    if (x0 > W - 1) {
      x0 = W - 1;
      wx = 0.f;
    }
    x1 = min(x0 + 1, W - 1);
  }
  const int o00 = (y0 * W + x0) * 4, o01 = (y0 * W + x1) * 4, o10 = (y1 * W + x0) * 4, o11 = (y1 * W + x1) * 4;
  const size_t in_step = static_cast<size_t>(B) * Pin * 4, out_step = static_cast<size_t>(B) * Pout * 4;
  const bool pad_col = ox == OW - 1 && Pout > OH * OW;  // an odd plane carries one extra pixel: keep it zero
  for (int base = oy_lo; base < oy_hi; base += kResizeRows) {
    const int cnt = min(kResizeRows, oy_hi - base);
    __syncthreads();  // the previous chunk's weights are no longer needed
    if (static_cast<int>(threadIdx.x) < cnt) {
      const I py = static_cast<I>(base + threadIdx.x) * static_cast<I>(ny);
      wy_s[threadIdx.x] = static_cast<float>(py - static_cast<I>(y0) * static_cast<I>(dy)) / static_cast<float>(dy);
    }
    __syncthreads();
    if (!active) continue;
    const T* plane = in + static_cast<size_t>(blockIdx.z) * Pin * 4;
    T* orow = out + static_cast<size_t>(blockIdx.z) * Pout * 4 + (static_cast<size_t>(base) * OW + ox) * 4;
    for (int s = 0; s < S; ++s, plane += in_step, orow += out_step) {
      const float4 a = Px<T>::load(plane + o00), c = Px<T>::load(plane + o01), d = Px<T>::load(plane + o10), e = Px<T>::load(plane + o11);
      const float4 top = make_float4(fmaf(c.x - a.x, wx, a.x), fmaf(c.y - a.y, wx, a.y), fmaf(c.z - a.z, wx, a.z), fmaf(c.w - a.w, wx, a.w));
      const float4 bot = make_float4(fmaf(e.x - d.x, wx, d.x), fmaf(e.y - d.y, wx, d.y), fmaf(e.z - d.z, wx, d.z), fmaf(e.w - d.w, wx, d.w));
      const float4 dif = make_float4(bot.x - top.x, bot.y - top.y, bot.z - top.z, bot.w - top.w);
      T* o = orow;
      for (int r = 0; r < cnt; ++r, o += static_cast<size_t>(OW) * 4) {
        const float wy = wy_s[r];
        Px<T>::store(o, make_float4(fmaf(dif.x, wy, top.x), fmaf(dif.y, wy, top.y), fmaf(dif.z, wy, top.z), fmaf(dif.w, wy, top.w)));
      }
      if (pad_col && base + cnt == OH) Px<T>::store(o - static_cast<size_t>(OW) * 4 + 4, make_float4(0.f, 0.f, 0.f, 0.f));
    }
  }
}

ConvGeom geom(const LaunchRec& r) {
  ConvGeom g;
  g.B = r.B;
  g.H = r.H;
  g.W = r.W;
  g.Sin = slices(r.C);
  g.Pin = plane_pixels(r.H, r.W);
  g.Ho = r.Ho;
  g.Wo = r.Wo;
  g.Sout = slices(r.Co);
  g.Pout = plane_pixels(r.Ho, r.Wo);
  g.kh = r.kh;
  g.kw = r.kw;
  g.sh = r.sh;
  g.sw = r.sw;
  g.dh = r.dh;
  g.dw = r.dw;
  g.pt = r.pt;
  g.pl = r.pl;
  return g;
}

inline unsigned blocks_for(size_t n, unsigned per) { return static_cast<unsigned>((n + per - 1) / per); }

}  // namespace

#define GI_BY_STORAGE(call_h, call_f) \
  do {                                \
    if (storage == GI_F16) {          \
      call_h;                         \
    } else {                          \
      call_f;                         \
    }                                 \
  } while (0)

int launch_pack(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int S = slices(r.C), P = plane_pixels(r.H, r.W), HW = r.H * r.W;
  if (storage == GI_F16 && r.C == 3 && HW % 4 == 0 && r.B <= 65535) {
    // P == HW here (no padding pixel), one slice: the planes of the images are back to back
    const int quads = HW / 4;
    launch_pdl(pack3_f16_kernel, dim3(blocks_for(quads, 256), r.B), 256, 0, st, static_cast<const uint2*>(p.in0),
               static_cast<uint4*>(p.out), quads);
    return static_cast<int>(cudaGetLastError());
  }
  const long long planes = static_cast<long long>(S) * r.B;
  if (planes > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  const dim3 grid(blocks_for(P, 256), static_cast<unsigned>(planes < 65535 ? planes : 65535));
  GI_BY_STORAGE((launch_pdl(pack_kernel<__half>, grid, 256, 0, st, static_cast<const __half*>(p.in0), static_cast<__half*>(p.out),
                            r.B, HW, r.C, P, S)),
                (launch_pdl(pack_kernel<float>, grid, 256, 0, st, static_cast<const float*>(p.in0), static_cast<float*>(p.out), r.B,
                            HW, r.C, P, S)));
  return static_cast<int>(cudaGetLastError());
}

int launch_unpack(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int S = slices(r.C), P = plane_pixels(r.H, r.W), HW = r.H * r.W;
  const size_t total = static_cast<size_t>(S) * r.B * HW;
  if (storage == GI_F16 && r.B <= 65535 && static_cast<size_t>(r.C) * 256 <= 48 * 1024) {
    launch_pdl(unpack_f16_kernel, dim3(blocks_for(HW, 128), r.B), 128, static_cast<size_t>(r.C) * 256, st,
               static_cast<const __half*>(p.in0), static_cast<__half*>(p.out), r.B, HW, r.C, P, S);
    return static_cast<int>(cudaGetLastError());
  }
  GI_BY_STORAGE((launch_pdl(unpack_kernel<__half>, blocks_for(total, 256), 256, 0, st, static_cast<const __half*>(p.in0),
                                                                               static_cast<__half*>(p.out), r.B, HW, r.C, P, S)),
                (launch_pdl(unpack_kernel<float>, blocks_for(total, 256), 256, 0, st, static_cast<const float*>(p.in0),
                                                                              static_cast<float*>(p.out), r.B, HW, r.C, P, S)));
  return static_cast<int>(cudaGetLastError());
}

template <typename T>
static void conv_dispatch(const LaunchRec& r, const Ptrs& p, cudaStream_t st) {
  const ConvGeom g = geom(r);
  const int os = r.tc_nt;
  const dim3 grid(blocks_for(g.Pout, 128), (g.Sout + os - 1) / os, r.B);
  const T* in = static_cast<const T*>(p.in0);
  const float4* w = static_cast<const float4*>(p.wts);
  const float* b = static_cast<const float*>(p.bias);
  const T* res = static_cast<const T*>(p.res);
  T* out = static_cast<T*>(p.out);
  switch (os) {
    case 8: launch_pdl(conv_simt_kernel<T, 8>, grid, 128, 0, st, in, w, b, res, out, g, r.ep); break;
    case 4: launch_pdl(conv_simt_kernel<T, 4>, grid, 128, 0, st, in, w, b, res, out, g, r.ep); break;
    case 2: launch_pdl(conv_simt_kernel<T, 2>, grid, 128, 0, st, in, w, b, res, out, g, r.ep); break;
    default: launch_pdl(conv_simt_kernel<T, 1>, grid, 128, 0, st, in, w, b, res, out, g, r.ep); break;
  }
}

int launch_conv_simt(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (r.B > 65535) return static_cast<int>(cudaErrorInvalidConfiguration);
  GI_BY_STORAGE(conv_dispatch<__half>(r, p, st), conv_dispatch<float>(r, p, st));
  return static_cast<int>(cudaGetLastError());
}

int launch_depthwise(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (r.dw_staged) return launch_depthwise_f16(r, p, stream);
  if (r.B > 65535) return static_cast<int>(cudaErrorInvalidConfiguration);
  const ConvGeom g = geom(r);
  const dim3 grid(blocks_for(g.Pout, 128), g.Sout, r.B);
  GI_BY_STORAGE((launch_pdl(depthwise_kernel<__half>, grid, 128, 0, st, static_cast<const __half*>(p.in0), static_cast<const float*>(p.wts),
                                                               static_cast<const float*>(p.bias), static_cast<const __half*>(p.res),
                                                               static_cast<__half*>(p.out), g, r.ep)),
                (launch_pdl(depthwise_kernel<float>, grid, 128, 0, st, static_cast<const float*>(p.in0), static_cast<const float*>(p.wts),
                                                              static_cast<const float*>(p.bias), static_cast<const float*>(p.res),
                                                              static_cast<float*>(p.out), g, r.ep)));
  return static_cast<int>(cudaGetLastError());
}

int launch_eltwise(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t n_px = static_cast<size_t>(slices(r.Co)) * r.B * plane_pixels(r.Ho, r.Wo);
  GI_BY_STORAGE((launch_pdl(eltwise_kernel<__half>, blocks_for(n_px, 256), 256, 0, st, static_cast<const __half*>(p.in0),
                                                                               static_cast<const __half*>(p.in1),
                                                                               static_cast<__half*>(p.out), n_px, r.ep)),
                (launch_pdl(eltwise_kernel<float>, blocks_for(n_px, 256), 256, 0, st, static_cast<const float*>(p.in0),
                                                                              static_cast<const float*>(p.in1),
                                                                              static_cast<float*>(p.out), n_px, r.ep)));
  return static_cast<int>(cudaGetLastError());
}

int launch_concat(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int P = plane_pixels(r.Ho, r.Wo), sout = slices(r.Co);
  const size_t n_px = static_cast<size_t>(r.B) * P;
  if (sout > 65535) return static_cast<int>(cudaErrorInvalidConfiguration);
  const dim3 grid(blocks_for(n_px, 256), sout);
  const int Ca = r.C, Cb = r.Co - r.C;
  GI_BY_STORAGE((launch_pdl(concat_kernel<__half>, grid, 256, 0, st, static_cast<const __half*>(p.in0), static_cast<const __half*>(p.in1),
                            static_cast<__half*>(p.out), n_px, P, r.Ho * r.Wo, Ca, Cb)),
                (launch_pdl(concat_kernel<float>, grid, 256, 0, st, static_cast<const float*>(p.in0), static_cast<const float*>(p.in1),
                            static_cast<float*>(p.out), n_px, P, r.Ho * r.Wo, Ca, Cb)));
  return static_cast<int>(cudaGetLastError());
}

int launch_pool(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int planes = slices(r.C) * r.B;
  const unsigned blocks = blocks_for(static_cast<size_t>(planes) * 8, 256);
  GI_BY_STORAGE((launch_pdl(pool_kernel<__half>, blocks, 256, 0, st, static_cast<const __half*>(p.in0), static_cast<__half*>(p.out), planes,
                                                            r.H * r.W, plane_pixels(r.H, r.W), plane_pixels(1, 1))),
                (launch_pdl(pool_kernel<float>, blocks, 256, 0, st, static_cast<const float*>(p.in0), static_cast<float*>(p.out), planes,
                                                           r.H * r.W, plane_pixels(r.H, r.W), plane_pixels(1, 1))));
  return static_cast<int>(cudaGetLastError());
}

int launch_resize(const LaunchRec& r, const Ptrs& p, int storage, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int ny, dy, nx, dx;
  if (r.align_corners) {
    ny = r.Ho > 1 ? r.H - 1 : 0;
    dy = r.Ho > 1 ? r.Ho - 1 : 1;
    nx = r.Wo > 1 ? r.W - 1 : 0;
    dx = r.Wo > 1 ? r.Wo - 1 : 1;
  } else {
    ny = r.H;
    dy = r.Ho;
    nx = r.W;
    dx = r.Wo;
  }
  const int Pout = plane_pixels(r.Ho, r.Wo), Pin = plane_pixels(r.H, r.W);
  if (r.H > 65535 || r.B > 65535) return static_cast<int>(cudaErrorInvalidConfiguration);
  const dim3 grid(blocks_for(r.Wo, 128), r.H, r.B);
  const bool narrow = (static_cast<long long>(r.Ho) + 1) * ny + static_cast<long long>(r.H + 1) * dy < (1LL << 31) &&
                      static_cast<long long>(r.Wo) * nx < (1LL << 31);
#define GI_RESIZE(T, I)                                                                                                       \
  launch_pdl(resize_kernel<T, I>, grid, 128, 0, st, static_cast<const T*>(p.in0), static_cast<T*>(p.out), r.B, slices(r.C), r.H, r.W, \
             Pin, r.Ho, r.Wo, Pout, ny, dy, nx, dx)
  if (narrow) {
    GI_BY_STORAGE(GI_RESIZE(__half, unsigned), GI_RESIZE(float, unsigned));
  } else {
    GI_BY_STORAGE(GI_RESIZE(__half, unsigned long long), GI_RESIZE(float, unsigned long long));
  }
#undef GI_RESIZE
  return static_cast<int>(cudaGetLastError());
}

}  // namespace gi
