// Full k x k convolution (k = 1, 2, 3; any stride, dilation and padding) of a tensor with any number of
// channels as an implicit GEMM on the tensor cores (Section 4, "For a 2D Convolution": each output iterates
// over the window and the input slices under it - here window and slices are unrolled into the K axis).
//
//   D[pixel][co] = sum_k A[pixel][k] * B[co][k],   k = (tap * S_in + slice) * 4 + channel-in-slice
//
// The K axis is walked in chunks of 16 pixel-slices (64 values, four tcgen05.mma of K = 16).  A tile of 128
// output pixels is one TMEM lane per pixel.  The 128 gather threads read the chunk's 8-byte pixel-slices of
// their pixel from the channel-sliced input (zero outside the image; consecutive pixels of a row are
// consecutive in memory, so a warp's loads coalesce; where each pixel-slice of the K walk lies relative to the
// window's first pixel is the same for every pixel and comes from a small table in shared memory) and write
// them, two per 16-byte unit, straight into the canonical K-major shared-memory operand layout; the weights
// sit in shared memory for the whole kernel.
// Three operand buffers (handed back by tcgen05.commit) and two accumulators decouple three roles: four gather warps,
// the MMA warp, and four epilogue warps that drain a tile (bias, fused element-wise tail, 8 bytes per output slice).
// (First version: the same 128 threads gathered tile i+1 and then drained tile i; a gather thread waits for its loads
// most of the time, an epilogue thread for tensor memory, and in one thread neither wait hides the other.)  Waits are
// bounded like in the other tensor-core kernels.  The 3 x 3 kernel for a single input slice (the stem of the
// MobileNets) is the special case with one chunk and no hand-back; it keeps its own file.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kRows = 128;             // output pixels per tile
// pixel-slices (4 channels each) per K chunk: 16 (64 values, four MMAs), or 8 for a short K axis, where
// the smaller operand buffers and register footprint let six CTAs instead of four share an SM (measured:
// the fire network 0.296 -> 0.284 ms with 8, while 3x3 32 -> 32 and 64 -> 64 lose 8-18 % with 8)
constexpr int kMaxUnits = 16;
constexpr int kGatherThreads = 128, kEpilogueWarps = 4;
constexpr int kThreads = kGatherThreads + 32 + 32 * kEpilogueWarps;  // warps 0-3 gather, 4 issues the MMAs, 5-8 drain
constexpr int kABufs = 3;
constexpr int kMaxN = 256;
constexpr int kHeaderBytes = 1024;
constexpr int kMaxWeightBytes = 150 * 1024;

__device__ unsigned int g_conv_kxk_error = 0;

struct ConvParams {
  const __half* in;
  const __half* res;
  __half* out;
  const unsigned char* wts;  // [n_groups][n_chunks * UNITS / 2][n_pad][8] fp16
  const float* bias;         // [n_groups * n_pad]
  int B, H, W, Pin, Ho, Wo, Pout;
  int k, s_in, stride, dil, pt, pl;
  int slice_step;            // B * Pin: pixel-slices between two slices of one pixel (the whole input is < 2^31 pixel-slices)
  int n_chunks;              // ceil(k * k * s_in / UNITS)
  int s_out, n_pad;          // output slices; output channels of one CTA group (a multiple of 16)
  int n_groups;              // CTA groups over the output channels (weights of one group fit shared memory)
  int tiles;                 // ceil(B * Pout / 128)
  int step_b, step_q;        // (gridDim.x / n_groups) * 128 pixels = step_b planes + step_q pixels
  unsigned m_total;          // B * Pout (< 2^31)
  int has_res, act_post;
  int a_bufs;                // operand buffers in the ring: 3, or 2 where the third would cost a CTA per SM
  unsigned tmem_cols;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long a_full[kABufs];
  unsigned long long a_empty[kABufs];
  unsigned long long acc_full[2], acc_empty[2];
  unsigned tmem_addr;
  unsigned abort_flag;
};

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

// UNITS: pixel-slices per K chunk; ACT: activation right after the bias; TAIL: a residual add and / or a second
// activation follow
template <int UNITS, int ACT, bool TAIL>
__global__ void __launch_bounds__(kThreads, UNITS == 8 ? 4 : 3) conv_kxk_tc_kernel(const ConvParams p) {
  constexpr int kUnits = UNITS;
  constexpr int kKCores = kUnits / 2;  // 16-byte K units per row and chunk
  constexpr int kABytes = kKCores * kRows * 16;
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  unsigned char* a_tiles = smem + kHeaderBytes;         // kABufs x kABytes
  unsigned char* b_tile = a_tiles + p.a_bufs * kABytes;  // n_chunks * 8 * n_pad * 16
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  // CTA group g computes output channels [g * n_pad, (g + 1) * n_pad) of every pixel tile it walks; the CTAs of
  // one group share the tiles among themselves (one group unless the weights exceed shared memory)
  // (the group's number is recomputed where it is needed rather than kept in a register across the tile loop)
  const bool one_group = p.n_groups == 1;
  const int cta = one_group ? static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x) / p.n_groups;
  const int ctas = one_group ? static_cast<int>(gridDim.x) : static_cast<int>(gridDim.x) / p.n_groups;
  const unsigned char* wts = p.wts + (one_group ? 0 : static_cast<size_t>(blockIdx.x % p.n_groups) * p.n_chunks * kKCores * p.n_pad * 16);

  if (threadIdx.x == 0) {
    for (int i = 0; i < kABufs; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kGatherThreads);
      mbar_init(smem_u32(&hdr->a_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), kEpilogueWarps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) tmem_alloc(smem_u32(&hdr->tmem_addr), p.tmem_cols);
  // weights: plain copy into shared memory, then made visible to the tensor core's proxy
  for (int i = threadIdx.x; i < p.n_chunks * kKCores * p.n_pad; i += kThreads)
    reinterpret_cast<uint4*>(b_tile)[i] = __ldg(reinterpret_cast<const uint4*>(wts) + i);
  // The K walk is the same for every pixel: per pixel-slice of the K axis, its distance (in pixel-slices) from
  // slice 0 of the window's first pixel, and the number of its tap (31 for the padding behind the last
  // pixel-slice: a tap that is never valid).
  int* unit_off = reinterpret_cast<int*>(b_tile + static_cast<size_t>(p.n_chunks) * kKCores * p.n_pad * 16);
  int* unit_tap = unit_off + p.n_chunks * kUnits;
  for (int u = threadIdx.x; u < p.n_chunks * kUnits; u += kThreads) {
    const int tap = u / p.s_in, sl = u - tap * p.s_in;
    const int ky = tap / p.k, kx = tap - ky * p.k;
    const bool exists = tap < p.k * p.k;
    unit_off[u] = exists ? sl * p.slice_step + ky * p.dil * p.W + kx * p.dil : 0;
    unit_tap[u] = exists ? tap : 31;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // everything above touched only weights and on-chip state; the activations come after the wait
  pdl_launch_dependents();
  pdl_wait();
  const unsigned tmem_base = hdr->tmem_addr;
  const unsigned n_cols = static_cast<unsigned>(p.n_pad);

  if (warp < 4) {
    const int t = threadIdx.x;  // row of the tile = TMEM lane
    const int real_px = p.Ho * p.Wo;
    const uint2* in8 = reinterpret_cast<const uint2*>(p.in);
    unsigned it = 0;  // K chunks gathered so far by this CTA
    // ---- gather of all K chunks of one tile; this thread's pixel is q of image b.  Returns false on a timeout.
    auto gather_tile = [&](int b, int q, bool in_tensor) -> bool {
      const bool live = in_tensor && q < real_px;
      int iy0 = 0, ix0 = 0;
      if (live) {
        const int oy = q / p.Wo, ox = q - oy * p.Wo;
        iy0 = oy * p.stride - p.pt;
        ix0 = ox * p.stride - p.pl;
      }
      // slice 0 of the window's first pixel (outside the tensor for border pixels: only dereferenced where valid)
      const uint2* base = in8 + (static_cast<long long>(b) * p.Pin + static_cast<long long>(iy0) * p.W + ix0);
      // bit `tap` says whether that tap of this pixel's window lies inside the image: one test per tile and
      // tap instead of one per gathered pixel-slice, and the same instructions for border and interior pixels
      unsigned tap_ok = 0;
      if (live) {
        for (int ky = 0; ky < p.k; ++ky)
          for (int kx = 0; kx < p.k; ++kx)
            if (static_cast<unsigned>(iy0 + ky * p.dil) < static_cast<unsigned>(p.H) &&
                static_cast<unsigned>(ix0 + kx * p.dil) < static_cast<unsigned>(p.W))
              tap_ok |= 1u << (ky * p.k + kx);
      }
      for (int c = 0; c < p.n_chunks; ++c, ++it) {
        // (two constant divisors instead of a division by a run-time value in every chunk)
        const int buf = static_cast<int>(p.a_bufs == 3 ? it % 3u : it & 1u);
        const unsigned e_phase = ((p.a_bufs == 3 ? it / 3u : it >> 1) & 1u) ^ 1u;
        // The loads do not touch the operand buffer: with 16-unit chunks they are issued before the wait for it
        // (3x3 64 -> 64 on 56x56 0.260 -> 0.246 ms, 128 -> 128 on 28x28 0.399 -> 0.358 ms); with 8-unit chunks
        // and their 64-register budget that order spills and measured 2-5 % slower, so there the wait comes first.
        constexpr bool kLoadsFirst = kUnits == 16;
        if (!kLoadsFirst &&
            !mbar_wait_warp(smem_u32(&hdr->a_empty[buf]), e_phase, abort_flag, p.timeout_ns, &g_conv_kxk_error, 1u))
          return false;
        uint2 unit[kUnits];
        const int4* off4 = reinterpret_cast<const int4*>(unit_off + c * kUnits);
        const int4* tap4 = reinterpret_cast<const int4*>(unit_tap + c * kUnits);
#pragma unroll
        for (int j4 = 0; j4 < kUnits / 4; ++j4) {
          const int4 o = off4[j4], tp = tap4[j4];
          const int of[4] = {o.x, o.y, o.z, o.w}, tn[4] = {tp.x, tp.y, tp.z, tp.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) unit[4 * j4 + e] = ((tap_ok >> tn[e]) & 1u) ? __ldg(base + of[e]) : make_uint2(0u, 0u);
        }
        if (kLoadsFirst &&
            !mbar_wait_warp(smem_u32(&hdr->a_empty[buf]), e_phase, abort_flag, p.timeout_ns, &g_conv_kxk_error, 1u))
          return false;
        uint4* dst = reinterpret_cast<uint4*>(a_tiles + buf * kABytes) + t;
#pragma unroll
        for (int j = 0; j < kKCores; ++j)
          dst[j * kRows] = make_uint4(unit[2 * j].x, unit[2 * j].y, unit[2 * j + 1].x, unit[2 * j + 1].y);
        // generic-proxy writes above must be visible to the MMA (async proxy) before the arrival
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&hdr->a_full[buf]));
      }
      return true;
    };
    // this thread's pixel advances by a fixed number of planes and pixels per tile: no divisions by the plane size in the loop
    const unsigned gp0 = static_cast<unsigned>(cta) * kRows + t;
    int b = static_cast<int>(gp0 / static_cast<unsigned>(p.Pout));
    int q = static_cast<int>(gp0 - static_cast<unsigned>(b) * p.Pout);
    unsigned gp = gp0;
    const unsigned gp_step = static_cast<unsigned>(ctas) * kRows;
    for (int tile = cta; tile < p.tiles; tile += ctas) {
      if (!gather_tile(b, q, gp < p.m_total)) break;
      gp += gp_step;
      b += p.step_b;
      q += p.step_q;
      if (q >= p.Pout) {
        q -= p.Pout;
        ++b;
      }
    }
  } else if (warp == 4) {
    // ---- MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = n_pad
      const unsigned idesc = (1u << 4) | ((n_cols >> 3) << 17) | ((kRows >> 4) << 24);
      const unsigned b_base = smem_u32(b_tile), b_lbo = n_cols * 16u;
      unsigned it = 0;
      int n = 0;
      bool ok = true;
      for (int tile = cta; tile < p.tiles && ok; tile += ctas, ++n) {
        const unsigned d_tmem = tmem_base + static_cast<unsigned>(n & 1) * n_cols;
        // the accumulator must have been read out by the epilogue of the tile that used it last
        if (!mbar_wait(smem_u32(&hdr->acc_empty[n & 1]), ((n >> 1) & 1) ^ 1, abort_flag, p.timeout_ns, &g_conv_kxk_error, 2u)) break;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const int buf = static_cast<int>(p.a_bufs == 3 ? it % 3u : it & 1u);
          if (!mbar_wait(smem_u32(&hdr->a_full[buf]), (p.a_bufs == 3 ? it / 3u : it >> 1) & 1u, abort_flag, p.timeout_ns, &g_conv_kxk_error, 2u)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const unsigned a_base = smem_u32(a_tiles + buf * kABytes);
          const unsigned bc_base = b_base + static_cast<unsigned>(c) * kKCores * b_lbo;
#pragma unroll
          for (int ks = 0; ks < kKCores / 2; ++ks) {
            const unsigned long long ad = smem_desc(a_base + ks * 2 * kRows * 16, kRows * 16, 128);
            const unsigned long long bd = smem_desc(bc_base + ks * 2 * b_lbo, b_lbo, 128);
            umma_f16(d_tmem, ad, bd, idesc, (c > 0 || ks > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&hdr->a_empty[buf]));  // the buffer is free once these MMAs have read it
        }
        // the accumulator's barrier, the one the epilogue waits on, is committed last
        if (ok) umma_commit(smem_u32(&hdr->acc_full[n & 1]));
      }
    }
  } else {
    // ---- epilogue warps: lane quarter = warp index modulo 4
    const int real_px = p.Ho * p.Wo;
    // ---- epilogue of one tile from accumulator `buf`; gp = this thread's pixel in the whole tensor
    auto epilogue = [&](int buf, unsigned phase, unsigned gp, bool in_tensor, bool real) -> bool {
      if (!mbar_wait_warp(smem_u32(&hdr->acc_full[buf]), phase, abort_flag, p.timeout_ns, &g_conv_kxk_error, 4u)) return false;
      tc_fence_after();
      const unsigned t_addr = tmem_base + buf * n_cols + (static_cast<unsigned>((warp & 3) * 32) << 16);
      const int grp = p.n_groups == 1 ? 0 : static_cast<int>(blockIdx.x) % p.n_groups, so0 = grp * (p.n_pad / 4);
      const float* bias = p.bias + grp * p.n_pad;
      auto finish = [&](const unsigned* r, unsigned c0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int sg = static_cast<int>(c0 / 4) + j, so = so0 + sg;  // slice within the group, within the tensor
          if (so >= p.s_out || !in_tensor) continue;
          const size_t off = (static_cast<size_t>(so) * p.m_total + gp) * 4;  // in halves
          uint2 o = make_uint2(0u, 0u);  // the padding pixel of an odd plane stays zero
          if (real) {
            const float4 bv = __ldg(reinterpret_cast<const float4*>(bias) + sg);
            float v[4] = {__uint_as_float(r[4 * j]) + bv.x, __uint_as_float(r[4 * j + 1]) + bv.y,
                          __uint_as_float(r[4 * j + 2]) + bv.z, __uint_as_float(r[4 * j + 3]) + bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = act1(v[e], ACT);
            if (TAIL) {
              if (p.has_res) {
                const uint2 qv = __ldg(reinterpret_cast<const uint2*>(p.res + off));
                const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&qv.x));
                const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&qv.y));
                v[0] += r0.x;
                v[1] += r0.y;
                v[2] += r1.x;
                v[3] += r1.y;
              }
#pragma unroll
              for (int e = 0; e < 4; ++e) v[e] = act1(v[e], p.act_post);
            }
            const __half2 h0 = __floats2half2_rn(v[0], v[1]), h1 = __floats2half2_rn(v[2], v[3]);
            o.x = *reinterpret_cast<const unsigned*>(&h0);
            o.y = *reinterpret_cast<const unsigned*>(&h1);
          }
          *reinterpret_cast<uint2*>(p.out + off) = o;
        }
      };
      // two 16-column reads in flight: the next one is issued before the current one is processed
      unsigned ra[16], rb[16];
      tmem_ld16(t_addr, ra);
      for (unsigned c0 = 0; c0 < n_cols; c0 += 32) {
        tmem_ld_wait16(ra);
        if (c0 + 16 < n_cols) tmem_ld16(t_addr + c0 + 16, rb);
        finish(ra, c0);
        if (c0 + 16 < n_cols) {
          tmem_ld_wait16(rb);
          if (c0 + 32 < n_cols) tmem_ld16(t_addr + c0 + 32, ra);
          finish(rb, c0 + 16);
        }
      }
      tc_fence_before();
      return true;
    };

    const unsigned gp0 = static_cast<unsigned>(cta) * kRows + static_cast<unsigned>((warp & 3) * 32 + lane);
    int q = static_cast<int>(gp0 % static_cast<unsigned>(p.Pout));
    unsigned gp = gp0;
    const unsigned gp_step = static_cast<unsigned>(ctas) * kRows;
    int n = 0;
    for (int tile = cta; tile < p.tiles; tile += ctas, ++n) {
      const bool in_tensor = gp < p.m_total;
      if (!epilogue(n & 1, (n >> 1) & 1, gp, in_tensor, in_tensor && q < real_px)) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[n & 1]));
      gp += gp_step;
      q += p.step_q;
      if (q >= p.Pout) q -= p.Pout;
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

int units_of(int k, int cin) { return k * k * slices(cin) <= 32 ? 8 : 16; }
int chunks_of(int k, int cin) { return (k * k * slices(cin) + units_of(k, cin) - 1) / units_of(k, cin); }
// 16-byte K units of the whole weight operand
int cores_of(int k, int cin) { return chunks_of(k, cin) * units_of(k, cin) / 2; }

// Output channels per CTA group: all of them (rounded up to 16) if their weights fit shared memory, else
// the largest multiple of 16 whose weights do; 0 if not even 16 output channels fit.
int group_channels(int k, int cin, int cout) {
  const int n_pad = (cout + 15) / 16 * 16;
  const long long per16 = static_cast<long long>(cores_of(k, cin)) * 16 * 16;  // weight bytes of 16 output channels
  long long fit = kMaxWeightBytes / per16 * 16;
  if (fit > kMaxN) fit = kMaxN;  // one MMA's N, and two accumulators in tensor memory
  if (fit < 16) return 0;
  if (fit >= n_pad) return n_pad;
  const int groups = static_cast<int>((n_pad + fit - 1) / fit);
  return ((n_pad / 16 + groups - 1) / groups) * 16;  // even split, rounded up to 16
}

}  // namespace

bool conv_kxk_tc_supported(int cin, int cout, int kh, int kw, int sh, int sw, int dh, int dw) {
  if (kh != kw || kh < 1 || kh > 3 || sh != sw || dh != dw || cout < 1 || cin < 1) return false;
  const int ng = group_channels(kh, cin, cout);
  if (ng == 0) return false;
  // a group re-gathers the input: beyond eight groups the CUDA-core kernel's single pass is no worse
  return ((cout + 15) / 16 * 16 + ng - 1) / ng <= 8;
}

// Weights as the B operand, per CTA group: [group][16-byte K units of all chunks][n_pad rows][8 halves],
// k = unit * 8 + e = ((tap * S_in + slice) * 4 + channel-in-slice); entries of channels and units that do not
// exist are zero.
void conv_kxk_tc_pack(const float* w, const float* bias, int cin, int cout, int k, std::vector<uint8_t>* blob, LaunchRec* r) {
  const int ng = group_channels(k, cin, cout), s_in = slices(cin), taps = k * k;
  const int groups = ((cout + 15) / 16 * 16 + ng - 1) / ng;
  const int cores = cores_of(k, cin);
  const size_t wbytes = static_cast<size_t>(groups) * cores * ng * 16;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(groups) * ng * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) {
    bp[co] = bias[co];  // group g's biases start at g * ng: the same index
    const int g = co / ng, cg = co - g * ng;
    for (int tap = 0; tap < taps; ++tap)
      for (int ci = 0; ci < cin; ++ci) {
        const int kk = (tap * s_in + ci / 4) * 4 + ci % 4;
        wp[((static_cast<size_t>(g) * cores + kk / 8) * ng + cg) * 8 + kk % 8] =
            f32_to_f16_rne(w[(static_cast<size_t>(co) * taps + tap) * cin + ci]);
      }
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = ng;
  r->tc_kc = groups;
}

int launch_conv_kxk_tc(const LaunchRec& r, const Ptrs& p, void* stream) {
  ConvParams k;
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
  k.k = r.kh;
  k.s_in = slices(r.C);
  k.stride = r.sh;
  k.dil = r.dh;
  k.pt = r.pt;
  k.pl = r.pl;
  k.n_chunks = chunks_of(r.kh, r.C);
  // distances inside the input are kept in 32 bits
  if (static_cast<long long>(k.s_in) * r.B * k.Pin >= (1LL << 31)) return static_cast<int>(cudaErrorInvalidConfiguration);
  k.slice_step = r.B * k.Pin;
  k.s_out = slices(r.Co);
  k.n_pad = r.tc_nt;
  k.n_groups = r.tc_kc;
  const long long m_total = static_cast<long long>(r.B) * k.Pout;
  const long long tiles = (m_total + kRows - 1) / kRows;
  // pixel indices are kept in 32 bits inside the kernel, with room for one step past the end
  if (m_total > (1LL << 30)) return static_cast<int>(cudaErrorInvalidConfiguration);
  k.tiles = static_cast<int>(tiles);
  k.m_total = static_cast<unsigned>(m_total);
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  unsigned cols = 32;
  while (cols < static_cast<unsigned>(2 * k.n_pad)) cols <<= 1;
  k.tmem_cols = cols;
  k.timeout_ns = 1000000000u;
  static bool attr_set_dev[kMaxDevices] = {};
  bool& attr_set = attr_set_dev[current_device_slot()];
  const int sms = device_sm_count();
  const int units = units_of(r.kh, r.C);
  auto smem_with = [&](int bufs) {
    return kHeaderBytes + bufs * static_cast<size_t>(units / 2) * kRows * 16 + static_cast<size_t>(cores_of(r.kh, r.C)) * k.n_pad * 16 +
           static_cast<size_t>(k.n_chunks) * units * 8;  // + the two per-unit tables
  };
  auto ctas_with = [&](int bufs) {
    int n = static_cast<int>((227 * 1024) / (smem_with(bufs) + 1024));
    const int cap = units == 8 ? 4 : 3;  // the register file
    return n > cap ? cap : n;
  };
  // a third operand buffer lets the gather run further ahead, unless it costs a resident CTA (3 x 3 64 -> 64 on 56 x 56:
  // 0.227 ms with two buffers and two CTAs per SM, 0.256 ms with three and one)
  k.a_bufs = ctas_with(kABufs) >= ctas_with(2) ? kABufs : 2;
  const size_t smem = smem_with(k.a_bufs);
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    // tables: at most 1/16 of the weights (n_pad >= 16)
    const int bytes = kHeaderBytes + kABufs * (kMaxUnits / 2) * kRows * 16 + kMaxWeightBytes + kMaxWeightBytes / 16;
#define GI_CK_ATTR(A, T)                                                                                                             \
  do {                                                                                                                               \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv_kxk_tc_kernel<8, A, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);  \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv_kxk_tc_kernel<16, A, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes); \
  } while (0)
    GI_CK_ATTR(GI_ACT_NONE, false);
    GI_CK_ATTR(GI_ACT_RELU, false);
    GI_CK_ATTR(GI_ACT_RELU6, false);
    GI_CK_ATTR(GI_ACT_NONE, true);
    GI_CK_ATTR(GI_ACT_RELU, true);
    GI_CK_ATTR(GI_ACT_RELU6, true);
#undef GI_CK_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  // a few CTAs per SM: tensor memory allows 512 / tmem_cols of them, shared memory 227 KB / smem, the register file
  // three (four with 8-unit chunks)
  int per_sm = static_cast<int>(512u / cols);
  const int by_smem = static_cast<int>((227 * 1024) / (smem + 1024));
  if (per_sm > by_smem) per_sm = by_smem;
  if (per_sm > (units == 8 ? 4 : 3)) per_sm = units == 8 ? 4 : 3;
  if (per_sm < 1) per_sm = 1;
  // the grid is a whole number of CTAs per group
  long long per_group = static_cast<long long>(sms) * per_sm / k.n_groups;
  if (per_group > tiles) per_group = tiles;
  if (per_group < 1) per_group = 1;
  const long long grid = per_group * k.n_groups;
  const long long step = per_group * kRows;
  k.step_b = static_cast<int>(step / k.Pout);
  k.step_q = static_cast<int>(step % k.Pout);
  const unsigned g = static_cast<unsigned>(grid);
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
  const int act = r.ep.act_pre;
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
#define GI_CK_LAUNCH(A, T)                                                                      \
  do {                                                                                          \
    if (units == 8) launch_pdl(conv_kxk_tc_kernel<8, A, T>, g, kThreads, smem, cu_stream, k);   \
    else launch_pdl(conv_kxk_tc_kernel<16, A, T>, g, kThreads, smem, cu_stream, k);             \
  } while (0)
  if (tail) {
    if (act == GI_ACT_RELU6) GI_CK_LAUNCH(GI_ACT_RELU6, true);
    else if (act == GI_ACT_RELU) GI_CK_LAUNCH(GI_ACT_RELU, true);
    else GI_CK_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (act == GI_ACT_RELU6) GI_CK_LAUNCH(GI_ACT_RELU6, false);
    else if (act == GI_ACT_RELU) GI_CK_LAUNCH(GI_ACT_RELU, false);
    else GI_CK_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_CK_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

unsigned int conv_kxk_tc_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_conv_kxk_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
