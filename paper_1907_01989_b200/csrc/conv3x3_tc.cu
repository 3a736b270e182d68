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
// produce the tile; 128 epilogue threads read their lane from tensor memory, add the bias,
// apply the fused element-wise tail and store 8 bytes per output slice (256 contiguous bytes per
// warp).  Gather and epilogue are different warps: a gather thread spends most of a tile waiting for its
// loads, an epilogue thread for tensor memory and its stores, and as one thread doing both in turn (the first
// version) neither wait hid the other - 0.104 ms for the MobileNet stem at batch 256 with six CTAs per SM.
// Three operand tiles and two accumulators decouple the three roles.  Waits are bounded like in the pointwise kernel.
//
// NHWC3: the input is the caller's NHWC tensor with 3 fp16 channels (stride 2, no padding above / left, even
// H and W): the layout conversion in front of the convolution (Section 3, "Running Inference") disappears,
// the image is read once, as 6 instead of 8 bytes per pixel.  The three pixels of a window row are 18
// contiguous bytes (4-byte aligned because the first pixel's index is even): five 32-bit loads, whose last
// half - the first channel of the next pixel - is masked off.  The K axis is then simply those 15 words + 1
// zero word: k = 10 * ky + 3 * kx + ci, 32 values (two MMAs instead of three), the weights packed to match.
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
constexpr int kGatherThreads = 128, kEpilogueWarps = 4;
constexpr int kFirstEpilogueWarp = kGatherThreads / 32 + 1;  // warps 0-3 gather, 4 issues the MMAs, 5-8 drain
constexpr int kThreads = kGatherThreads + 32 + 32 * kEpilogueWarps;
constexpr int kABufs = 3, kAccs = 2;
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
  int step_b, step_q;        // gridDim.x * 128 pixels = step_b planes + step_q pixels
  unsigned m_total;          // B * Pout (< 2^31)
  int has_res, act_post;
  unsigned tmem_cols;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long a_full[kABufs], a_empty[kABufs];
  unsigned long long acc_full[kAccs], acc_empty[kAccs];
  unsigned tmem_addr;
  unsigned abort_flag;
};

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

// ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow
template <int ACT, bool TAIL, bool NHWC3>
__global__ void __launch_bounds__(kThreads, 3) conv3x3_tc_kernel(const StemParams p) {
  constexpr int kCoresUsed = NHWC3 ? 4 : kKCores;  // 16-byte K units per row actually multiplied
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  unsigned char* a_tiles = smem + 1024;                 // kABufs x kABytes
  unsigned char* b_tile = a_tiles + kABufs * kABytes;   // 6 * n_pad * 16
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kABufs; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kGatherThreads);
      mbar_init(smem_u32(&hdr->a_empty[i]), 1);
    }
    for (int i = 0; i < kAccs; ++i) {
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), kEpilogueWarps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) tmem_alloc(smem_u32(&hdr->tmem_addr), p.tmem_cols);
  // weights: plain copy into shared memory, then made visible to the tensor core's proxy
  for (int i = threadIdx.x; i < kCoresUsed * p.n_pad; i += kThreads)
    reinterpret_cast<uint4*>(b_tile)[i] = __ldg(reinterpret_cast<const uint4*>(p.wts) + i);
  // K elements 40..47 of both operand buffers are padding: zeroed once, never written again
  if (!NHWC3 && threadIdx.x < kRows) {
    for (int i = 0; i < kABufs; ++i)
      reinterpret_cast<uint4*>(a_tiles + i * kABytes)[5 * kRows + threadIdx.x] = make_uint4(0u, 0u, 0u, 0u);
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
    constexpr int kWords = NHWC3 ? 16 : 20;  // 32-bit words a thread gathers for its pixel
    // ---- loads of one tile: this thread's pixel is q = (oy, ox) of image b
    auto load_tile = [&](unsigned (&w)[kWords], int b, int q, int oy, int ox, bool in_tensor) {
#pragma unroll
      for (int k = 0; k < kWords; ++k) w[k] = 0u;
      if (!(in_tensor && q < real_px)) return;
      if (NHWC3) {
        const int iy0 = 2 * oy, ix0 = 2 * ox;  // even: the window's first pixel starts on a 4-byte boundary
        // 32-bit words: a pixel is 1.5 words, a row p.W * 3 / 2 words (W is even)
        const unsigned* row = reinterpret_cast<const unsigned*>(p.in) +
                              ((static_cast<long long>(b) * p.H + iy0) * p.W + ix0) / 2 * 3;
        const int row_words = p.W / 2 * 3;
        const bool third = ix0 + 2 < p.W;  // the window's last column exists (else it is padding)
#pragma unroll
        for (int ky = 0; ky < 3; ++ky, row += row_words) {
          if (iy0 + ky >= p.H) break;  // padding row below the image
          w[5 * ky] = __ldg(row);
          w[5 * ky + 1] = __ldg(row + 1);
          w[5 * ky + 2] = __ldg(row + 2);
          if (third) {
            w[5 * ky + 3] = __ldg(row + 3);
            w[5 * ky + 4] = __ldg(row + 4);  // its upper half, the first channel of the next pixel, is masked off when stored
          }
        }
        return;
      }
      const int iy0 = oy * p.stride - p.pt, ix0 = ox * p.stride - p.pl;
      const uint2* in8 = reinterpret_cast<const uint2*>(p.in);
      const long long first = static_cast<long long>(b) * p.Pin + static_cast<long long>(iy0) * p.W + ix0;
      if (iy0 >= 0 && ix0 >= 0 && iy0 + 2 * p.dil < p.H && ix0 + 2 * p.dil < p.W) {
        // whole window inside the image (all but the border pixels): no per-tap tests
        const uint2* row = in8 + first;
        const int row_step = p.dil * p.W;
#pragma unroll
        for (int ky = 0; ky < 3; ++ky, row += row_step) {
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) {
            const uint2 v = __ldg(row + kx * p.dil);
            w[2 * (ky * 3 + kx)] = v.x;
            w[2 * (ky * 3 + kx) + 1] = v.y;
          }
        }
      } else {
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
          const int iy = iy0 + ky * p.dil;
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) {
            const int ix = ix0 + kx * p.dil;
            if (iy >= 0 && iy < p.H && ix >= 0 && ix < p.W) {
              const uint2 v = __ldg(in8 + (first + static_cast<long long>(ky * p.dil) * p.W + kx * p.dil));
              w[2 * (ky * 3 + kx)] = v.x;
              w[2 * (ky * 3 + kx) + 1] = v.y;
            }
          }
        }
      }
    };
    // ---- the gathered words into operand buffer `buf` (16-byte K units of this thread's row), then the arrival
    auto store_tile = [&](int buf, unsigned (&w)[kWords]) {
      if (NHWC3) {
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) w[5 * ky + 4] &= 0xffffu;
      }
      uint4* dst = reinterpret_cast<uint4*>(a_tiles + buf * kABytes) + t;
#pragma unroll
      for (int j = 0; j < kWords / 4; ++j) dst[j * kRows] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
      // generic-proxy writes above must be visible to the MMA (async proxy) before the arrival
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&hdr->a_full[buf]));
    };
    // this thread's pixel advances by a fixed number of planes and pixels per tile: no divisions in the loop
    const unsigned gp0 = static_cast<unsigned>(blockIdx.x) * kRows + t;
    int b = static_cast<int>(gp0 / static_cast<unsigned>(p.Pout));
    int q = static_cast<int>(gp0 - static_cast<unsigned>(b) * p.Pout);
    // (row, column) of pixel q, advanced with it: the only divisions are these
    int oy = q / p.Wo, ox = q - oy * p.Wo;
    const int step_oy = p.step_q / p.Wo, step_ox = p.step_q - step_oy * p.Wo;
    const int plane_pad = p.Pout - real_px;  // 1 if the stored plane has a padding pixel
    unsigned gp = gp0;
    const unsigned gp_step = gridDim.x * kRows;
    auto advance = [&]() {
      gp += gp_step;
      b += p.step_b;
      q += p.step_q;
      oy += step_oy;
      ox += step_ox;
      if (ox >= p.Wo) {
        ox -= p.Wo;
        ++oy;
      }
      if (q >= p.Pout) {
        q -= p.Pout;
        ++b;
        oy -= p.Ho;
        ox -= plane_pad;
        if (ox < 0) {
          ox += p.Wo;
          --oy;
        }
      }
    };
    // The loads of tile n + 1 are issued before tile n is stored: a thread's time per tile is then the longer of the
    // load latency and the store / fence / wait, not their sum.  Two register sets, so the loop takes two tiles a turn.
    const int my_tiles = (p.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    unsigned wa[kWords], wb[kWords];
    if (my_tiles > 0) {
      load_tile(wa, b, q, oy, ox, gp < p.m_total);
      advance();
    }
    for (int n = 0; n < my_tiles; n += 2) {
      if (n + 1 < my_tiles) {
        load_tile(wb, b, q, oy, ox, gp < p.m_total);
        advance();
      }
      // the MMAs of the tile that used this operand buffer last have read it
      if (!mbar_wait(smem_u32(&hdr->a_empty[n % kABufs]), ((n / kABufs) & 1) ^ 1, abort_flag, p.timeout_ns, &g_conv_tc_error, 1u)) break;
      store_tile(n % kABufs, wa);
      if (n + 1 >= my_tiles) break;
      if (n + 2 < my_tiles) {
        load_tile(wa, b, q, oy, ox, gp < p.m_total);
        advance();
      }
      if (!mbar_wait(smem_u32(&hdr->a_empty[(n + 1) % kABufs]), (((n + 1) / kABufs) & 1) ^ 1, abort_flag, p.timeout_ns, &g_conv_tc_error, 1u)) break;
      store_tile((n + 1) % kABufs, wb);
    }
  } else if (warp == 4) {
    // ---- MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = n_pad
      const unsigned idesc = (1u << 4) | ((n_cols >> 3) << 17) | ((kRows >> 4) << 24);
      const unsigned b_base = smem_u32(b_tile), b_lbo = n_cols * 16u;
      int n = 0;
      for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++n) {
        const int buf = n % kABufs, acc = n % kAccs;
        if (!mbar_wait(smem_u32(&hdr->a_full[buf]), (n / kABufs) & 1, abort_flag, p.timeout_ns, &g_conv_tc_error, 2u)) break;
        // the accumulator must have been read out by the epilogue of the tile that used it last
        if (!mbar_wait(smem_u32(&hdr->acc_empty[acc]), ((n / kAccs) & 1) ^ 1, abort_flag, p.timeout_ns, &g_conv_tc_error, 2u)) break;
        tc_fence_after();
        const unsigned a_base = smem_u32(a_tiles + buf * kABytes);
#pragma unroll
        for (int ks = 0; ks < kCoresUsed / 2; ++ks) {
          const unsigned long long ad = smem_desc(a_base + ks * 2 * kRows * 16, kRows * 16, 128);
          const unsigned long long bd = smem_desc(b_base + ks * 2 * b_lbo, b_lbo, 128);
          umma_f16(tmem_base + acc * n_cols, ad, bd, idesc, ks > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&hdr->a_empty[buf]));
        umma_commit(smem_u32(&hdr->acc_full[acc]));
      }
    }
  } else {
    // ---- epilogue warps: lane quarter = warp index modulo 4
    const int row = (warp & 3) * 32 + lane;
    const int real_px = p.Ho * p.Wo;
    // ---- epilogue of one tile from accumulator `buf`; gp = this thread's pixel in the whole tensor
    auto epilogue = [&](int buf, unsigned phase, unsigned gp, bool in_tensor, bool real) -> bool {
      if (!mbar_wait_warp(smem_u32(&hdr->acc_full[buf]), phase, abort_flag, p.timeout_ns, &g_conv_tc_error, 4u)) return false;
      tc_fence_after();
      const unsigned t_addr = tmem_base + buf * n_cols + (static_cast<unsigned>((warp & 3) * 32) << 16);
      const size_t slice_stride = static_cast<size_t>(p.m_total) * 4;  // halves between two output slices of a pixel
      auto finish = [&](const unsigned* r, unsigned c0) {
        const size_t off0 = (static_cast<size_t>(c0 / 4) * p.m_total + gp) * 4;  // in halves
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int so = static_cast<int>(c0 / 4) + j;
          if (so >= p.s_out || !in_tensor) continue;
          const size_t off = off0 + static_cast<size_t>(j) * slice_stride;
          uint2 o = make_uint2(0u, 0u);  // the padding pixel of an odd plane stays zero
          if (real) {
            const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias) + so);
            const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1])), make_float2(bv.x, bv.y));
            const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])), make_float2(bv.z, bv.w));
            __half2 h0, h1;
            if (!TAIL) {
              // the conversion clamps at zero itself; clamping at 6 after the rounding equals rounding after the clamp
              const unsigned u0 = pack_f16x2<ACT != GI_ACT_NONE>(v0.x, v0.y), u1 = pack_f16x2<ACT != GI_ACT_NONE>(v1.x, v1.y);
              h0 = *reinterpret_cast<const __half2*>(&u0);
              h1 = *reinterpret_cast<const __half2*>(&u1);
              if (ACT == GI_ACT_RELU6) {
                h0 = __hmin2(h0, __float2half2_rn(6.f));
                h1 = __hmin2(h1, __float2half2_rn(6.f));
              }
            } else {
              float2 r0 = make_float2(0.f, 0.f), r1 = make_float2(0.f, 0.f);
              if (p.has_res) {
                const uint2 q = __ldg(reinterpret_cast<const uint2*>(p.res + off));
                r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
                r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
              }
              h0 = __floats2half2_rn(act1(act1(v0.x, ACT) + r0.x, p.act_post), act1(act1(v0.y, ACT) + r0.y, p.act_post));
              h1 = __floats2half2_rn(act1(act1(v1.x, ACT) + r1.x, p.act_post), act1(act1(v1.y, ACT) + r1.y, p.act_post));
            }
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

    const unsigned gp0 = static_cast<unsigned>(blockIdx.x) * kRows + row;
    int q = static_cast<int>(gp0 % static_cast<unsigned>(p.Pout));
    unsigned gp = gp0;
    const unsigned gp_step = gridDim.x * kRows;
    int n = 0;
    for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++n) {
      const int acc = n % kAccs;
      const bool in_tensor = gp < p.m_total;
      if (!epilogue(acc, (n / kAccs) & 1, gp, in_tensor, in_tensor && q < real_px)) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[acc]));
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

}  // namespace

bool conv3x3_tc_supported(int cin, int cout, int kh, int kw, int sh, int sw, int dh, int dw) {
  return kh == 3 && kw == 3 && cin <= 4 && cout >= 1 && cout <= kMaxN && sh == sw && dh == dw;
}

// The convolution can read the caller's NHWC input itself (no layout conversion in front of it): three fp16
// channels, stride 2 with no padding above / left, even H and W (the window's first pixel then starts on a
// 4-byte boundary and the pixel after the window's last one always exists in the same row).
bool conv3x3_tc_reads_nhwc(int cin, int H, int W, int stride, int dil, int pt, int pl) {
  return cin == 3 && stride == 2 && dil == 1 && pt == 0 && pl == 0 && H % 2 == 0 && W % 2 == 0;
}

// Weights as the B operand: [6 K units][n_pad rows][8 halves], k = unit * 8 + e = tap * 4 + ci; for the
// NHWC-reading variant (r->nhwc_in) [4 K units][n_pad rows][8 halves], k = 10 * ky + 3 * kx + ci.
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
        const int k = r->nhwc_in ? 10 * (tap / 3) + 3 * (tap % 3) + ci : tap * 4 + ci;
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
  // pixel indices are kept in 32 bits inside the kernel, with room for one step past the end
  if (m_total > (1LL << 30)) return static_cast<int>(cudaErrorInvalidConfiguration);
  k.tiles = static_cast<int>(tiles);
  k.m_total = static_cast<unsigned>(m_total);
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  unsigned cols = 32;
  while (cols < static_cast<unsigned>(kAccs * k.n_pad)) cols <<= 1;
  k.tmem_cols = cols;
  k.timeout_ns = 1000000000u;
  static bool attr_set_dev[kMaxDevices] = {};
  bool& attr_set = attr_set_dev[current_device_slot()];
  const int sms = device_sm_count();
  const size_t smem = 1024 + kABufs * kABytes + static_cast<size_t>(kKCores) * k.n_pad * 16;
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    const int bytes = 1024 + kABufs * kABytes + kKCores * kMaxN * 16;
#define GI_C3_ATTR(A, T)                                                                                                               \
  do {                                                                                                                                 \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_tc_kernel<A, T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes); \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_tc_kernel<A, T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);  \
  } while (0)
    GI_C3_ATTR(GI_ACT_NONE, false);
    GI_C3_ATTR(GI_ACT_RELU, false);
    GI_C3_ATTR(GI_ACT_RELU6, false);
    GI_C3_ATTR(GI_ACT_NONE, true);
    GI_C3_ATTR(GI_ACT_RELU, true);
    GI_C3_ATTR(GI_ACT_RELU6, true);
#undef GI_C3_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  // a few CTAs per SM: tensor memory allows 512 / tmem_cols of them, the register file three
  int per_sm = static_cast<int>(512u / cols);
  if (per_sm > 3) per_sm = 3;
  if (per_sm < 1) per_sm = 1;
  long long grid = static_cast<long long>(sms) * per_sm;
  if (grid > tiles) grid = tiles;
  const long long step = grid * kRows;
  k.step_b = static_cast<int>(step / k.Pout);
  k.step_q = static_cast<int>(step % k.Pout);
  const unsigned g = static_cast<unsigned>(grid);
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
  const int act = r.ep.act_pre;
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
#define GI_C3_LAUNCH(A, T)                                                                              \
  do {                                                                                                  \
    if (r.nhwc_in) launch_pdl(conv3x3_tc_kernel<A, T, true>, g, kThreads, smem, cu_stream, k);          \
    else launch_pdl(conv3x3_tc_kernel<A, T, false>, g, kThreads, smem, cu_stream, k);                   \
  } while (0)
  if (tail) {
    if (act == GI_ACT_RELU6) GI_C3_LAUNCH(GI_ACT_RELU6, true);
    else if (act == GI_ACT_RELU) GI_C3_LAUNCH(GI_ACT_RELU, true);
    else GI_C3_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (act == GI_ACT_RELU6) GI_C3_LAUNCH(GI_ACT_RELU6, false);
    else if (act == GI_ACT_RELU) GI_C3_LAUNCH(GI_ACT_RELU, false);
    else GI_C3_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_C3_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

unsigned int conv3x3_tc_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_conv_tc_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
