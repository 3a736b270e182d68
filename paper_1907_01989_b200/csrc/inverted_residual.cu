// One inverted-residual block - expansion 1x1 -> activation -> depthwise 3x3 -> activation ->
// projection 1x1 (-> + residual) - as ONE kernel (fp16 storage).  The paper's cure for an engine
// bound by memory is fewer, fatter programs (Section 3.2, "Shader Program Optimization"); on the small
// planes of a MobileNet (14x14, 7x7) three launches per block spend more time filling and draining
// than computing, and the 6x expanded tensor makes four trips through L2 / HBM that exist only
// because the block is three kernels.  Here it never leaves the SM.
//
// Work unit = `n_img` whole images (one 14x14 image, two 7x7 images), i.e. at most 256 input pixels =
// one or two 128-row MMA tiles; row r of the tiles is pixel r of the unit.  One CTA per SM walks units.
//   * The block input X is copied once per unit into shared memory in the canonical K-major operand
//     layout (8 channels = 16 bytes per row and K group; 8-byte cp.async straight from the
//     channel-sliced tensor, two slices interleaved).
//   * The hidden channels are processed in chunks of 64:
//       expansion     D1[rows x 64]   = X * We[chunk]^T                  tcgen05.mma, accumulator in TMEM (two buffers)
//       drain         bias, activation, fp16 -> a zero-bordered tile in shared memory, one plane per (slice, image)
//       depthwise     3x3 stencil from that tile (a thread walks down one column of one 4-channel slice, every
//                     input row feeding three running accumulators), bias, activation, fp16 -> the A operand of
//                     the projection, written into shared memory in the canonical layout
//       projection    D2[rows x Cout] += A2 * Wp[:, chunk]^T             tcgen05.mma, accumulating over the chunks
//     The chunk's weights (We rows, Wp columns, depthwise taps, both biases: one contiguous block, packed at
//     compile time) stream from L2 through a ring of stages filled by bulk copies.
//   * After the last chunk D2 is drained: bias, activation, residual, activation, fp16, 8-byte stores.
// Results are those of the three operators run one after the other: both hidden tensors are rounded to fp16
// exactly as the stored tensors would have been.
//
// Warps: 0 = weight copies, 1 = MMA issuer and TMEM owner, 2..17 = compute (drain, stencil, epilogue; they also
// issue the cp.async copies of the next unit's X as soon as the last expansion of the current unit is done).
// The MMA thread runs one chunk ahead: expansion(c+1) is in flight while the compute warps work on chunk c.
// Every wait is bounded; a wait that runs out raises the abort flag, after which all roles skip their work but
// still meet at every barrier, so the CTA leaves in order.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstring>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kNh = 64;  // hidden channels per chunk
constexpr int kComputeWarps = 16;
constexpr int kComputeThreads = 32 * kComputeWarps;
constexpr int kThreads = 64 + kComputeThreads;
constexpr int kTeamWarps = kComputeWarps / 2, kTeamThreads = 32 * kTeamWarps;  // two teams take alternate chunks
constexpr int kMaxStages = 3;
constexpr int kHeader = 1024;
constexpr int kSmemMax = 227 * 1024;
constexpr int kDwBytes = (9 * kNh + kNh + kNh) * 4;  // depthwise taps, depthwise bias, expansion bias of a chunk

__device__ unsigned int g_ir_error = 0;
#ifndef GI_TRACE_UNIT
#define GI_TRACE_UNIT 0
#endif
#ifdef GI_TRACE
__device__ unsigned long long g_ir_trace[256 * 64];
#define IR_EV(idx)                                           \
  do {                                                       \
    if (blockIdx.x < 256 && (idx) < 64) {                    \
      unsigned long long t_;                                 \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
      g_ir_trace[blockIdx.x * 64 + (idx)] = t_;              \
    }                                                        \
  } while (0)
#else
#define IR_EV(idx) ((void)0)
#endif
enum : unsigned { kErrCopy = 1u, kErrMma = 2u, kErrCompute = 4u, kErrDrain = 8u };

struct IrParams {
  const __half* in;
  const __half* res;
  __half* out;
  const unsigned char* wts;  // n_chunks blocks of stage_bytes
  const float* bias2;        // cout_pad floats
  int B, H, W, Pin, Ho, Wo, Pout;
  int stride, pt, pl;
  int s_in;                  // input slices (input channels are a multiple of 16)
  int n_chunks;
  int cout_pad, s_out;
  int n_split, n_each;       // the projection's N per MMA: cout_pad = n_split * n_each, n_each <= 256
  int n_img, r_in, r_out;    // images per unit, pixels per image on the input / output side
  int mt_in, mt_out;         // 128-row tiles on the input / output side
  int units;
  int Wp, plane_words;       // padded hidden tile: row pitch and plane pitch in 8-byte words
  int n_bands, band_rows;
  int stages;
  unsigned stage_bytes, we_bytes, wp_bytes;
  unsigned x_bytes, a2_bytes, h_bytes;  // h_bytes: ONE hidden tile (there are two)
  unsigned x_pitch, a2_pitch;           // byte distance between the K groups (8 channels) of X / A2: rows x 16
  unsigned d2_col0;
  int act1, act2, act3, has_res, act4;  // after expansion, after depthwise, after projection, residual, after the sum
  unsigned timeout_ns;
};

struct Header {
  unsigned long long w_full[kMaxStages], w_empty[kMaxStages];
  unsigned long long d1_full[2], d1_empty[2];
  unsigned long long a2_full[2], a2_empty[2], d2_full, d2_empty, x_full;
  unsigned tmem_addr, abort_flag;
};
static_assert(sizeof(Header) <= kHeader, "header too large");

__device__ __forceinline__ float act1f(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}
// two floats -> fp16 pair with the activation applied: clamping the rounded value equals rounding the clamped
// one because 0 and 6 are fp16 values
__device__ __forceinline__ unsigned pack_act(float x, float y, int kind) {
  if (kind == GI_ACT_NONE) return pack_f16x2<false>(x, y);
  const unsigned d = pack_f16x2<true>(x, y);  // the conversion clamps at zero itself
  if (kind != GI_ACT_RELU6) return d;
  const __half2 h = __hmin2(*reinterpret_cast<const __half2*>(&d), __float2half2_rn(6.f));
  return *reinterpret_cast<const unsigned*>(&h);
}
__device__ __forceinline__ uint2 lds64(unsigned addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds128f(unsigned addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts64(unsigned addr, unsigned x, unsigned y) {
  asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void cp_async8(unsigned dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// barrier of the compute warps only (id 1); the copy and MMA warps never join it
__device__ __forceinline__ void bar_compute() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }
// barrier of one team of compute warps (ids 2 and 3)
__device__ __forceinline__ void bar_team(int team) { asm volatile("bar.sync %0, %1;" ::"r"(2 + team), "n"(kTeamThreads) : "memory"); }

struct Tap {
  float2 lo, hi;
};
__device__ __forceinline__ Tap tap_of(uint2 v) {
  Tap t;
  t.lo = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
  t.hi = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
  return t;
}

// 16 accumulator columns (four 4-channel slices of one pixel) -> bias, activation, fp16 -> the pixel's place in the
// four slices' planes of the hidden tile (`pitch` bytes apart)
__device__ __forceinline__ void store_hidden(const unsigned (&r)[16], const float4 (&b)[4], unsigned at, unsigned pitch, bool valid, int act) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1])), make_float2(b[i].x, b[i].y));
    const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), make_float2(b[i].z, b[i].w));
    if (valid) sts64(at + static_cast<unsigned>(i) * pitch, pack_act(v0.x, v0.y, act), pack_act(v1.x, v1.y, act));
  }
}

// Stride-1 stencil of one thread over a whole plane column of compile-time height, as straight-line code: `h` is
// the shared-memory address of the thread's column in padded row 0 of its plane (row pitch WP pixel-slices), `a2` the
// address of its channels in A2 for output row 0.  Padded row iy is tap row 0 of output row iy, row 1 of output row
// iy - 1 and row 2 of iy - 2, so three accumulators rotate; with the trip count and the pitches known at compile time
// the rotation costs no register moves and every address is an immediate offset.
template <int ROWS, int WP>
__device__ __forceinline__ void stencil_column(unsigned h, unsigned a2, const float2 (&wlo)[9], const float2 (&whi)[9], const Tap& bias,
                                               int act) {
  constexpr int WO = WP - 2;
  Tap acc[3] = {bias, bias, bias};
#pragma unroll
  for (int iy = 0; iy < ROWS + 2; ++iy) {
    const unsigned at = h + static_cast<unsigned>(iy * WP) * 8u;
    const Tap t0 = tap_of(lds64(at)), t1 = tap_of(lds64(at + 8u)), t2 = tap_of(lds64(at + 16u));
    Tap& done = acc[(iy + 1) % 3];  // output row iy - 2
    Tap& mid = acc[(iy + 2) % 3];   // output row iy - 1
    Tap& fresh = acc[iy % 3];       // output row iy
    if (iy >= 2) {
      done.lo = __ffma2_rn(t0.lo, wlo[6], done.lo);
      done.hi = __ffma2_rn(t0.hi, whi[6], done.hi);
      done.lo = __ffma2_rn(t1.lo, wlo[7], done.lo);
      done.hi = __ffma2_rn(t1.hi, whi[7], done.hi);
      done.lo = __ffma2_rn(t2.lo, wlo[8], done.lo);
      done.hi = __ffma2_rn(t2.hi, whi[8], done.hi);
      sts64(a2 + static_cast<unsigned>((iy - 2) * WO) * 16u, pack_act(done.lo.x, done.lo.y, act), pack_act(done.hi.x, done.hi.y, act));
    }
    if (iy >= 1 && iy <= ROWS) {
      mid.lo = __ffma2_rn(t0.lo, wlo[3], mid.lo);
      mid.hi = __ffma2_rn(t0.hi, whi[3], mid.hi);
      mid.lo = __ffma2_rn(t1.lo, wlo[4], mid.lo);
      mid.hi = __ffma2_rn(t1.hi, whi[4], mid.hi);
      mid.lo = __ffma2_rn(t2.lo, wlo[5], mid.lo);
      mid.hi = __ffma2_rn(t2.hi, whi[5], mid.hi);
    }
    if (iy < ROWS) {
      fresh.lo = __ffma2_rn(t0.lo, wlo[0], bias.lo);
      fresh.hi = __ffma2_rn(t0.hi, whi[0], bias.hi);
      fresh.lo = __ffma2_rn(t1.lo, wlo[1], fresh.lo);
      fresh.hi = __ffma2_rn(t1.hi, whi[1], fresh.hi);
      fresh.lo = __ffma2_rn(t2.lo, wlo[2], fresh.lo);
      fresh.hi = __ffma2_rn(t2.hi, whi[2], fresh.hi);
    }
  }
}

// STRIDE: of the depthwise convolution; PLANE: 14 or 7 = the hidden planes are 14x14 / 7x7 and a thread walks a whole
// column (straight-line stencil); 0 = any supported plane (loops)
template <int STRIDE, int PLANE>
__global__ void __launch_bounds__(kThreads, 1) inverted_residual_kernel(const IrParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned x0 = smem_u32(smem + kHeader);
  const unsigned a20 = x0 + p.x_bytes;
  const unsigned h0 = a20 + 2u * p.a2_bytes;      // two A2 buffers, then two hidden tiles of h_bytes each: one per team
  const unsigned st0 = h0 + 2u * p.h_bytes;
  const unsigned d1_cols = static_cast<unsigned>(p.mt_in) * kNh;  // one D1 buffer

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->w_full[i]), 1);
      mbar_init(smem_u32(&hdr->w_empty[i]), 1 + kTeamWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->d1_full[i]), 1);
      mbar_init(smem_u32(&hdr->d1_empty[i]), kTeamWarps);
      mbar_init(smem_u32(&hdr->a2_full[i]), 1);
      mbar_init(smem_u32(&hdr->a2_empty[i]), 1);
    }
    mbar_init(smem_u32(&hdr->d2_full), 1);
    mbar_init(smem_u32(&hdr->d2_empty), kTeamWarps);
    mbar_init(smem_u32(&hdr->x_full), 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_proxy();
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------ weight copies (weights never change: no wait
    // for the previous kernel)
    if (lane == 0) {
      unsigned g = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
        for (int c = 0; c < p.n_chunks; ++c, ++g) {
          const unsigned stage = g % p.stages, phase = (g / p.stages) & 1u;
          if (!mbar_wait_parked(smem_u32(&hdr->w_empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrCopy)) {
            ok = false;
            break;
          }
          const unsigned full = smem_u32(&hdr->w_full[stage]);
          mbar_expect_tx(full, p.stage_bytes);
          bulk_load(st0 + stage * p.stage_bytes, p.wts + static_cast<size_t>(c) * p.stage_bytes, p.stage_bytes, full);
        }
      }
      if (!ok) {
        // copies already issued still land in shared memory: give them a bounded grace before leaving
        const unsigned first = g > static_cast<unsigned>(p.stages) ? g - p.stages : 0u;
        for (unsigned j = first; j < g; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->w_full[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_ir_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const unsigned idesc1 = (1u << 4) | ((static_cast<unsigned>(kNh) >> 3) << 17) | ((128u >> 4) << 24);
      const unsigned idesc2 = (1u << 4) | ((static_cast<unsigned>(p.n_each) >> 3) << 17) | ((128u >> 4) << 24);
      const unsigned we_lbo = kNh * 16u, wp_lbo = static_cast<unsigned>(p.cout_pad) * 16u;
      const int k_steps1 = p.s_in / 4;  // 16 input channels per MMA
      unsigned g = 0, ul = 0;
      unsigned n_exp[2] = {0u, 0u}, n_prj[2] = {0u, 0u};  // expansions issued into D1[k], projections issued from A2[k]
      bool ok = true;
      // expansion of chunk c of the current unit (its weights are chunk number gc of the copy warp's sequence) into D1[c & 1]
      auto expand = [&](unsigned gc, int c) -> bool {
        const unsigned stage = gc % p.stages, buf = static_cast<unsigned>(c) & 1u;
        if (!mbar_wait_parked(smem_u32(&hdr->w_full[stage]), (gc / p.stages) & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrMma) ||
            !mbar_wait_parked(smem_u32(&hdr->d1_empty[buf]), (n_exp[buf] & 1u) ^ 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrMma))
          return false;
        ++n_exp[buf];
        tc_fence_after();
        const unsigned we = st0 + stage * p.stage_bytes;
        for (int t = 0; t < p.mt_in; ++t) {
          const unsigned d = tmem_base + buf * d1_cols + static_cast<unsigned>(t) * kNh;
          unsigned long long ad = smem_desc(x0 + static_cast<unsigned>(t) * 2048u, p.x_pitch, 128);
          unsigned long long bd = smem_desc(we, we_lbo, 128);
          const unsigned long long ad_step = static_cast<unsigned long long>((2u * p.x_pitch) >> 4);
          const unsigned long long bd_step = static_cast<unsigned long long>((2u * we_lbo) >> 4);
          for (int ks = 0; ks < k_steps1; ++ks) {
            umma_f16(d, ad, bd, idesc1, ks > 0 ? 1u : 0u);
            ad += ad_step;
            bd += bd_step;
          }
        }
        umma_commit(smem_u32(&hdr->d1_full[buf]));
        return true;
      };
      for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++ul) {
        if (!mbar_wait_parked(smem_u32(&hdr->x_full), ul & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrMma)) break;
        tc_fence_after();
        // one expansion per team is in flight ahead of the projections
        ok = expand(g, 0);
        if (ok && p.n_chunks > 1) ok = expand(g + 1, 1);
        for (int c = 0; c < p.n_chunks && ok; ++c) {
          const unsigned gp = g + c, stage = gp % p.stages, k = static_cast<unsigned>(c) & 1u;
          // with three stages the weights of chunk c + 2 arrive while chunk c is being worked on; with two, its stage
          // is the one projection(c) frees, so that expansion can only follow the projection
          const bool early = p.stages >= 3 && c + 2 < p.n_chunks;
          if (early) {
            ok = expand(gp + 2, c + 2);
            if (!ok) break;
          }
          if (c == 0 && !mbar_wait_parked(smem_u32(&hdr->d2_empty), (ul & 1u) ^ 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrMma)) {
            ok = false;
            break;
          }
          if (!mbar_wait_parked(smem_u32(&hdr->a2_full[k]), n_prj[k] & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrMma)) {
            ok = false;
            break;
          }
          ++n_prj[k];
          tc_fence_after();
          const unsigned wp = st0 + stage * p.stage_bytes + p.we_bytes;
          const unsigned a2 = a20 + k * p.a2_bytes;
          for (int t = 0; t < p.mt_out; ++t)
            for (int h = 0; h < p.n_split; ++h) {
              const unsigned d = tmem_base + p.d2_col0 + static_cast<unsigned>(t * p.cout_pad + h * p.n_each);
              unsigned long long ad = smem_desc(a2 + static_cast<unsigned>(t) * 2048u, p.a2_pitch, 128);
              unsigned long long bd = smem_desc(wp + static_cast<unsigned>(h * p.n_each) * 16u, wp_lbo, 128);
              const unsigned long long ad_step = static_cast<unsigned long long>((2u * p.a2_pitch) >> 4);
              const unsigned long long bd_step = static_cast<unsigned long long>((2u * wp_lbo) >> 4);
#pragma unroll
              for (int ks = 0; ks < kNh / 16; ++ks) {
                umma_f16(d, ad, bd, idesc2, (c > 0 || ks > 0) ? 1u : 0u);
                ad += ad_step;
                bd += bd_step;
              }
            }
          umma_commit(smem_u32(&hdr->a2_empty[k]));
          umma_commit(smem_u32(&hdr->w_empty[stage]));
          if (c == p.n_chunks - 1) umma_commit(smem_u32(&hdr->d2_full));
          if (ul == GI_TRACE_UNIT) IR_EV(8 * c + 7);
          if (!early && p.stages < 3 && c + 2 < p.n_chunks) ok = expand(gp + 2, c + 2);
        }
        g += p.n_chunks;
      }
    }
  } else {
    // ------------------------------------------------------------ compute warps
    // Two teams of eight warps take alternate chunks of a unit (team = chunk parity), each with its own expansion
    // accumulator, hidden tile and A2 buffer: while one team waits for tensor memory or a barrier, the other one's
    // stencil keeps the FMA pipe busy.  Warps 0-3 and 8-11 of the sixteen form team 0, so each team has two warps on
    // every TMEM lane quarter (and on every scheduler).
    const int cw = warp - 2, ctid = threadIdx.x - 64;
    const int team = (cw >> 2) & 1;
    const int ttid = ((cw & 3) | ((cw >> 3) << 2)) * 32 + lane;  // 0 .. 255 within the team
    const int quarter = warp & 3, qsub = cw >> 3;                // TMEM lane quarter; index among the team's two warps on it
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int rows_in = p.n_img * p.r_in, rows_out = p.n_img * p.r_out;
    const unsigned hb = h0 + static_cast<unsigned>(team) * p.h_bytes;    // this team's hidden tile
    const unsigned a2b = a20 + static_cast<unsigned>(team) * p.a2_bytes; // ... and A2 buffer

    // copies of a unit's X by `nthr` threads (index `tid`): thread i takes (slice, row) pairs i, i + nthr, ...; consecutive
    // threads take consecutive pixels of one slice (coalesced 8-byte reads); rows of images beyond the batch are left as
    // they are (their results are never stored)
    auto issue_x = [&](int u, int tid, int nthr) {
      const int b0 = u * p.n_img;
      const bool second_ok = b0 + 1 < p.B;  // a unit holds one or two images
      for (int r = tid; r < rows_in; r += nthr) {
        const int img = r >= p.r_in ? 1 : 0, q = r - img * p.r_in;
        if (img && !second_ok) continue;
        const __half* src = p.in + (static_cast<size_t>(b0 + img) * p.Pin + q) * 4;
        const size_t slice_stride = static_cast<size_t>(p.B) * p.Pin * 4;  // halves between two slices of the tensor
        unsigned dst = x0 + static_cast<unsigned>(r) * 16u;
        for (int s = 0; s < p.s_in; s += 2) {
          cp_async8(dst, src);
          cp_async8(dst + 8u, src + slice_stride);
          src += 2 * slice_stride;
          dst += p.x_pitch;
        }
      }
    };

    // the hidden tiles' borders are the zero padding of the depthwise convolution: cleared once, never written again
    for (unsigned i = ctid; i < 2u * p.h_bytes / 16u; i += kComputeThreads)
      asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(h0 + i * 16u), "r"(0u) : "memory");

    // where this thread's accumulator rows go in a hidden tile (its rows are fixed: lane of the quarter, per 128-row tile)
    unsigned dr_off[2];
    bool dr_valid[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int row = t * 128 + quarter * 32 + lane;
      const int img = row / p.r_in, q = row - img * p.r_in;
      const int y = q / p.W, x = q - y * p.W;
      dr_valid[t] = t < p.mt_in && row < rows_in;
      dr_off[t] = (static_cast<unsigned>(img) * p.plane_words + static_cast<unsigned>((y + 1) * p.Wp + x + 1)) * 8u;
    }
    const unsigned slice_pitch = static_cast<unsigned>(p.n_img) * p.plane_words * 8u;  // planes of one slice: one per image

    // this thread's place in its team's stencil: (band, plane = slice of the chunk x image, output column)
    const int planes = (kNh / 4) * p.n_img;
    const int per_band = planes * p.Wo;
    const int band = ttid / per_band;
    const bool st_active = band < p.n_bands;
    const int st_rem = ttid - band * per_band;
    const int st_plane = st_rem / p.Wo, st_ox = st_rem - st_plane * p.Wo;
    const int st_slice = st_plane / p.n_img, st_img = st_plane - st_slice * p.n_img;
    const int st_r0 = band * p.band_rows, st_r1 = min(p.Ho, st_r0 + p.band_rows);
    const unsigned st_h = hb + static_cast<unsigned>(st_plane) * p.plane_words * 8u;
    const unsigned st_a2 = a2b + static_cast<unsigned>(st_slice >> 1) * p.a2_pitch + static_cast<unsigned>(st_img * p.r_out) * 16u +
                           static_cast<unsigned>(st_slice & 1) * 8u;

    bool ok = true;
    if (ctid == 0) IR_EV(60);
    pdl_wait();  // activations are read and written only below
    if (ctid == 0) IR_EV(61);
    if (static_cast<int>(blockIdx.x) < p.units) issue_x(blockIdx.x, ctid, kComputeThreads);
    cp_async_wait_all();
    fence_async_proxy();
    bar_compute();
    if (ctid == 0 && static_cast<int>(blockIdx.x) < p.units) mbar_arrive(smem_u32(&hdr->x_full));
    if (ctid == 0) IR_EV(62);

    unsigned g = 0, ul = 0, uses = 0;  // uses: chunks this team has worked on (the phase of its barriers)
    for (int u = blockIdx.x; u < p.units; u += gridDim.x, ++ul) {
      const int b0 = u * p.n_img;
      const bool more = u + static_cast<int>(gridDim.x) < p.units;
      for (int c = team; c < p.n_chunks; c += 2, ++uses) {
        const unsigned gc = g + c, stage = gc % p.stages;
        const unsigned dw0 = st0 + stage * p.stage_bytes + p.we_bytes + p.wp_bytes;  // depthwise taps [9][64], depthwise bias [64], expansion bias [64]
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 0);
        // ---- drain this chunk's expansion: 16 hidden channels of one pixel per tcgen05.ld; bias, activation, fp16 -> hidden tile
        ok = ok && mbar_wait_warp(smem_u32(&hdr->w_full[stage]), (gc / p.stages) & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrCompute);
        ok = ok && mbar_wait_warp(smem_u32(&hdr->d1_full[team]), uses & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrCompute);
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 2);
        if (ok) {
          tc_fence_after();
          // a team warp takes two of the four 16-column groups of its lane quarter, in both 128-row tiles; a group's 16
          // biases are requested together with the accumulator columns
          for (int e = 0; e < 2 * p.mt_in; ++e) {
            const int t = e >> 1, j = qsub * 2 + (e & 1);
            unsigned r[16];
            tmem_ld16(tmem_base + lane_bits + static_cast<unsigned>(team) * d1_cols + static_cast<unsigned>(t * kNh + j * 16), r);
            float4 b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) b[i] = lds128f(dw0 + 10u * kNh * 4u + static_cast<unsigned>(j * 4 + i) * 16u);
            tmem_ld_wait16(r);
            store_hidden(r, b, hb + static_cast<unsigned>(j * 4) * slice_pitch + (t ? dr_off[1] : dr_off[0]), slice_pitch,
                         t ? dr_valid[1] : dr_valid[0], p.act1);
          }
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(smem_u32(&hdr->d1_empty[team]));
        // the unit's last expansion is complete (its accumulator has just been read, and MMAs finish in order): X may
        // be overwritten with the next unit's
        if (c == p.n_chunks - 1 && more && ok) issue_x(u + gridDim.x, ttid, kTeamThreads);
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 1);
        bar_team(team);  // the hidden tile is complete

        // ---- this thread's depthwise weights (its slice of the chunk) into registers, then the stage is released
        float2 wlo[9], whi[9];
        Tap bias;
        if (ok && st_active) {
#pragma unroll
          for (int k = 0; k < 9; ++k) {
            const float4 w = lds128f(dw0 + (k * kNh + st_slice * 4) * 4u);
            wlo[k] = make_float2(w.x, w.y);
            whi[k] = make_float2(w.z, w.w);
          }
          const float4 b = lds128f(dw0 + (9 * kNh + st_slice * 4) * 4u);
          bias.lo = make_float2(b.x, b.y);
          bias.hi = make_float2(b.z, b.w);
        }
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(smem_u32(&hdr->w_empty[stage]));
        ok = ok && mbar_wait_warp(smem_u32(&hdr->a2_empty[team]), (uses & 1u) ^ 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrCompute);
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 3);

        // ---- depthwise 3x3 from the hidden tile -> A operand of the projection
        if (ok && st_active) {
          auto emit = [&](const Tap& a, int oy) {
            sts64(st_a2 + static_cast<unsigned>(oy * p.Wo + st_ox) * 16u, pack_act(a.lo.x, a.lo.y, p.act2), pack_act(a.hi.x, a.hi.y, p.act2));
          };
          if (STRIDE == 1 && PLANE == 14) {
            stencil_column<14, 16>(st_h + static_cast<unsigned>(st_ox) * 8u, st_a2 + static_cast<unsigned>(st_ox) * 16u, wlo, whi, bias, p.act2);
          } else if (STRIDE == 1 && PLANE == 7) {
            stencil_column<7, 9>(st_h + static_cast<unsigned>(st_ox) * 8u, st_a2 + static_cast<unsigned>(st_ox) * 16u, wlo, whi, bias, p.act2);
          } else if (STRIDE == 1) {
            // padded row iy (image row iy - 1) is tap row 0 of output row iy, row 1 of iy - 1, row 2 of iy - 2
            Tap a0 = bias, a1 = bias, a2 = bias;
            auto step = [&](Tap& done, Tap& mid, Tap& fresh, int iy) {
              const unsigned at = st_h + static_cast<unsigned>(iy * p.Wp + st_ox) * 8u;
              const Tap t0 = tap_of(lds64(at)), t1 = tap_of(lds64(at + 8u)), t2 = tap_of(lds64(at + 16u));
              done.lo = __ffma2_rn(t0.lo, wlo[6], done.lo);
              done.hi = __ffma2_rn(t0.hi, whi[6], done.hi);
              done.lo = __ffma2_rn(t1.lo, wlo[7], done.lo);
              done.hi = __ffma2_rn(t1.hi, whi[7], done.hi);
              done.lo = __ffma2_rn(t2.lo, wlo[8], done.lo);
              done.hi = __ffma2_rn(t2.hi, whi[8], done.hi);
              if (iy - 2 >= st_r0) emit(done, iy - 2);
              mid.lo = __ffma2_rn(t0.lo, wlo[3], mid.lo);
              mid.hi = __ffma2_rn(t0.hi, whi[3], mid.hi);
              mid.lo = __ffma2_rn(t1.lo, wlo[4], mid.lo);
              mid.hi = __ffma2_rn(t1.hi, whi[4], mid.hi);
              mid.lo = __ffma2_rn(t2.lo, wlo[5], mid.lo);
              mid.hi = __ffma2_rn(t2.hi, whi[5], mid.hi);
              fresh.lo = __ffma2_rn(t0.lo, wlo[0], bias.lo);
              fresh.hi = __ffma2_rn(t0.hi, whi[0], bias.hi);
              fresh.lo = __ffma2_rn(t1.lo, wlo[1], fresh.lo);
              fresh.hi = __ffma2_rn(t1.hi, whi[1], fresh.hi);
              fresh.lo = __ffma2_rn(t2.lo, wlo[2], fresh.lo);
              fresh.hi = __ffma2_rn(t2.hi, whi[2], fresh.hi);
            };
            // with one row of padding above, output row oy reads padded rows oy .. oy + 2
            const int last = st_r1 + 1;
            for (int iy = st_r0;;) {
              step(a0, a1, a2, iy);
              if (++iy > last) break;
              step(a1, a2, a0, iy);
              if (++iy > last) break;
              step(a2, a0, a1, iy);
              if (++iy > last) break;
            }
          } else {
            for (int oy = st_r0; oy < st_r1; ++oy) {
              Tap a = bias;
#pragma unroll
              for (int ky = 0; ky < 3; ++ky) {
                const unsigned at = st_h + static_cast<unsigned>((oy * 2 - p.pt + ky + 1) * p.Wp + st_ox * 2 - p.pl + 1) * 8u;
#pragma unroll
                for (int kx = 0; kx < 3; ++kx) {
                  const Tap t = tap_of(lds64(at + kx * 8u));
                  a.lo = __ffma2_rn(t.lo, wlo[ky * 3 + kx], a.lo);
                  a.hi = __ffma2_rn(t.hi, whi[ky * 3 + kx], a.hi);
                }
              }
              emit(a, oy);
            }
          }
        }
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 4);
        fence_async_proxy();  // the A operand was written with ordinary stores; the MMA reads it through the async proxy
        // the team that worked on the unit's last chunk also requested the next unit's X: its copies must have landed
        // before the barrier that publishes them
        if (c == p.n_chunks - 1 && more) {
          cp_async_wait_all();
          fence_async_proxy();
        }
        bar_team(team);       // A2 is complete; nobody in the team reads this hidden tile any more
        if (ttid == 0 && ok) {
          mbar_arrive(smem_u32(&hdr->a2_full[team]));
          if (c == p.n_chunks - 1 && more) mbar_arrive(smem_u32(&hdr->x_full));
        }
        if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(8 * c + 5);
      }
      g += p.n_chunks;
      // ---- unit end.  Team 0 goes straight on to the next unit; team 1 first drains D2 (the next unit's first
      // projection, which needs D2 free, comes a whole chunk of team 0's work later), which also puts the two teams
      // half a chunk apart: while one runs its stencil the other waits for tensor memory.
      if (team == 0) continue;

      // the residual does not depend on the accumulator: the first item's is fetched before waiting for the last
      // projection, each further item's while the one before it is processed
      const int groups = p.cout_pad >> 4, n_items = p.mt_out * groups;
      const size_t o_slice = static_cast<size_t>(p.B) * p.Pout * 4;  // halves between two slices of the output
      // where this thread's rows of the two output tiles are stored (a unit holds one or two images)
      size_t ep_off[2];
      bool ep_valid[2], ep_last[2];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int row = t * 128 + quarter * 32 + lane;
        const int img = row >= p.r_out ? 1 : 0, q = row - img * p.r_out;
        ep_valid[t] = t < p.mt_out && row < rows_out && b0 + img < p.B;
        ep_off[t] = (static_cast<size_t>(b0 + img) * p.Pout + q) * 4;
        ep_last[t] = q == p.r_out - 1;
      }
      auto fetch_res = [&](uint2* dstq, int e) {
        const int t = e / groups, j = e - t * groups;
        const bool valid = e < n_items && (t ? ep_valid[1] : ep_valid[0]);
        const __half* src = p.res + (t ? ep_off[1] : ep_off[0]) + static_cast<size_t>(j * 4) * o_slice;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          dstq[i] = make_uint2(0u, 0u);
          if (p.has_res && valid && j * 4 + i < p.s_out) dstq[i] = __ldg(reinterpret_cast<const uint2*>(src + i * o_slice));
        }
      };
      uint2 res_cur[4], res_nxt[4];
      fetch_res(res_cur, qsub);
      ok = ok && mbar_wait_warp(smem_u32(&hdr->d2_full), ul & 1u, abort_flag, p.timeout_ns, &g_ir_error, kErrCompute);
      if (ok) {
        tc_fence_after();
        const bool plain = p.act3 == GI_ACT_NONE && p.act4 == GI_ACT_NONE;  // the linear projection of an inverted-residual block
        for (int e = qsub; e < n_items; e += 2) {
          const int t = e / groups, j = e - t * groups;
          const bool valid = t ? ep_valid[1] : ep_valid[0], last_px = t ? ep_last[1] : ep_last[0];
          unsigned r[16];
          tmem_ld16(tmem_base + lane_bits + p.d2_col0 + static_cast<unsigned>(t * p.cout_pad + j * 16), r);
          fetch_res(res_nxt, e + 2);
          __half* dst = p.out + (t ? ep_off[1] : ep_off[0]) + static_cast<size_t>(j * 4) * o_slice;
          tmem_ld_wait16(r);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int so = j * 4 + i;
            if (so >= p.s_out || !valid) continue;
            const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias2) + so);
            float v0 = __uint_as_float(r[4 * i]) + b.x, v1 = __uint_as_float(r[4 * i + 1]) + b.y;
            float v2 = __uint_as_float(r[4 * i + 2]) + b.z, v3 = __uint_as_float(r[4 * i + 3]) + b.w;
            if (!plain) {
              v0 = act1f(v0, p.act3);
              v1 = act1f(v1, p.act3);
              v2 = act1f(v2, p.act3);
              v3 = act1f(v3, p.act3);
            }
            if (p.has_res) {
              const float2 q0 = __half22float2(*reinterpret_cast<const __half2*>(&res_cur[i].x));
              const float2 q1 = __half22float2(*reinterpret_cast<const __half2*>(&res_cur[i].y));
              v0 += q0.x;
              v1 += q0.y;
              v2 += q1.x;
              v3 += q1.y;
            }
            if (!plain) {
              v0 = act1f(v0, p.act4);
              v1 = act1f(v1, p.act4);
              v2 = act1f(v2, p.act4);
              v3 = act1f(v3, p.act4);
            }
            uint2 o;
            o.x = pack_f16x2<false>(v0, v1);
            o.y = pack_f16x2<false>(v2, v3);
            __half* at = dst + i * o_slice;
            *reinterpret_cast<uint2*>(at) = o;
            // an odd plane is stored with one extra pixel, which readers expect to be finite: zero it
            if (p.Pout > p.r_out && last_px) *reinterpret_cast<uint2*>(at + 4) = make_uint2(0u, 0u);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) res_cur[i] = res_nxt[i];
        }
        tc_fence_before();
      }
      __syncwarp();
      if (lane == 0 && ok) mbar_arrive(smem_u32(&hdr->d2_empty));
      if (ttid == 0 && ul == GI_TRACE_UNIT) IR_EV(63);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

struct Shape {
  int n_img, mt_in, mt_out, r_in, r_out, n_chunks, cout_pad, n_split, n_each, Wp, plane_words, n_bands, band_rows, stages;
  unsigned we_bytes, wp_bytes, stage_bytes, x_bytes, a2_bytes, h_bytes, x_pitch, a2_pitch;
  size_t smem;
  long long units;
  bool ok;
};

Shape shape_of(int B, int H, int W, int Ho, int Wo, int stride, int cin, int chid, int cout) {
  Shape s{};
  s.ok = false;
  if (cin <= 0 || cin % 16 != 0 || chid <= 0 || cout <= 0) return s;
  s.r_in = H * W;
  s.r_out = Ho * Wo;
  if (s.r_in > 256 || s.r_in < 4) return s;
  // as many whole images as fill one 128-row tile; a larger image takes two tiles by itself
  s.n_img = s.r_in <= 128 ? 128 / s.r_in : 1;
  if (s.n_img > B) s.n_img = B;
  if (s.n_img > 2) s.n_img = 2;  // planes of the hidden tile: 16 slices x images; more images only shorten the columns walked
  s.mt_in = (s.n_img * s.r_in + 127) / 128;
  s.mt_out = (s.n_img * s.r_out + 127) / 128;
  s.n_chunks = (chid + kNh - 1) / kNh;
  s.cout_pad = (cout + 15) / 16 * 16;
  s.n_split = (s.cout_pad + 255) / 256;
  while (s.cout_pad % (16 * s.n_split) != 0) ++s.n_split;
  s.n_each = s.cout_pad / s.n_split;
  // tensor memory: two expansion accumulators and the projection accumulator
  if (2 * s.mt_in * kNh + s.mt_out * s.cout_pad > 512) return s;
  s.Wp = W + 2;
  s.plane_words = (H + 2) * s.Wp;
  while (s.plane_words % 16 != W % 16) ++s.plane_words;  // consecutive planes start W words apart (mod 16): no bank conflicts
  const int planes = (kNh / 4) * s.n_img;
  int bands = kTeamThreads / (planes * Wo);
  if (bands < 1) return s;
  if (bands > Ho) bands = Ho;
  s.band_rows = (Ho + bands - 1) / bands;
  s.n_bands = (Ho + s.band_rows - 1) / s.band_rows;
  s.we_bytes = static_cast<unsigned>(kNh) * cin * 2u;
  s.wp_bytes = static_cast<unsigned>(s.cout_pad) * kNh * 2u;
  s.stage_bytes = s.we_bytes + s.wp_bytes + kDwBytes;
  // The K groups of an operand lie `rows x 16 bytes` apart, rows = the unit's real pixel count.  An MMA reads 128
  // rows per tile, so the tail of the last tile reads on into the next K group (and, for the last group, into the
  // region behind the operand): rows that hold no pixel, whose results are never stored.
  s.x_pitch = static_cast<unsigned>(s.n_img * s.r_in) * 16u;
  s.a2_pitch = static_cast<unsigned>(s.n_img * s.r_out) * 16u;
  s.x_bytes = (static_cast<unsigned>(cin / 8) * s.x_pitch + 127u) / 128u * 128u;
  s.a2_bytes = (static_cast<unsigned>(kNh / 8) * s.a2_pitch + 127u) / 128u * 128u;
  s.h_bytes = (static_cast<unsigned>(planes) * s.plane_words * 8u + 127u) / 128u * 128u;
  // (the tail reads of A2's last K group land in the hidden tiles, 2 x h_bytes >= 2 KB, those of X in A2 or behind)
  const long long fixed = kHeader + static_cast<long long>(s.x_bytes) + 2ll * s.a2_bytes + 2ll * s.h_bytes;
  long long stages = (kSmemMax - fixed) / s.stage_bytes;
  if (stages < 2) return s;
  s.stages = stages > kMaxStages ? kMaxStages : static_cast<int>(stages);
  s.smem = static_cast<size_t>(fixed) + static_cast<size_t>(s.stages) * s.stage_bytes;
  s.units = (static_cast<long long>(B) + s.n_img - 1) / s.n_img;
  (void)stride;
  s.ok = true;
  return s;
}

}  // namespace

bool inverted_residual_supported(int B, int H, int W, int Ho, int Wo, int stride, int dil, int pt, int pl, int cin, int chid,
                                 int cout, long long* units) {
  if (stride < 1 || stride > 2 || dil != 1 || pt < 0 || pt > 1 || pl < 0 || pl > 1) return false;
  // every tap must stay inside the padded hidden tile (one zero row / column on each side)
  if ((Ho - 1) * stride - pt + 2 > H || (Wo - 1) * stride - pl + 2 > W) return false;
  if (stride == 1 && (pt != 1 || pl != 1 || Ho != H || Wo != W)) return false;
  const Shape s = shape_of(B, H, W, Ho, Wo, stride, cin, chid, cout);
  if (!s.ok) return false;
  if (units) *units = s.units;
  return true;
}

// Per chunk of 64 hidden channels one contiguous block: We[cin/8][64][8] (expansion rows of the chunk, K-major core
// matrices), Wp[8][cout_pad][8] (projection columns of the chunk), depthwise taps [9][64], depthwise bias [64],
// expansion bias [64] (floats).  Hidden channels beyond `chid` are zero throughout, so they contribute nothing.
void inverted_residual_pack(const float* we, const float* be, const float* wd, const float* bd, const float* wp, const float* bp,
                            int cin, int chid, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Shape s = shape_of(r->B, r->H, r->W, r->Ho, r->Wo, r->sh, cin, chid, cout);
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + static_cast<size_t>(s.n_chunks) * s.stage_bytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(s.cout_pad) * sizeof(float), 0);
  for (int c = 0; c < s.n_chunks; ++c) {
    uint8_t* base = blob->data() + woff + static_cast<size_t>(c) * s.stage_bytes;
    uint16_t* pe = reinterpret_cast<uint16_t*>(base);
    uint16_t* pp = reinterpret_cast<uint16_t*>(base + s.we_bytes);
    float* pd = reinterpret_cast<float*>(base + s.we_bytes + s.wp_bytes);
    for (int n = 0; n < kNh; ++n) {
      const int hch = c * kNh + n;
      if (hch >= chid) continue;
      for (int ci = 0; ci < cin; ++ci)
        pe[(static_cast<size_t>(ci / 8) * kNh + n) * 8 + ci % 8] = f32_to_f16_rne(we[static_cast<size_t>(hch) * cin + ci]);
      for (int co = 0; co < cout; ++co)
        pp[(static_cast<size_t>(n / 8) * s.cout_pad + co) * 8 + n % 8] = f32_to_f16_rne(wp[static_cast<size_t>(co) * chid + hch]);
      for (int k = 0; k < 9; ++k) {
        // the depthwise taps take part in the arithmetic as the fp16 values the stored weights would have
        const uint16_t hb = f32_to_f16_rne(wd[static_cast<size_t>(k) * chid + hch]);
        const uint32_t sg = (hb & 0x8000u) << 16, ex = (hb >> 10) & 0x1fu, m = hb & 0x3ffu;
        float v;
        uint32_t bits;
        if (ex == 0) {
          v = static_cast<float>(m) * (1.0f / 16777216.0f);
          std::memcpy(&bits, &v, 4);
        } else if (ex == 31) {
          bits = 0x7f800000u | (m << 13);
        } else {
          bits = ((ex + 112u) << 23) | (m << 13);
        }
        bits |= sg;
        std::memcpy(&v, &bits, 4);
        pd[k * kNh + n] = v;
      }
      pd[9 * kNh + n] = bd[hch];
      pd[10 * kNh + n] = be[hch];
    }
  }
  float* b2 = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) b2[co] = bp[co];
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias2 = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = static_cast<uint64_t>(s.n_chunks) * s.stage_bytes;
}

int launch_inverted_residual(const LaunchRec& r, const Ptrs& p, void* stream) {
  const Shape s = shape_of(r.B, r.H, r.W, r.Ho, r.Wo, r.sh, r.C, r.Cmid, r.Co2);
  if (!s.ok) return static_cast<int>(cudaErrorInvalidConfiguration);
  IrParams k{};
  k.in = static_cast<const __half*>(p.in0);
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.bias2 = static_cast<const float*>(p.bias2);
  k.B = r.B;
  k.H = r.H;
  k.W = r.W;
  k.Pin = plane_pixels(r.H, r.W);
  k.Ho = r.Ho;
  k.Wo = r.Wo;
  k.Pout = plane_pixels(r.Ho, r.Wo);
  k.stride = r.sh;
  k.pt = r.pt;
  k.pl = r.pl;
  k.s_in = r.C / 4;
  k.n_chunks = s.n_chunks;
  k.cout_pad = s.cout_pad;
  k.s_out = slices(r.Co2);
  k.n_split = s.n_split;
  k.n_each = s.n_each;
  k.n_img = s.n_img;
  k.r_in = s.r_in;
  k.r_out = s.r_out;
  k.mt_in = s.mt_in;
  k.mt_out = s.mt_out;
  k.units = static_cast<int>(s.units);
  k.Wp = s.Wp;
  k.plane_words = s.plane_words;
  k.n_bands = s.n_bands;
  k.band_rows = s.band_rows;
  k.stages = s.stages;
  k.stage_bytes = s.stage_bytes;
  k.we_bytes = s.we_bytes;
  k.wp_bytes = s.wp_bytes;
  k.x_bytes = s.x_bytes;
  k.a2_bytes = s.a2_bytes;
  k.h_bytes = s.h_bytes;
  k.x_pitch = s.x_pitch;
  k.a2_pitch = s.a2_pitch;
  k.d2_col0 = 2u * static_cast<unsigned>(s.mt_in) * kNh;
  k.act1 = r.ep.act_pre;
  k.act2 = r.ep_mid.act_pre;
  k.act3 = r.ep2.act_pre;
  k.has_res = r.ep2.has_res;
  k.act4 = r.ep2.act_post;
  k.timeout_ns = 1000000000u;
  static bool attr_done_dev[kMaxDevices] = {};
  bool& attr_done = attr_done_dev[current_device_slot()];
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(inverted_residual_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(inverted_residual_kernel<1, 14>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(inverted_residual_kernel<1, 7>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(inverted_residual_kernel<2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_done = true;
  }
  const int sms = device_sm_count();
  const unsigned grid = static_cast<unsigned>(s.units < sms ? s.units : sms);
  // the kernel reserves all of tensor memory: ask for enough shared memory that no second CTA shares the SM
  size_t smem = s.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool whole_column = r.sh == 1 && s.n_bands == 1 && r.H == r.W;  // a thread walks a whole column of its plane
  if (whole_column && r.H == 14) launch_pdl(inverted_residual_kernel<1, 14>, grid, kThreads, smem, st, k);
  else if (whole_column && r.H == 7) launch_pdl(inverted_residual_kernel<1, 7>, grid, kThreads, smem, st, k);
  else if (r.sh == 1) launch_pdl(inverted_residual_kernel<1, 0>, grid, kThreads, smem, st, k);
  else launch_pdl(inverted_residual_kernel<2, 0>, grid, kThreads, smem, st, k);
  return static_cast<int>(cudaGetLastError());
}

#ifdef GI_TRACE
int inverted_residual_trace(unsigned long long* dst, int n) {
  const size_t bytes = sizeof(unsigned long long) * (n < 256 * 64 ? n : 256 * 64);
  return static_cast<int>(cudaMemcpyFromSymbol(dst, g_ir_trace, bytes));
}
#endif

unsigned int inverted_residual_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_ir_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
