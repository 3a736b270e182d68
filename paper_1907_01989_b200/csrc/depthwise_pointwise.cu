// Depthwise 3x3 convolution and the pointwise (1x1) convolution that consumes it, as ONE kernel
// (fp16 storage).  The paper's cure for a memory-bound engine is fewer, fatter programs (Section
// 3.3 folds element-wise operators into their producer); this goes one step further and folds a
// whole operator: the depthwise output - in an inverted-residual block the widest tensor of the
// network - is never written to memory.  It is produced 16 channels at a time, rounded to fp16
// exactly as the stored tensor would have been, and written straight into TENSOR MEMORY as the A
// operand of the 1x1 convolution's MMAs.
//
// A pixel tile is a band of `th` output rows of `nb` images.  A TMEM lane is an output COLUMN
// (image, x) of the tile - nb * Wo <= 128 of them - and each output row of the band is its own
// 128-row accumulator (row j of the band = accumulator j).  That is the shape the stencil wants:
// a thread owns one column and walks down the band, every staged input row feeding three running
// accumulators, exactly as in the stand-alone depthwise kernel; what it would have stored to
// memory it stores to tensor memory instead (tcgen05.st, two 32-bit columns = one 4-channel
// slice).  Sixteen compute warps form four groups; the groups take the four slices of a 16-channel
// chunk, so one pass of all warps produces the A operand of one MMA K step for every row of the
// band.  The MMA warp then multiplies A[row] (tensor memory) with the chunk's rows of the resident
// weight matrix (shared memory) into accumulator[row].  A chunks are double-buffered in tensor
// memory; input rows are staged by bulk copies into a ring of shared-memory stages (copy warp),
// one stage = the four slices of a chunk.  After the last chunk the compute warps drain the
// accumulators (bias, activation, residual, fp16; a warp's 32 lanes write 32 consecutive pixels of
// an output row) while the copy warp already fetches the next tile.  All waits are bounded.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kGroups = 4;  // compute warp groups = slices of a chunk
constexpr int kComputeWarps = 4 * kGroups;
constexpr int kComputeThreads = 32 * kComputeWarps;
constexpr int kCopyWarp = kComputeWarps, kMmaWarp = kComputeWarps + 1;
constexpr int kThreads = 32 * (kComputeWarps + 2);
constexpr int kHeader = 1024;
constexpr int kMaxBuf = 4;
constexpr int kTmemCols = 512;
constexpr int kACols = 8;  // 16 fp16 channels of one pixel = 8 32-bit columns

__device__ unsigned int g_fu_error = 0;
enum : unsigned { kErrCopy = 1u, kErrMma = 2u, kErrCompute = 4u, kErrDrain = 8u };

#ifdef GI_TRACE
__device__ unsigned long long g_fu_trace[1024 * 64];
#define FU_EV(idx)                                           \
  do {                                                       \
    if (blockIdx.x < 1024 && (idx) < 64) {                   \
      unsigned long long t_;                                 \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
      g_fu_trace[blockIdx.x * 64 + (idx)] = t_;              \
    }                                                        \
  } while (0)
#else
#define FU_EV(idx) ((void)0)
#endif

struct FuGeom {
  int B, H, W, Pin, Ho, Wo, Pout, S;  // S: slices of the depthwise tensor (a multiple of 4)
  int stride, pt, pl;
  int nb;  // images per pixel tile (nb * Wo <= 128 lanes)
  int th;  // output rows per tile = accumulators
  int bands, bchunks, tiles;
  int head_px, tail_px, plane_stride_px, nbuf;  // staging area of a plane: zero head, staged rows, room for a zero row behind
  int n_pad, s_out;  // output channels rounded up to 16; output slices
  int act_dw;        // activation of the depthwise op
  int act_pre, has_res, act_post;  // epilogue of the pointwise op
  int in_dead;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long full[kMaxBuf], empty[kMaxBuf];
  unsigned long long a_full[2], a_empty[2];
  unsigned long long acc_full, acc_free, b_ready;
  unsigned tmem_addr, abort_flag;
};
static_assert(sizeof(Header) <= kHeader, "header too large");

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

struct Row {
  float2 lo[3], hi[3];
};
struct Acc {
  float2 lo, hi;
};
__device__ __forceinline__ void fma_row(Acc& a, const Row& r, const float2* wlo, const float2* whi) {
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    a.lo = __ffma2_rn(r.lo[k], wlo[k], a.lo);
    a.hi = __ffma2_rn(r.hi[k], whi[k], a.hi);
  }
}
__device__ __forceinline__ Acc fma_row_from(const Acc& bias, const Row& r, const float2* wlo, const float2* whi) {
  Acc a;
  a.lo = __ffma2_rn(r.lo[0], wlo[0], bias.lo);
  a.hi = __ffma2_rn(r.hi[0], whi[0], bias.hi);
#pragma unroll
  for (int k = 1; k < 3; ++k) {
    a.lo = __ffma2_rn(r.lo[k], wlo[k], a.lo);
    a.hi = __ffma2_rn(r.hi[k], whi[k], a.hi);
  }
  return a;
}
__device__ __forceinline__ uint2 lds64(unsigned addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds128(unsigned addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ Row widen(const uint2* u) {
  Row r;
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    r.lo[k] = __half22float2(*reinterpret_cast<const __half2*>(&u[k].x));
    r.hi[k] = __half22float2(*reinterpret_cast<const __half2*>(&u[k].y));
  }
  return r;
}
// this warp's 32 lanes x 2 consecutive 32-bit columns of tensor memory
__device__ __forceinline__ void tmem_st2(unsigned taddr, unsigned a, unsigned b) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};" ::"r"(taddr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]^T, 128 x N x 16
__device__ __forceinline__ void umma_f16_ts(unsigned d_tmem, unsigned a_tmem, unsigned long long b_desc, unsigned idesc,
                                            unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// MODE 0: stride 1; MODE 1: stride 2 (both: dilation 1, at most one padding row / column on each
// side).  Staging area of one plane: [head_px zeros][rows of the band][a zero row behind the image
// when the band reaches its bottom]: the rows above and below the image read as zeros with no test
// in the loop; a tap column outside the image points at a zero pixel.  The zero row is a bulk copy
// from a zero-filled region of the weight buffer, so no thread has to write it.
// ACT6: the depthwise op ends in ReLU6 (the usual case; otherwise its activation is tested at run time).
template <int MODE, bool ACT6>
__global__ void __launch_bounds__(kThreads, 1)  // 96 registers: one scheduler holds five of the 18 warps
    depthwise_pointwise_kernel(const __half* __restrict__ in, const float* __restrict__ w, const float* __restrict__ bias,
                               const unsigned char* __restrict__ pw_w, const float* __restrict__ pw_bias,
                               const __half* __restrict__ res, __half* __restrict__ out, const FuGeom g) {
  // pw_bias: n_pad floats, followed by tail_px zero pixels
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned b_bytes = static_cast<unsigned>(g.S) * g.n_pad * 8u;  // S/2 K units x n_pad rows x 16 bytes
  const unsigned dw_bytes = static_cast<unsigned>(g.S) * 160u;         // depthwise weights [9][C] and bias [C], fp32
  const unsigned pb_bytes = static_cast<unsigned>(g.n_pad) * 4u;       // bias of the 1x1 convolution
  const unsigned b0 = smem_u32(smem + kHeader);
  const unsigned w_sm = b0 + b_bytes, pb_sm = w_sm + dw_bytes;
  const unsigned st0 = pb_sm + pb_bytes;
  const unsigned slice_bytes = static_cast<unsigned>(g.plane_stride_px) * 8u * g.nb;  // one slice of a tile's planes
  const unsigned buf_bytes = 4u * slice_bytes;                                          // a stage: the four slices of a chunk
  const int W = g.W, H = g.H, Wo = g.Wo, stride = g.stride, pt = g.pt;
  const int n_chunks = g.S >> 2;
  // TMEM: th accumulators, then two A buffers of th (rounded up to a multiple of three) x 8 columns
  const unsigned a_col0 = static_cast<unsigned>(g.th * g.n_pad);
  const unsigned a_buf_cols = static_cast<unsigned>((g.th + 2) / 3 * 3) * kACols;

  // contiguous, balanced range of pixel tiles for this CTA
  const int per = g.tiles / gridDim.x, extra = g.tiles % gridDim.x;
  const int first = blockIdx.x * per + min(static_cast<int>(blockIdx.x), extra);
  const int count = per + (static_cast<int>(blockIdx.x) < extra ? 1 : 0);

  auto tile_rows = [&](int tile, int& b0i, int& nbk, int& oy0, int& oy1, int& start_px, unsigned& bytes, bool& below) {
    const int bc = tile / g.bands, band = tile - bc * g.bands;
    b0i = bc * g.nb;
    nbk = min(g.nb, g.B - b0i);
    oy0 = band * g.th;
    oy1 = min(g.Ho, oy0 + g.th);
    const int in_y0 = max(0, oy0 * stride - pt);
    const int in_y1 = min(H, (oy1 - 1) * stride - pt + 3);
    start_px = in_y0 * W;
    start_px -= start_px & 1;  // copies start on a 16-byte boundary: at most one pixel early
    const int end_px = min((in_y1 * W + 1) & ~1, g.Pin);
    bytes = static_cast<unsigned>(end_px - start_px) * 8u;
    below = (oy1 - 1) * stride - pt + 2 >= H;  // the band reads row H: a zero row follows the staged rows
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < g.nbuf; ++i) {
      mbar_init(smem_u32(&hdr->full[i]), 1);
      mbar_init(smem_u32(&hdr->empty[i]), kComputeWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kComputeWarps);
      mbar_init(smem_u32(&hdr->a_empty[i]), 1);
    }
    mbar_init(smem_u32(&hdr->acc_full), 1);
    mbar_init(smem_u32(&hdr->acc_free), kComputeWarps);
    mbar_init(smem_u32(&hdr->b_ready), 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // zero pixels the copies never touch: the head of each plane's staging area
  {
    unsigned char* stg = smem + kHeader + b_bytes + dw_bytes + pb_bytes;
    for (int i = threadIdx.x; i < g.nbuf * 4 * g.nb * g.head_px; i += blockDim.x) {
      const int plane = i / g.head_px, px = i - plane * g.head_px;
      *reinterpret_cast<uint2*>(stg + (static_cast<size_t>(plane) * g.plane_stride_px + px) * 8) = make_uint2(0u, 0u);
    }
  }
  if (warp == kMmaWarp) tmem_alloc(smem_u32(&hdr->tmem_addr), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  pdl_launch_dependents();
  // weights never change after binding: their copy may start while the previous kernel still runs
  if (warp == kCopyWarp && lane == 0) {
    const unsigned bar = smem_u32(&hdr->b_ready);
    mbar_expect_tx(bar, b_bytes + dw_bytes + pb_bytes);
    for (unsigned off = 0; off < b_bytes; off += 16384u)
      bulk_load(b0 + off, pw_w + off, min(16384u, b_bytes - off), bar);
    bulk_load(w_sm, w, dw_bytes - static_cast<unsigned>(g.S) * 16u, bar);
    bulk_load(w_sm + dw_bytes - static_cast<unsigned>(g.S) * 16u, bias, static_cast<unsigned>(g.S) * 16u, bar);
    bulk_load(pb_sm, pw_bias, pb_bytes, bar);
  }
  pdl_wait();  // activations are read and written only below
  if (threadIdx.x == 0) FU_EV(48);

  if (warp == kCopyWarp) {
    // ------------------------------------------------------------ copy warp: input rows -> staging ring
    unsigned long long pol;
    if (g.in_dead) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    unsigned it = 0;
    bool ok = true;
    for (int t = 0; t < count && ok; ++t) {
      int b0i, nbk, oy0, oy1, start_px;
      unsigned bytes;
      bool below;
      tile_rows(first + t, b0i, nbk, oy0, oy1, start_px, bytes, below);
      for (int c = 0; c < n_chunks; ++c, ++it) {
        const unsigned stage = it % g.nbuf, phase = (it / g.nbuf) & 1u;
        if (!mbar_wait_parked(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, g.timeout_ns, &g_fu_error, kErrCopy)) {
          ok = false;
          break;
        }
        const unsigned bar = smem_u32(&hdr->full[stage]);
        const unsigned zero_bytes = below ? static_cast<unsigned>(g.tail_px) * 8u : 0u;
        // the phase cannot complete before this arrival, whatever order the copies land in
        if (lane == 0) mbar_expect_tx(bar, (bytes + zero_bytes) * nbk * 4u);
        __syncwarp();
        for (int q = lane; q < 4 * nbk; q += 32) {  // one copy per (slice of the chunk, plane)
          const int j = q / nbk, pi = q - j * nbk;
          const __half* src = in + ((static_cast<size_t>(4 * c + j) * g.B + b0i + pi) * g.Pin + start_px) * 4;
          const unsigned dst =
              st0 + stage * buf_bytes + j * slice_bytes + (static_cast<unsigned>(pi) * g.plane_stride_px + g.head_px) * 8u;
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                       "l"(src), "r"(bytes), "r"(bar), "l"(pol)
                       : "memory");
          if (below) bulk_load(dst + bytes, pw_bias + g.n_pad, zero_bytes, bar);
        }
        if (lane == 0 && it < 8) FU_EV(it);
      }
    }
    if (!ok && lane == 0) {
      // copies already issued may still land: wait (bounded) for them before the CTA may exit
      const unsigned first_it = it > static_cast<unsigned>(g.nbuf) ? it - g.nbuf : 0u;
      for (unsigned j = first_it; j < it; ++j) {
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&hdr->full[j % g.nbuf]), (j / g.nbuf) & 1u)) {
          if (global_timer_ns() - t0 > g.timeout_ns) {
            atomicOr(&g_fu_error, kErrDrain);
            break;
          }
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA warp
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, B K-major, M = 128, N = n_pad
      const unsigned idesc = (1u << 4) | ((static_cast<unsigned>(g.n_pad) >> 3) << 17) | ((128u >> 4) << 24);
      const unsigned b_lbo = static_cast<unsigned>(g.n_pad) * 16u;  // between consecutive 8-channel K units of the weights
      bool ok = mbar_wait(smem_u32(&hdr->b_ready), 0u, abort_flag, g.timeout_ns, &g_fu_error, kErrMma);
      unsigned ci = 0;
      for (int t = 0; t < count && ok; ++t) {
        int b0i, nbk, oy0, oy1, start_px;
        unsigned bytes;
        bool below;
        tile_rows(first + t, b0i, nbk, oy0, oy1, start_px, bytes, below);
        const int rows = oy1 - oy0;
        for (int c = 0; c < n_chunks; ++c, ++ci) {
          const unsigned abuf = ci & 1u, a_phase = (ci >> 1) & 1u;
          if (!mbar_wait_parked(smem_u32(&hdr->a_full[abuf]), a_phase, abort_flag, g.timeout_ns, &g_fu_error, kErrMma)) {
            ok = false;
            break;
          }
          // the first MMA of a tile overwrites the accumulators: the previous tile must have been drained
          if (c == 0 && t > 0 &&
              !mbar_wait(smem_u32(&hdr->acc_free), static_cast<unsigned>(t - 1) & 1u, abort_flag, g.timeout_ns, &g_fu_error, kErrMma)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (ci < 8) FU_EV(24 + ci);
          const unsigned long long bd = smem_desc(b0 + static_cast<unsigned>(c) * 2u * b_lbo, b_lbo, 128);
          const unsigned a_tmem = tmem_base + a_col0 + abuf * a_buf_cols;
          for (int j = 0; j < rows; ++j)
            umma_f16_ts(tmem_base + static_cast<unsigned>(j * g.n_pad), a_tmem + static_cast<unsigned>(j) * kACols, bd, idesc,
                        c > 0 ? 1u : 0u);
          umma_commit(smem_u32(&hdr->a_empty[abuf]));
          if (ci < 8) FU_EV(32 + ci);
        }
        if (ok) umma_commit(smem_u32(&hdr->acc_full));
      }
    }
  } else {
    // ------------------------------------------------------------ compute warps: stencil, then drain
    const int tid = threadIdx.x;
    const int group = warp >> 2, quarter = warp & 3;
    const int col = quarter * 32 + lane;  // TMEM lane = output column (image, x) of the tile
    const int C4 = g.S * 4;
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    unsigned it = 0, ci = 0;
    // the weights of both operators arrive once, before the first tile
    bool ok = mbar_wait_warp(smem_u32(&hdr->b_ready), 0u, abort_flag, g.timeout_ns, &g_fu_error, kErrCompute);
    // a finished tile waiting for its drain: accumulator row j -> pixel pend_off + j * Wo of every output slice
    bool pend = false;
    int pend_t = 0;
    const bool plain = g.act_pre == GI_ACT_NONE && g.act_post == GI_ACT_NONE;
    const size_t slice_stride = static_cast<size_t>(g.B) * g.Pout;  // pixels between output slices
    auto drain = [&]() {
      if (!mbar_wait_warp(smem_u32(&hdr->acc_full), static_cast<unsigned>(pend_t) & 1u, abort_flag, g.timeout_ns, &g_fu_error, kErrCompute)) {
        ok = false;
        return;
      }
      tc_fence_after();
      if (tid == 0 && pend_t < 4) FU_EV(40 + 2 * pend_t);
      // the tile's geometry is recomputed rather than carried through the stencil loop in registers
      int pend_b0, pend_nbk, p_oy0, p_oy1, p_start;
      unsigned p_bytes;
      bool p_below;
      tile_rows(first + pend_t, pend_b0, pend_nbk, p_oy0, p_oy1, p_start, p_bytes, p_below);
      const bool pend_ok = col < pend_nbk * Wo;
      const int p_pi = pend_ok ? col / Wo : 0;
      const size_t pend_off = static_cast<size_t>(pend_b0 + p_pi) * g.Pout + static_cast<size_t>(p_oy0) * Wo + (pend_ok ? col - p_pi * Wo : 0);
      const int pend_rows = p_oy1 - p_oy0;
      const bool pend_last = p_oy1 == g.Ho;
      if (tid == 0 && pend_t == 1) FU_EV(50);
      const int ngrp = g.n_pad >> 4;
      const int n_items = ((pend_rows - group + kGroups - 1) / kGroups) * ngrp;  // (row, 16-column group) pairs of this warp
      unsigned r[2][16];
      if (n_items > 0) tmem_ld16(tmem_base + lane_bits + static_cast<unsigned>(group * g.n_pad), r[0]);
      int j = group, grp = 0;
#pragma unroll 1
      for (int i = 0; i < n_items; i += 2) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {  // two register sets: the next load is in flight while one is processed
          if (i + h >= n_items) break;
          tmem_ld_wait16(r[h]);
          if (tid == 0 && pend_t == 1 && i + h < 4) FU_EV(51 + i + h);
          int jn = j, gn = grp + 1;
          if (gn == ngrp) {
            gn = 0;
            jn += kGroups;
          }
          if (i + h + 1 < n_items) tmem_ld16(tmem_base + lane_bits + static_cast<unsigned>(jn * g.n_pad + gn * 16), r[h ^ 1]);
          const size_t px = pend_off + static_cast<size_t>(j) * Wo;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int so = grp * 4 + q;
            if (so >= g.s_out || !pend_ok) continue;
            const float4 b = lds128(pb_sm + static_cast<unsigned>(so) * 16u);
            const size_t off = (static_cast<size_t>(so) * slice_stride + px) * 4;  // in halves
            float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[h][4 * q]), __uint_as_float(r[h][4 * q + 1])), make_float2(b.x, b.y));
            float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[h][4 * q + 2]), __uint_as_float(r[h][4 * q + 3])), make_float2(b.z, b.w));
            if (!plain) {
              v0 = make_float2(act1(v0.x, g.act_pre), act1(v0.y, g.act_pre));
              v1 = make_float2(act1(v1.x, g.act_pre), act1(v1.y, g.act_pre));
            }
            if (g.has_res) {
              const uint2 rq = __ldg(reinterpret_cast<const uint2*>(res + off));
              v0 = __fadd2_rn(v0, __half22float2(*reinterpret_cast<const __half2*>(&rq.x)));
              v1 = __fadd2_rn(v1, __half22float2(*reinterpret_cast<const __half2*>(&rq.y)));
            }
            if (!plain) {
              v0 = make_float2(act1(v0.x, g.act_post), act1(v0.y, g.act_post));
              v1 = make_float2(act1(v1.x, g.act_post), act1(v1.y, g.act_post));
            }
            uint2 o;
            o.x = pack_f16x2<false>(v0.x, v0.y);
            o.y = pack_f16x2<false>(v1.x, v1.y);
            *reinterpret_cast<uint2*>(out + off) = o;
          }
          j = jn;
          grp = gn;
        }
      }
      tc_fence_before();
      if (tid == 0 && pend_t < 4) FU_EV(41 + 2 * pend_t);
      // an odd plane carries one extra pixel: keep it zero
      if (pend_last && g.Pout > g.Ho * Wo) {
        for (int i = tid; i < pend_nbk * g.s_out; i += kComputeThreads) {
          const int so = i / pend_nbk, p2 = i - so * pend_nbk;
          const size_t off = ((static_cast<size_t>(so) * g.B + pend_b0 + p2) * g.Pout + g.Ho * Wo) * 4;
          *reinterpret_cast<uint2*>(out + off) = make_uint2(0u, 0u);
        }
      }
      pend = false;
    };
    for (int t = 0; t < count && ok; ++t) {
      int b0i, nbk, oy0, oy1, start_px;
      unsigned bytes;
      bool below;
      tile_rows(first + t, b0i, nbk, oy0, oy1, start_px, bytes, below);
      // lanes beyond the tile's columns repeat column 0: they compute and store into lanes nobody drains
      const bool col_ok = col < nbk * Wo;
      const int pi = col_ok ? col / Wo : 0;
      const int x = col_ok ? col - pi * Wo : 0;
      for (int ch = 0; ch < n_chunks && ok; ++ch, ++it, ++ci) {
        const unsigned abuf = ci & 1u;
        const int s = ch * 4 + group;
        float2 wlo[9], whi[9];
#pragma unroll
        for (int k = 0; k < 9; ++k) {
          const float4 v = lds128(w_sm + static_cast<unsigned>(k * C4 + s * 4) * 4u);
          wlo[k] = make_float2(v.x, v.y);
          whi[k] = make_float2(v.z, v.w);
        }
        Acc bias_acc;
        {
          const float4 v = lds128(w_sm + static_cast<unsigned>(9 * C4 + s * 4) * 4u);
          bias_acc.lo = make_float2(v.x, v.y);
          bias_acc.hi = make_float2(v.z, v.w);
        }
        if (!mbar_wait_warp(smem_u32(&hdr->a_empty[abuf]), ((ci >> 1) & 1u) ^ 1u, abort_flag, g.timeout_ns, &g_fu_error, kErrCompute)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const unsigned stage = it % g.nbuf;
        if (!mbar_wait_warp(smem_u32(&hdr->full[stage]), (it / g.nbuf) & 1u, abort_flag, g.timeout_ns, &g_fu_error, kErrCompute)) {
          ok = false;
          break;
        }
        if (tid == 0 && it < 8) FU_EV(8 + it);
        // this group's slice of the stage; plane_zero: a pixel of the zero head; data: where pixel (0,0) would be
        const unsigned plane_zero =
            st0 + stage * buf_bytes + group * slice_bytes + static_cast<unsigned>(pi) * g.plane_stride_px * 8u;
        const unsigned data = plane_zero + static_cast<unsigned>(g.head_px - start_px) * 8u;
        // A operand: row j of the band is accumulator j; this slice is columns 2*group, 2*group + 1 of its 8
        unsigned taddr = tmem_base + lane_bits + a_col0 + abuf * a_buf_cols + static_cast<unsigned>(group) * 2u;
        auto emit = [&](const Acc& a) {
          uint2 u;
          // clamping after the rounding equals rounding after the clamp: 0 and 6 are fp16 values.  ReLU6: the
          // lower clamp rides in the conversion, the upper one is a signed 16-bit integer min on the bit
          // patterns (non-negative fp16 values order like integers)
          if (ACT6) {
            u.x = __vmins2(pack_f16x2<true>(a.lo.x, a.lo.y), 0x46004600u);
            u.y = __vmins2(pack_f16x2<true>(a.hi.x, a.hi.y), 0x46004600u);
          } else {
            u.x = pack_f16x2<false>(a.lo.x, a.lo.y);
            u.y = pack_f16x2<false>(a.hi.x, a.hi.y);
            if (g.act_dw != GI_ACT_NONE) {
              u.x = __vmaxs2(u.x, 0u);
              u.y = __vmaxs2(u.y, 0u);
            }
            if (g.act_dw == GI_ACT_RELU6) {
              u.x = __vmins2(u.x, 0x46004600u);
              u.y = __vmins2(u.y, 0x46004600u);
            }
          }
          tmem_st2(taddr, u.x, u.y);
          taddr += kACols;
        };
        unsigned tp[3], step[3];
        const int iy_first = oy0 * stride - pt;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          const int ix = x * stride - g.pl + k;
          const bool v = ix >= 0 && ix < W;
          tp[k] = v ? data + static_cast<unsigned>((iy_first * W + ix) * 8) : plane_zero;
          step[k] = v ? static_cast<unsigned>(W) * 8u : 0u;
        }
        auto next_row = [&]() {  // row -1 lies in the zero head, row H in the zero row behind the image
          uint2 u[3];
#pragma unroll
          for (int k = 0; k < 3; ++k) {
            u[k] = lds64(tp[k]);
            tp[k] += step[k];
          }
          return widen(u);
        };
        if (MODE == 0) {
          Acc a0r, a1r, a2r;
          Row r = next_row();
          a0r = fma_row_from(bias_acc, r, wlo, whi);
          r = next_row();
          fma_row(a0r, r, wlo + 3, whi + 3);
          a1r = fma_row_from(bias_acc, r, wlo, whi);
          // three output rows per trip and no exit inside: a band whose height is not a multiple of three
          // computes up to two rows too many, from stale staged rows into A tiles no MMA reads
#pragma unroll 1
          for (int oy = oy0; oy < oy1; oy += 3) {
            r = next_row();
            fma_row(a0r, r, wlo + 6, whi + 6);
            emit(a0r);
            fma_row(a1r, r, wlo + 3, whi + 3);
            a2r = fma_row_from(bias_acc, r, wlo, whi);
            r = next_row();
            fma_row(a1r, r, wlo + 6, whi + 6);
            emit(a1r);
            fma_row(a2r, r, wlo + 3, whi + 3);
            a0r = fma_row_from(bias_acc, r, wlo, whi);
            r = next_row();
            fma_row(a2r, r, wlo + 6, whi + 6);
            emit(a2r);
            fma_row(a0r, r, wlo + 3, whi + 3);
            a1r = fma_row_from(bias_acc, r, wlo, whi);
          }
        } else {
          Acc carry = fma_row_from(bias_acc, next_row(), wlo, whi);
          for (int oy = oy0; oy < oy1; ++oy) {
            fma_row(carry, next_row(), wlo + 3, whi + 3);
            const Row r2 = next_row();
            fma_row(carry, r2, wlo + 6, whi + 6);
            emit(carry);
            carry = fma_row_from(bias_acc, r2, wlo, whi);
          }
        }
        // the staged rows are consumed: hand the stage back to the copy warp; this warp's part of the
        // chunk is in tensor memory: tell the MMA warp
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&hdr->empty[stage]));
          mbar_arrive(smem_u32(&hdr->a_full[abuf]));
        }
        if (tid == 0 && it < 8) FU_EV(16 + it);
        if (ch == 0 && pend) {
          // the previous tile's accumulators: its MMAs finished while this chunk was computed
          drain();
          if (!ok) break;
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_free));
        }
      }
      if (!ok) break;
      // this tile's accumulators are drained after the next tile's first chunk, when its last MMAs are long done
      pend = true;
      pend_t = t;
    }
    if (ok && pend) drain();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

constexpr size_t kSmemCap = 224 * 1024;
constexpr size_t kSmemAttr = 226 * 1024;

struct FuPlan {
  bool ok = false;
  FuGeom g{};
  int mode = 0;
  size_t smem = 0;
};

FuPlan plan_fused(const LaunchRec& r, int cout, int sms) {
  FuPlan p;
  FuGeom& g = p.g;
  if (r.kh != 3 || r.kw != 3 || r.sh != r.sw || (r.sh != 1 && r.sh != 2) || r.dh != 1 || r.dw != 1) return p;
  if (r.C % 16 != 0 || cout <= 0 || r.pt > 1 || r.pl > 1 || r.pt < 0 || r.pl < 0) return p;
  g.B = r.B;
  g.H = r.H;
  g.W = r.W;
  g.Pin = plane_pixels(r.H, r.W);
  g.Ho = r.Ho;
  g.Wo = r.Wo;
  g.Pout = plane_pixels(r.Ho, r.Wo);
  g.S = r.C / 4;
  g.stride = r.sh;
  g.pt = r.pt;
  g.pl = r.pl;
  // at most one padding row / column behind the image as well
  if ((g.Ho - 1) * g.stride - g.pt + 2 - (g.H - 1) > 1 || (g.Wo - 1) * g.stride - g.pl + 2 - (g.W - 1) > 1) return p;
  g.n_pad = (cout + 15) / 16 * 16;
  g.s_out = slices(cout);
  if (g.n_pad > 256 || g.Wo > 128) return p;
  const size_t fixed = kHeader + static_cast<size_t>(g.S) * g.n_pad * 8 + static_cast<size_t>(g.S) * 160 + static_cast<size_t>(g.n_pad) * 4;
  if (fixed > 150 * 1024) return p;
  g.nb = 128 / g.Wo;
  if (g.nb > g.B) g.nb = g.B;
  g.bchunks = (g.B + g.nb - 1) / g.nb;
  g.head_px = (g.W + 3) & ~1;
  g.tail_px = (g.W + 3) & ~1;
  // rows per tile: bounded by tensor memory (th accumulators of n_pad columns + two A buffers of th x 8)
  int th_cap = kTmemCols / (g.n_pad + 2 * kACols);
  while (th_cap > 0 && th_cap * g.n_pad + 2 * ((th_cap + 2) / 3 * 3) * kACols > kTmemCols) --th_cap;
  const int th_target = g.stride == 1 ? 16 : 8;
  if (th_cap > th_target) th_cap = th_target;
  if (th_cap > g.Ho) th_cap = g.Ho;
  if (th_cap < 1) return p;
  auto stage_bytes = [&](int th) {
    const int rows_in = (th - 1) * g.stride + 3;
    int px = (rows_in < g.H ? rows_in : g.H) * g.W + 2;  // + alignment pixel in front, rounding pixel behind
    if (px > g.Pin) px = g.Pin;
    // (+ two rows of slack: the stride-1 row loop may read up to two rows past the band, results unused)
    g.plane_stride_px = g.head_px + ((px + 1) & ~1) + g.tail_px + 2 * g.W;
    return 4 * static_cast<size_t>(g.plane_stride_px) * 8 * g.nb;  // a stage holds the four slices of a chunk
  };
  // fewest waves of tiles over the SMs first, then the tallest band (fewest halo rows), with at least two stages
  long long best_cost = -1;
  int best_th = 0;
  for (int th = th_cap; th >= 1; --th) {
    if (fixed + 2 * stage_bytes(th) > kSmemCap) continue;
    const long long bands = (g.Ho + th - 1) / th;
    const long long tiles = bands * g.bchunks;
    const long long waves = (tiles + sms - 1) / sms;
    const long long cost = waves * (th * g.stride + 2 + 3);  // rows a CTA reads per slice, plus a fixed cost per chunk
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best_th = th;
    }
  }
  if (best_th == 0) return p;
  g.th = best_th;
  g.bands = (g.Ho + g.th - 1) / g.th;
  const size_t stage = stage_bytes(g.th);
  long long nbuf = static_cast<long long>((kSmemCap - fixed) / stage);
  if (nbuf > kMaxBuf) nbuf = kMaxBuf;
  g.nbuf = static_cast<int>(nbuf);
  p.smem = fixed + stage * g.nbuf;
  const long long tiles = static_cast<long long>(g.bchunks) * g.bands;
  if (tiles > 2147483647LL) return p;
  g.tiles = static_cast<int>(tiles);
  p.mode = g.stride == 1 ? 0 : 1;
  p.ok = true;
  return p;
}

}  // namespace

// The pair can run as one kernel: `dw` holds the depthwise op's geometry, `cout` the 1x1 convolution's
// output channels.  `tiles` receives the number of pixel tiles (the kernel's parallelism), `lanes` how
// many of the 128 rows of an MMA a tile fills.
bool depthwise_pointwise_supported(const LaunchRec& dw, int cout, long long* tiles, int* lanes) {
  const FuPlan p = plan_fused(dw, cout, 148);
  if (tiles) *tiles = p.ok ? p.g.tiles : 0;
  if (lanes) *lanes = p.ok ? p.g.nb * p.g.Wo : 0;
  return p.ok;
}

// 1x1 weights as the resident B operand: [C/8 K units][n_pad rows][8 halves]; bias padded to n_pad.
// Behind the bias: a zero-filled region of one image row (+ 3 pixels), the source of the zero row staged below an image.
void depthwise_pointwise_pack(const float* w, const float* bias, int cin, int cout, int width, std::vector<uint8_t>* blob,
                              LaunchRec* r) {
  const int n_pad = (cout + 15) / 16 * 16;
  const size_t wbytes = static_cast<size_t>(cin / 8) * n_pad * 16;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(n_pad) * sizeof(float) + static_cast<size_t>((width + 3) & ~1) * 8, 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) {
    bp[co] = bias[co];
    for (int ci = 0; ci < cin; ++ci)
      wp[(static_cast<size_t>(ci / 8) * n_pad + co) * 8 + ci % 8] = f32_to_f16_rne(w[static_cast<size_t>(co) * cin + ci]);
  }
  r->wts2 = Loc{W_WEIGHTS, 0, woff};
  r->bias2 = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes += wbytes;
}

int launch_depthwise_pointwise(const LaunchRec& r, const Ptrs& p, void* stream) {
  const int sms = device_sm_count();
  FuPlan pl = plan_fused(r, r.Co2, sms);
  if (!pl.ok) return static_cast<int>(cudaErrorInvalidConfiguration);
  FuGeom& g = pl.g;
  g.act_dw = r.ep.act_pre;
  g.act_pre = r.ep2.act_pre;
  g.has_res = r.ep2.has_res;
  g.act_post = r.ep2.act_post;
  g.in_dead = r.in0_dead;
  g.timeout_ns = 1000000000u;
  static bool attr_dev[kMaxDevices] = {};
  bool& attr_set = attr_dev[current_device_slot()];
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    void (*const kernels[4])(const __half*, const float*, const float*, const unsigned char*, const float*, const __half*, __half*,
                             const FuGeom) = {depthwise_pointwise_kernel<0, false>, depthwise_pointwise_kernel<0, true>,
                                              depthwise_pointwise_kernel<1, false>, depthwise_pointwise_kernel<1, true>};
    for (int m = 0; m < 4 && e == cudaSuccess; ++m)
      e = cudaFuncSetAttribute(kernels[m], cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemAttr));
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  long long grid = sms;
  if (grid > g.tiles) grid = g.tiles;
  // the kernel reserves all of tensor memory, so exactly one CTA may live on an SM: ask for enough
  // shared memory that a second one cannot be co-resident
  size_t smem = pl.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* in = static_cast<const __half*>(p.in0);
  const float* w = static_cast<const float*>(p.wts);
  const float* b = static_cast<const float*>(p.bias);
  const unsigned char* w2 = static_cast<const unsigned char*>(p.wts2);
  const float* b2 = static_cast<const float*>(p.bias2);
  const __half* res = static_cast<const __half*>(p.res);
  __half* out = static_cast<__half*>(p.out);
  const bool act6 = g.act_dw == GI_ACT_RELU6;
#define GI_FU_LAUNCH(M, A) \
  launch_pdl(depthwise_pointwise_kernel<M, A>, static_cast<unsigned>(grid), kThreads, smem, st, in, w, b, w2, b2, res, out, g)
  if (pl.mode == 0) {
    if (act6) GI_FU_LAUNCH(0, true);
    else GI_FU_LAUNCH(0, false);
  } else {
    if (act6) GI_FU_LAUNCH(1, true);
    else GI_FU_LAUNCH(1, false);
  }
#undef GI_FU_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

unsigned int depthwise_pointwise_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_fu_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

#ifdef GI_TRACE
int depthwise_pointwise_trace(unsigned long long* dst, int n) {
  const size_t bytes = sizeof(unsigned long long) * (n < 1024 * 64 ? n : 1024 * 64);
  return static_cast<int>(cudaMemcpyFromSymbol(dst, g_fu_trace, bytes));
}
#endif

}  // namespace gi
