// Pointwise (1x1) convolution, second tensor-core variant: weights stationary in shared memory,
// the activation operand in TENSOR MEMORY (tcgen05.mma with A in TMEM).
//
// A pixel-slice is 4 fp16 = two 32-bit words, and a TMEM lane holds the K axis of an fp16 A
// operand two elements per 32-bit column - so "lane = pixel, columns 2s, 2s+1 = slice s" IS the
// operand layout, with nothing padded or duplicated: the tensor pipe does exactly 2*M*N*K flops
// and the weight operand is the dense [Cout][Cin] matrix, small enough to stay in shared memory
// for the whole kernel (each CTA keeps the rows of its share of the output channels).  What
// streams is the activation only: TMA boxes of 128 pixels x ks slices land in a ring of shared
// memory stages, eight transfer warps move a stage into tensor memory (8-byte ld.shared per lane,
// tcgen05.st), and every byte of shared memory that is not weights is activation in flight -
// which is what a layer bound by HBM latency x bandwidth needs.  The pixel-pair variant
// (pointwise_tc.cu) keeps the layers with few input channels and large planes; this one takes
// the layers where that variant's 4x expanded weight tile crowded the activations out of shared
// memory.
//
// CTA = 26 warps: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-9 transfer
// (two per TMEM lane quarter, taking alternate groups of 8 slices: with deep inputs and a single tile per CTA - batch 1 - the
// transfer of K through four warps was a third of a launch; MobileNetV2 batch 1 0.240 -> 0.2375 ms, 0.2215 -> 0.218 ms as a
// CUDA graph), warps 10-25 drain the accumulator (four per quarter: bias,
// activation, residual, fp16 pack, 8-byte stores, 256 contiguous bytes per warp).  Accumulators
// and A chunks are double-buffered in the 512 TMEM columns.  If a CTA's weight share does not
// fit, the weights stream through the same stages instead.  All waits are bounded.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.h"
#include "trace.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kRows = 128;
constexpr int kTransferWarps = 8;  // two per TMEM lane quarter: each moves every other group of 8 slices of a chunk
constexpr int kDrainWarps = 16;
constexpr int kThreads = 32 * (2 + kTransferWarps + kDrainWarps);
constexpr int kMaxStages = 8;
constexpr int kSmemHeader = 1024;
constexpr int kSmemBudget = 208 * 1024;        // stages + resident weights
constexpr int kResidentLimit = 144 * 1024;     // weights larger than this stream through the stages
constexpr int kMaxNcta = 192;

__device__ unsigned int g_ts_error = 0;
GI_TRACE_TABLE(g_ts_trace);

struct TsParams {
  const __half* res;
  __half* out;
  const float* bias;
  const unsigned char* wts;
  unsigned int m_total_px;
  int s_out;
  int ks, n_chunks;      // input slices per A chunk (multiple of 8), chunks per pixel tile
  int n_cta, n_parts;    // output channels per CTA (multiple of 16), CTAs sharing one pixel tile
  int b_resident;        // 1: the CTA's weights are loaded once; 0: a weight chunk rides in every stage
  int stages;
  int m_tiles;
  int box_px;            // pixels per TMA box: 128, or 64 / 32 when the whole layer has no more (the rest of the tile is never fetched)
  int has_res, act_post;
  int in_dead;           // the input is not read again: its TMA loads carry the evict-first L2 hint
  unsigned int timeout_ns;
};

struct Header {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long a_full[2];
  unsigned long long a_empty[2];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned long long b_ready;
  unsigned tmem_addr;
  unsigned abort_flag;
};
constexpr int kBiasOffset = 256;  // the CTA's bias values (at most kMaxNcta floats) follow the barriers in the header
static_assert(sizeof(Header) <= kBiasOffset && kBiasOffset + kMaxNcta * sizeof(float) <= kSmemHeader, "header too large");

__device__ __forceinline__ void tmem_st16(unsigned taddr, const unsigned* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint2 lds64(unsigned addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

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

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

enum : unsigned { kErrProducer = 1u, kErrMma = 2u, kErrData = 4u, kErrDrain = 8u };

// ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow
template <int ACT, bool TAIL>
__global__ void __launch_bounds__(kThreads, 1) pointwise_ts_kernel(const __grid_constant__ CUtensorMap tmap_a, const TsParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned slice_bytes = static_cast<unsigned>(p.box_px) * 8u;              // one slice of a box: box_px pixels x 8 bytes
  const unsigned a_stage_bytes = static_cast<unsigned>(p.ks) * slice_bytes;       // ks slices
  const unsigned b_chunk_bytes = static_cast<unsigned>(p.ks) * p.n_cta * 8u;      // ks/2 K units x n_cta rows x 16 bytes
  const unsigned stage_bytes = a_stage_bytes + (p.b_resident ? 0u : b_chunk_bytes);
  const unsigned b_res_bytes = p.b_resident ? b_chunk_bytes * p.n_chunks : 0u;
  const unsigned b_res0 = smem_u32(smem + kSmemHeader);                          // resident weights first
  const unsigned stage0 = b_res0 + b_res_bytes;
  const unsigned a_cols = static_cast<unsigned>(p.ks) * 2u, acc_cols = static_cast<unsigned>(p.n_cta);
  const unsigned a_col0 = 2u * acc_cols;  // TMEM columns: two accumulators, then two A chunk buffers

  // this CTA's share of the output channels is fixed; it walks over pixel tiles
  const int n_part = blockIdx.x % p.n_parts;
  const int m_first = blockIdx.x / p.n_parts, m_step = gridDim.x / p.n_parts;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_a);
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->full[i]), 1);
      mbar_init(smem_u32(&hdr->empty[i]), kTransferWarps + (p.b_resident ? 0 : 1));
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kTransferWarps);
      mbar_init(smem_u32(&hdr->a_empty[i]), 1);
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), kDrainWarps);
    }
    mbar_init(smem_u32(&hdr->b_ready), 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), 512u);
  // this CTA's bias (its output channels are the same for every tile) in shared memory, behind the barriers: the
  // epilogue reads it per slice, and a load from global memory there queues behind everything the SM has in flight
  float* bias_s = reinterpret_cast<float*>(smem + kBiasOffset);
  for (int i = threadIdx.x; i < p.n_cta; i += kThreads) bias_s[i] = __ldg(p.bias + n_part * p.n_cta + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  const unsigned char* w_part = p.wts + static_cast<size_t>(n_part) * p.n_chunks * b_chunk_bytes;
  if (threadIdx.x == 0) GI_TRACE_EVENT(g_ts_trace, 0);
  pdl_launch_dependents();
  // the weights never change after binding: their copy starts while the previous kernel still runs
  if (warp == 0 && lane == 0 && p.b_resident) {
    const unsigned bar = smem_u32(&hdr->b_ready);
    mbar_expect_tx(bar, b_res_bytes);
    for (int c = 0; c < p.n_chunks; ++c)
      bulk_load(b_res0 + c * b_chunk_bytes, w_part + static_cast<size_t>(c) * b_chunk_bytes, b_chunk_bytes, bar);
  }
  pdl_wait();  // activations are read and written only below
  if (threadIdx.x == 0) GI_TRACE_EVENT(g_ts_trace, 1);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      const unsigned long long evict_first = policy_evict_first();
      for (int m = m_first; m < p.m_tiles && ok; m += m_step) {
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
          if (!mbar_wait(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrProducer)) {
            ok = false;
            break;
          }
          const unsigned full = smem_u32(&hdr->full[stage]);
          mbar_expect_tx(full, stage_bytes);
          const unsigned dst = stage0 + stage * stage_bytes;
          // pixels / slices outside the tensor arrive as zeros
          if (p.in_dead) tma_load_2d_hint(dst, &tmap_a, m * kRows, c * p.ks, full, evict_first);
          else tma_load_2d(dst, &tmap_a, m * kRows, c * p.ks, full);
          if (it == 0) GI_TRACE_EVENT(g_ts_trace, 2);
          if (!p.b_resident) bulk_load(dst + a_stage_bytes, w_part + static_cast<size_t>(c) * b_chunk_bytes, b_chunk_bytes, full);
        }
      }
      if (!ok) {
        const unsigned first = it > static_cast<unsigned>(p.stages) ? it - p.stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->full[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_ts_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, B K-major, M = 128, N = n_cta
      const unsigned idesc = (1u << 4) | ((acc_cols >> 3) << 17) | ((kRows >> 4) << 24);
      const unsigned b_lbo = acc_cols * 16u;  // distance between consecutive 8-element K units of the weight tile
      unsigned it = 0, tile = 0;
      bool ok = true;
      if (p.b_resident) ok = mbar_wait(smem_u32(&hdr->b_ready), 0u, abort_flag, p.timeout_ns, &g_ts_error, kErrMma);
      GI_TRACE_EVENT(g_ts_trace, 3);
      for (int m = m_first; m < p.m_tiles && ok; m += m_step, ++tile) {
        const unsigned acc = tile & 1u, acc_phase = (tile >> 1) & 1u;
        if (!mbar_wait(smem_u32(&hdr->acc_empty[acc]), acc_phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrMma)) break;
        const unsigned d_tmem = tmem_base + acc * acc_cols;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, s_phase = (it / p.stages) & 1u;
          const unsigned abuf = it & 1u, a_phase = (it >> 1) & 1u;
          if (!p.b_resident && !mbar_wait(smem_u32(&hdr->full[stage]), s_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrMma)) {
            ok = false;
            break;
          }
          if (!mbar_wait(smem_u32(&hdr->a_full[abuf]), a_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrMma)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (it == 0) GI_TRACE_EVENT(g_ts_trace, 4);
          const unsigned a_tmem = tmem_base + a_col0 + abuf * a_cols;
          const unsigned b_base = p.b_resident ? b_res0 + c * b_chunk_bytes : stage0 + stage * stage_bytes + a_stage_bytes;
          // 16 channels = 4 slices = 8 TMEM columns = 2 K units per MMA.  The issuing thread's own
          // instructions bound the tensor-heavy layers, so the descriptor is built once per chunk and
          // advanced by an add (the address field counts 16-byte units and cannot carry out of its 14 bits)
          unsigned long long bd = smem_desc(b_base, b_lbo, 128);
          const unsigned long long bd_step = static_cast<unsigned long long>((2u * b_lbo) >> 4);
          const int n_mma = p.ks / 4;
          umma_f16_ts(d_tmem, a_tmem, bd, idesc, c > 0 ? 1u : 0u);
          for (int ks = 1; ks < n_mma; ++ks) {
            bd += bd_step;
            umma_f16_ts(d_tmem, a_tmem + ks * 8, bd, idesc, 1u);
          }
          umma_commit(smem_u32(&hdr->a_empty[abuf]));
          if (!p.b_resident) umma_commit(smem_u32(&hdr->empty[stage]));
        }
        if (ok) umma_commit(smem_u32(&hdr->acc_full[acc]));
        if (tile == 0) GI_TRACE_EVENT(g_ts_trace, 5);
      }
      GI_TRACE_EVENT(g_ts_trace, 9);
    }
  } else if (warp < 2 + kTransferWarps) {
    // ------------------------------------------------------------ transfer: shared memory -> tensor memory
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, +32)
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const unsigned row_off = static_cast<unsigned>(quarter * 32 + lane) * 8u;
    const int part = (warp - 2) >> 2;  // which of the quarter's two transfer warps
    unsigned it = 0;
    bool ok = true;
    for (int m = m_first; m < p.m_tiles && ok; m += m_step) {
      for (int c = 0; c < p.n_chunks; ++c, ++it) {
        const unsigned stage = it % p.stages, s_phase = (it / p.stages) & 1u;
        const unsigned abuf = it & 1u, a_phase = (it >> 1) & 1u;
        if (!mbar_wait_warp(smem_u32(&hdr->full[stage]), s_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrData) ||
            !mbar_wait_warp(smem_u32(&hdr->a_empty[abuf]), a_phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrData)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const unsigned src = stage0 + stage * stage_bytes + row_off;
        const unsigned t_addr = tmem_base + lane_bits + a_col0 + abuf * a_cols;
        // a box narrower than 128 pixels leaves the upper lane quarters without data: their rows of the
        // accumulator are never stored, so their lanes of the A operand may hold anything
        for (int j = 8 * part; j < p.ks && quarter * 32 < p.box_px; j += 8 * (kTransferWarps / 4)) {
          unsigned r[16];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const uint2 v = lds64(src + static_cast<unsigned>(j + q) * slice_bytes);
            r[2 * q] = v.x;
            r[2 * q + 1] = v.y;
          }
          tmem_st16(t_addr + j * 2, r);
        }
        // the stage's activations are in registers / on their way to tensor memory: release it
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[stage]));
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->a_full[abuf]));
      }
    }
  } else {
    // ------------------------------------------------------------ drain: accumulator -> global memory
    const int quarter = warp & 3;
    constexpr int kParts = kDrainWarps / 4;                     // warps sharing one lane quarter
    const int part_id = (warp - (2 + kTransferWarps)) >> 2;     // takes every kParts-th 16-column group
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int groups = p.n_cta >> 4;
    unsigned tile = 0;
    for (int m = m_first; m < p.m_tiles; m += m_step, ++tile) {
      const unsigned acc = tile & 1u, acc_phase = (tile >> 1) & 1u;
      const unsigned pixel = static_cast<unsigned>(m) * kRows + quarter * 32 + lane;
      const bool px_ok = pixel < p.m_total_px;
      // the residual does not depend on the accumulator: the first group's is fetched before waiting
      // for the MMAs, each further group's while the one before it is processed
      auto fetch_res = [&](uint2* q, int g) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int so = (n_part * p.n_cta) / 4 + g * 4 + j;
          q[j] = make_uint2(0u, 0u);
          if (p.has_res && g < groups && so < p.s_out && px_ok)
            q[j] = __ldg(reinterpret_cast<const uint2*>(p.res + (static_cast<size_t>(so) * p.m_total_px + pixel) * 4));
        }
      };
      uint2 res_cur[4], res_next[4];
      if (TAIL) fetch_res(res_cur, part_id);
      if (!mbar_wait_warp(smem_u32(&hdr->acc_full[acc]), acc_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrData)) break;
      tc_fence_after();
      if (tile == 0 && threadIdx.x == 32 * (2 + kTransferWarps)) GI_TRACE_EVENT(g_ts_trace, 6);
      const unsigned t_addr = tmem_base + lane_bits + acc * acc_cols;
      for (int g = part_id; g < groups; g += kParts) {
        if (TAIL) fetch_res(res_next, g + kParts);
        unsigned r[16];
        tmem_ld16(t_addr + g * 16, r);
        tmem_ld_wait16(r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int so = (n_part * p.n_cta) / 4 + g * 4 + j;
          if (so >= p.s_out || !px_ok) continue;
          const float4 b = *reinterpret_cast<const float4*>(bias_s + g * 16 + 4 * j);
          const size_t off = (static_cast<size_t>(so) * p.m_total_px + pixel) * 4;  // in halves
          const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1])), make_float2(b.x, b.y));
          const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])), make_float2(b.z, b.w));
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
            const uint2 q = res_cur[j];
            const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
            const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
            // the usual tail is the residual sum of a linear projection: no activation on either side of it
            float2 s0 = __fadd2_rn(make_float2(act1(v0.x, ACT), act1(v0.y, ACT)), r0);
            float2 s1 = __fadd2_rn(make_float2(act1(v1.x, ACT), act1(v1.y, ACT)), r1);
            if (p.act_post != GI_ACT_NONE) {
              s0 = make_float2(act1(s0.x, p.act_post), act1(s0.y, p.act_post));
              s1 = make_float2(act1(s1.x, p.act_post), act1(s1.y, p.act_post));
            }
            h0 = __floats2half2_rn(s0.x, s0.y);
            h1 = __floats2half2_rn(s1.x, s1.y);
          }
          uint2 o;
          o.x = *reinterpret_cast<const unsigned*>(&h0);
          o.y = *reinterpret_cast<const unsigned*>(&h1);
          *reinterpret_cast<uint2*>(p.out + off) = o;
        }
        if (TAIL) {
#pragma unroll
          for (int j = 0; j < 4; ++j) res_cur[j] = res_next[j];
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[acc]));
    }
    if (threadIdx.x == 32 * (2 + kTransferWarps)) GI_TRACE_EVENT(g_ts_trace, 7);
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) GI_TRACE_EVENT(g_ts_trace, 8);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

struct Tiling {
  int s_in, s_out, ks, n_chunks, n_cta, n_parts, b_resident, stages, box_px;
  size_t smem;
};

// `m_px`: pixels of the layer (batch x H x W; 0 = unknown).  A layer with few pixel tiles - batch 1, or the
// classifier behind the global pool - is a handful of CTAs that each stream a wide share of the weights from
// L2: there the output channels are split into narrower shares (down to 32 channels) until every SM
// takes part (measured: better than half of them, and than 16- or 48-channel shares), so that the weights arrive
// through many SMs at once.
Tiling choose_tiling(int cin, int cout, long long m_px) {
  Tiling t;
  t.s_in = slices(cin);
  t.s_out = slices(cout);
  const int n_pad = (cout + 15) / 16 * 16;
  t.n_parts = (n_pad + kMaxNcta - 1) / kMaxNcta;
  // a layer of at most 64 (32) pixels is fetched in boxes of 64 (32) pixels: less zero fill in shared memory,
  // fewer lanes to move into tensor memory, and room for twice (four times) the slices per chunk
  t.box_px = m_px > 0 && m_px <= 32 ? 32 : m_px > 0 && m_px <= 64 ? 64 : kRows;
  const int slice_bytes = t.box_px * 8;
  if (m_px > 0) {
    const long long m_tiles = (m_px + kRows - 1) / kRows;
    while (m_tiles * t.n_parts < 148 && ((n_pad + t.n_parts - 1) / t.n_parts + 15) / 16 * 16 > 32) ++t.n_parts;
    const int n_cta = ((n_pad + t.n_parts - 1) / t.n_parts + 15) / 16 * 16;
    t.n_parts = (n_pad + n_cta - 1) / n_cta;  // no share left empty by the rounding to 16 channels
  }
  const int s_pad = (t.s_in + 7) / 8 * 8;
  for (;; ++t.n_parts) {
    t.n_cta = ((n_pad + t.n_parts - 1) / t.n_parts + 15) / 16 * 16;
    // TMEM: 2 accumulators of n_cta columns + 2 A buffers of 2*ks columns <= 512
    int ks_max = (512 - 2 * t.n_cta) / 4 / 8 * 8;
    if (ks_max > 64 * (kRows / t.box_px)) ks_max = 64 * (kRows / t.box_px);
    t.n_chunks = (s_pad + ks_max - 1) / ks_max;
    t.ks = ((s_pad + t.n_chunks - 1) / t.n_chunks + 7) / 8 * 8;
    const size_t b_all = static_cast<size_t>(t.n_chunks) * t.ks * t.n_cta * 8;
    // prefer resident weights: split the output channels over more CTAs while that gets there and
    // the share stays at least 64 channels wide
    t.b_resident = b_all <= static_cast<size_t>(kResidentLimit);
    if (t.b_resident || t.n_cta <= 64) break;
  }
  // two activation stages must fit beside the weights: shrink the chunk if they do not
  for (;;) {
    const size_t bc = static_cast<size_t>(t.ks) * t.n_cta * 8;
    const size_t res = t.b_resident ? bc * t.n_chunks : 0;
    const size_t st = static_cast<size_t>(t.ks) * slice_bytes + (t.b_resident ? 0 : bc);
    if (t.ks <= 8 || res + 2 * st <= static_cast<size_t>(kSmemBudget)) break;
    t.ks = (t.ks / 2 + 7) / 8 * 8;
    t.n_chunks = (s_pad + t.ks - 1) / t.ks;
  }
  const size_t b_chunk = static_cast<size_t>(t.ks) * t.n_cta * 8;
  const size_t resident = t.b_resident ? b_chunk * t.n_chunks : 0;
  const size_t stage = static_cast<size_t>(t.ks) * slice_bytes + (t.b_resident ? 0 : b_chunk);
  long long stages = (static_cast<long long>(kSmemBudget) - static_cast<long long>(resident)) / static_cast<long long>(stage);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) stages = 2;
  t.stages = static_cast<int>(stages);
  t.smem = kSmemHeader + resident + stage * t.stages;
  return t;
}

}  // namespace

bool pointwise_ts_supported(int cin, int cout) {
  if (cin <= 0 || cout <= 0) return false;
  return choose_tiling(cin, cout, 0).smem <= static_cast<size_t>(kSmemHeader + kSmemBudget + 16 * 1024);
}

// Dense weights as the B operand, per (CTA share, K chunk): [ks/2 K units][n_cta rows][8 halves].
void pointwise_ts_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Tiling t = choose_tiling(cin, cout, static_cast<long long>(r->B) * plane_pixels(r->H, r->W));
  const size_t chunk_bytes = static_cast<size_t>(t.ks) * t.n_cta * 8;
  const size_t wbytes = static_cast<size_t>(t.n_parts) * t.n_chunks * chunk_bytes;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(t.n_parts) * t.n_cta * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) {
    const int part = co / t.n_cta, row = co % t.n_cta;
    bp[co] = bias[co];
    for (int ci = 0; ci < cin; ++ci) {
      const int chunk = ci / (t.ks * 4), k = ci % (t.ks * 4);
      uint16_t* base = wp + (static_cast<size_t>(part) * t.n_chunks + chunk) * (chunk_bytes / 2);
      base[(static_cast<size_t>(k / 8) * t.n_cta + row) * 8 + k % 8] = f32_to_f16_rne(w[static_cast<size_t>(co) * cin + ci]);
    }
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = t.n_cta;
  r->tc_kc = t.ks;
  r->tc_stages = t.stages;
}

int launch_pointwise_ts(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream) {
  const Tiling t = choose_tiling(r.C, r.Co, static_cast<long long>(r.B) * plane_pixels(r.H, r.W));
  TsParams k;
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.bias = static_cast<const float*>(p.bias);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.m_total_px = static_cast<unsigned>(r.B) * static_cast<unsigned>(plane_pixels(r.H, r.W));
  k.s_out = t.s_out;
  k.ks = t.ks;
  k.n_chunks = t.n_chunks;
  k.n_cta = t.n_cta;
  k.n_parts = t.n_parts;
  k.b_resident = t.b_resident;
  k.stages = t.stages;
  k.m_tiles = static_cast<int>((k.m_total_px + kRows - 1) / kRows);
  k.box_px = t.box_px;
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  k.in_dead = r.in0_dead;
  k.timeout_ns = 1000000000u;
  static bool attr_set_dev[kMaxDevices] = {};
  bool& attr_set = attr_set_dev[current_device_slot()];
  const int sms = device_sm_count();
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    const int bytes = kSmemHeader + kSmemBudget + 16 * 1024;
#define GI_TS_ATTR(A, T) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(pointwise_ts_kernel<A, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)
    GI_TS_ATTR(GI_ACT_NONE, false);
    GI_TS_ATTR(GI_ACT_RELU, false);
    GI_TS_ATTR(GI_ACT_RELU6, false);
    GI_TS_ATTR(GI_ACT_NONE, true);
    GI_TS_ATTR(GI_ACT_RELU, true);
    GI_TS_ATTR(GI_ACT_RELU6, true);
#undef GI_TS_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  CUtensorMap tmap;
  {
    const int err = map_cache_lookup(state, launch_index, p.in0, &tmap, [&](CUtensorMap* m) {
      return encode_plane_map(m, p.in0, k.m_total_px, t.s_in, t.box_px, t.ks);
    });
    if (err != 0) return err;
  }
  // CTAs come in groups of n_parts (one per share of the output channels) that walk the pixel tiles together
  long long groups = sms / t.n_parts;
  if (groups < 1) groups = 1;
  if (groups > k.m_tiles) groups = k.m_tiles;
  const unsigned grid = static_cast<unsigned>(groups * t.n_parts);
  // the kernel reserves all of tensor memory, so exactly one CTA may live on an SM: ask for enough
  // shared memory that a second one cannot be co-resident
  size_t smem = t.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
  const int act = r.ep.act_pre;
#define GI_TS_LAUNCH(A, T) launch_pdl(pointwise_ts_kernel<A, T>, grid, kThreads, smem, cu_stream, tmap, k)
  if (tail) {
    if (act == GI_ACT_RELU6) GI_TS_LAUNCH(GI_ACT_RELU6, true);
    else if (act == GI_ACT_RELU) GI_TS_LAUNCH(GI_ACT_RELU, true);
    else GI_TS_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (act == GI_ACT_RELU6) GI_TS_LAUNCH(GI_ACT_RELU6, false);
    else if (act == GI_ACT_RELU) GI_TS_LAUNCH(GI_ACT_RELU, false);
    else GI_TS_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_TS_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

#ifdef GI_TRACE
int pointwise_ts_trace(unsigned long long* dst, int n) {
  const size_t bytes = sizeof(unsigned long long) * (n < GI_TRACE_CTAS * GI_TRACE_EVENTS ? n : GI_TRACE_CTAS * GI_TRACE_EVENTS);
  return static_cast<int>(cudaMemcpyFromSymbol(dst, g_ts_trace, bytes));
}
#endif

unsigned int pointwise_ts_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_ts_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
