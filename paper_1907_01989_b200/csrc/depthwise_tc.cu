// Depthwise 3x3 convolution (fp16 storage, even planes) with the multiply-accumulates on the
// tensor cores.
//
// The CUDA-core stencil (depthwise.cu) is bound by the fp16 -> fp32 widening and the FMAs of
// its 9 taps, not by memory.  Here the tensor pipe does both.  Two adjacent pixels of a slice
// are 16 bytes = one K-major operand row of 8 fp16 (pixel parity x 4 channels); a small 16 x 8
// weight block maps the 8 inputs of a pair to the outputs of a pair (diagonal in the channel,
// one tap per pixel-parity combination).  Neighbouring pairs and rows are the SAME bytes read
// at a shifted start address, so the whole 3x3 window becomes a handful of 128 x 16 x 16 MMAs
// whose A operands are shifted views of one staged tile - nothing is gathered or copied.
//
//   staging   TMA, 4-D map (x, row parity, row / 2, plane), box = (W + 4 pixels, 1, rows, planes):
//             even and odd input rows land in two regions with the same pitch; the two zero
//             pixels left and right of every row and the rows above / below the image are the
//             TMA's out-of-bounds fill.  A lane of the MMA tile is one pair position of the
//             padded rows, lanes run linearly through a region, so a tap at (dy, dx) is the
//             region read (dy * pitch + dx) pairs further on.
//   stride 1  a lane produces the pair at output rows 2r and 2r+1 (16 accumulator columns):
//             4 input rows x 3 pair shifts = 12 K-chunks of 8 -> 6 MMAs per 128 lanes
//   stride 2  a lane produces output pixel (r, c) (4 accumulator columns): 3 rows x 2 pair
//             shifts -> 3 MMAs per 128 lanes
//   epilogue  8 warps read the fp32 accumulators (tcgen05.ld), add the bias, apply the fused
//             tail and store 16 (8) contiguous bytes per lane.
//
// CTAs are persistent over a contiguous range of work items (a band of rows of one plane, or a
// few whole small planes); warp 0 produces, warp 1 issues the MMAs, the accumulators form a ring
// of 8 in tensor memory.  All waits are bounded.
//
// Measured on B200: correct, but SLOWER than the stencil (0.158 vs 0.101 ms for 112x112x32,
// batch 256, stride 1; 0.33 vs 0.15 ms for 112x112x96 stride 2).  One SM accepts a tcgen05.mma
// or tcgen05.commit only every ~47 cycles whatever its size up to N = 64, so the 7 (4)
// instructions a 128-lane tile needs already cost as much as the tile's HBM time, and the
// commit -> wait -> commit chain of the issuing thread adds ~400 cycles per tile.  The kernel
// therefore runs only on request (GI_DW_TC); the default stays the stencil.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace gi {
namespace {

using namespace ptx;

constexpr int kRows = 128;          // lanes per MMA tile
constexpr int kMaxInstr = 8;
constexpr int kAcc = 8;             // accumulator ring
constexpr int kAccCols = 16;
constexpr int kMaxStages = 4;
constexpr int kEpiSets = 2;         // epilogue warp sets (4 warps each) taking alternate tiles
constexpr int kThreads = 64 + 128 * kEpiSets;
constexpr int kBTile = 512;         // one 16 x 16 fp16 weight tile
constexpr int kHeader = 1024;
constexpr int kLead = 128;          // readable bytes in front of the first stage (lane 0, shift -1)
constexpr int kRegionTarget = 14 * 1024;
constexpr int kSmemPerCta = 100 * 1024;

__device__ unsigned int g_dwtc_error = 0;

struct DtParams {
  const __half* res;
  __half* out;
  const float* bias;
  const unsigned char* wts;
  int B, W, Pout;
  int PW;          // pairs per staged row: W / 2 + 2
  int half_w;      // valid pairs per row
  int RB, RPP;     // lane rows per band; staged rows per plane and parity (RB + 1)
  int NP;          // planes per item
  int bands, pchunks, items;
  int rows_total;  // lane rows per plane: H / 2 (stride 1, a lane row = two output rows) or Ho (stride 2)
  int first_e, first_o;  // first staged row (in units of two image rows) relative to the band start
  int n_instr;
  int a_off[kMaxInstr];      // byte offset, from the stage start, of lane 0's first K-chunk
  unsigned lbo[kMaxInstr];   // byte distance to the second K-chunk
  unsigned region_stride;    // bytes between the even-row and the odd-row region
  unsigned region_bytes;     // bytes one TMA box delivers
  unsigned b_bytes;          // n_instr weight tiles
  unsigned stage_bytes;
  int stages;
  unsigned magic_pw, magic_rpp;  // floor(2^32 / d) + 1: n / d == umulhi(n, magic) for the small n used here
  int out_row_px;                // pixels per output row
  int out_plane_real;            // Ho * Wo
  int has_res, act_post;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long acc_full[kAcc];
  unsigned long long acc_empty[kAcc];
  int held[kMaxStages];  // slice whose weight tiles a stage holds (producer only)
  unsigned tmem_addr;
  unsigned abort_flag;
};
static_assert(sizeof(Header) <= kHeader, "header too large");

enum : unsigned { kErrProducer = 1u, kErrMma = 2u, kErrEpilogue = 4u, kErrDrain = 8u };

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_ld4(unsigned taddr, unsigned* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait4(unsigned* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]) : : "memory");
}

// work items are numbered band-fastest, then plane chunk, then slice
struct Item {
  int s, pc, band;
};
__device__ __forceinline__ Item item_decode(int idx, const DtParams& p) {
  Item it;
  it.band = idx % p.bands;
  const int rest = idx / p.bands;
  it.pc = rest % p.pchunks;
  it.s = rest / p.pchunks;
  return it;
}
__device__ __forceinline__ void item_advance(Item& it, const DtParams& p) {
  if (++it.band == p.bands) {
    it.band = 0;
    if (++it.pc == p.pchunks) {
      it.pc = 0;
      ++it.s;
    }
  }
}
// tiles of 128 lanes that hold at least one valid lane
__device__ __forceinline__ int item_tiles(const Item& it, const DtParams& p, int& nbk, int& rows_valid) {
  nbk = min(p.NP, p.B - it.pc * p.NP);
  rows_valid = min(p.RB, p.rows_total - it.band * p.RB);
  const int lanes = ((nbk - 1) * p.RPP + rows_valid) * p.PW;
  return (lanes + kRows - 1) / kRows;
}

// one pixel (4 channels): bias, fused tail, fp16
template <int ACT, bool TAIL>
__device__ __forceinline__ uint2 finish_px(const unsigned* r, float2 blo, float2 bhi, uint2 resq, int act_post) {
  const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[0]), __uint_as_float(r[1])), blo);
  const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[2]), __uint_as_float(r[3])), bhi);
  __half2 h0, h1;
  if (!TAIL) {
    // clamping after the rounding equals rounding after the clamp: 0 and 6 are fp16 values
    h0 = __floats2half2_rn(v0.x, v0.y);
    h1 = __floats2half2_rn(v1.x, v1.y);
    if (ACT != GI_ACT_NONE) {
      h0 = __hmax2(h0, __float2half2_rn(0.f));
      h1 = __hmax2(h1, __float2half2_rn(0.f));
    }
    if (ACT == GI_ACT_RELU6) {
      h0 = __hmin2(h0, __float2half2_rn(6.f));
      h1 = __hmin2(h1, __float2half2_rn(6.f));
    }
  } else {
    const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&resq.x));  // zero when there is no residual
    const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&resq.y));
    h0 = __floats2half2_rn(act1(act1(v0.x, ACT) + r0.x, act_post), act1(act1(v0.y, ACT) + r0.y, act_post));
    h1 = __floats2half2_rn(act1(act1(v1.x, ACT) + r1.x, act_post), act1(act1(v1.y, ACT) + r1.y, act_post));
  }
  uint2 o;
  o.x = *reinterpret_cast<const unsigned*>(&h0);
  o.y = *reinterpret_cast<const unsigned*>(&h1);
  return o;
}

// STRIDE 1 or 2; ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow
template <int STRIDE, int ACT, bool TAIL>
__global__ void __launch_bounds__(kThreads, 2) depthwise_tc_kernel(const __grid_constant__ CUtensorMap tmap, const DtParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned data0 = smem_u32(smem + kHeader + kLead);

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap);
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->full[i]), 1);
      mbar_init(smem_u32(&hdr->empty[i]), 1);
      hdr->held[i] = -1;
    }
    for (int i = 0; i < kAcc; ++i) {
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), 4);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), kAcc * kAccCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // the prologue above touched only on-chip state; activations are read and written after the wait
  pdl_launch_dependents();
  pdl_wait();
  const unsigned tmem_base = hdr->tmem_addr;

  // contiguous, balanced range of work items for this CTA: items of one slice stay together
  const int per = p.items / gridDim.x, extra = p.items % gridDim.x;
  const int first = blockIdx.x * per + min(static_cast<int>(blockIdx.x), extra);
  const int count = per + (static_cast<int>(blockIdx.x) < extra ? 1 : 0);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      Item it = item_decode(first, p);
      int n = 0;
      bool ok = true;
      for (; n < count; ++n, item_advance(it, p)) {
        const unsigned stage = n % p.stages, phase = (n / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_dwtc_error, kErrProducer)) {
          ok = false;
          break;
        }
        const unsigned full = smem_u32(&hdr->full[stage]);
        const bool need_b = hdr->held[stage] != it.s;
        mbar_expect_tx(full, 2u * p.region_bytes + (need_b ? p.b_bytes : 0u));
        const unsigned dst = data0 + stage * p.stage_bytes;
        const int r0 = it.band * p.RB, plane0 = it.s * p.B + it.pc * p.NP;
        // x starts two pixels left of the image: those, the two right of it, rows outside the
        // image and planes beyond the tensor arrive as zeros
        tma_load_4d(dst, &tmap, -2, 0, r0 + p.first_e, plane0, full);
        tma_load_4d(dst + p.region_stride, &tmap, -2, 1, r0 + p.first_o, plane0, full);
        if (need_b) {
          bulk_load(dst + 2u * p.region_stride, p.wts + static_cast<size_t>(it.s) * p.b_bytes, p.b_bytes, full);
          hdr->held[stage] = it.s;
        }
      }
      if (!ok) {
        // copies already issued still land in shared memory: wait for them (bounded) before leaving
        const int lo = n > p.stages ? n - p.stages : 0;
        for (int j = lo; j < n; ++j) {
          unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->full[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_dwtc_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = 16
      const unsigned idesc = (1u << 4) | ((kAccCols >> 3) << 17) | ((kRows >> 4) << 24);
      Item it = item_decode(first, p);
      unsigned tile = 0;
      bool ok = true;
      for (int n = 0; n < count && ok; ++n, item_advance(it, p)) {
        const unsigned stage = n % p.stages, phase = (n / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&hdr->full[stage]), phase, abort_flag, p.timeout_ns, &g_dwtc_error, kErrMma)) break;
        tc_fence_after();
        int nbk, rows_valid;
        const int n_tiles = item_tiles(it, p, nbk, rows_valid);
        const unsigned base = data0 + stage * p.stage_bytes, b_base = base + 2u * p.region_stride;
        for (int t = 0; t < n_tiles; ++t, ++tile) {
          const unsigned acc = tile % kAcc, acc_phase = (tile / kAcc) & 1u;
          if (!mbar_wait(smem_u32(&hdr->acc_empty[acc]), acc_phase ^ 1u, abort_flag, p.timeout_ns, &g_dwtc_error, kErrMma)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const unsigned d_tmem = tmem_base + acc * kAccCols;
          const unsigned lane0 = base + static_cast<unsigned>(t) * (kRows * 16u);
          for (int q = 0; q < p.n_instr; ++q) {
            const unsigned long long ad = smem_desc(lane0 + p.a_off[q], p.lbo[q], 128u);
            const unsigned long long bd = smem_desc(b_base + q * kBTile, 256u, 128u);
            umma_f16(d_tmem, ad, bd, idesc, q > 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&hdr->acc_full[acc]));
        }
        if (ok) umma_commit(smem_u32(&hdr->empty[stage]));  // the stage is free once these MMAs have read it
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int set = (warp - 2) >> 2;
    Item it = item_decode(first, p);
    unsigned tile = 0;
    bool ok = true;
    for (int n = 0; n < count && ok; ++n, item_advance(it, p)) {
      int nbk, rows_valid;
      const int n_tiles = item_tiles(it, p, nbk, rows_valid);
      const int r0 = it.band * p.RB;
      const size_t plane0 = static_cast<size_t>(it.s) * p.B + static_cast<size_t>(it.pc) * p.NP;
      const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias) + it.s);
      const float2 blo = make_float2(bv.x, bv.y), bhi = make_float2(bv.z, bv.w);
      const bool last_band = it.band == p.bands - 1;
      for (int t = 0; t < n_tiles; ++t, ++tile) {
        if (static_cast<int>(tile % kEpiSets) != set) continue;
        const unsigned acc = tile % kAcc, acc_phase = (tile / kAcc) & 1u;
        if (!mbar_wait(smem_u32(&hdr->acc_full[acc]), acc_phase, abort_flag, p.timeout_ns, &g_dwtc_error, kErrEpilogue)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const unsigned t_addr = tmem_base + acc * kAccCols + (static_cast<unsigned>(quarter * 32) << 16);
        unsigned r[STRIDE == 1 ? 16 : 4];
        if (STRIDE == 1) {
          tmem_ld16(t_addr, r);
          tmem_ld_wait16(r);
        } else {
          tmem_ld4(t_addr, r);
          tmem_ld_wait4(r);
        }
        // the accumulator is in registers: hand the buffer back before the arithmetic
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[acc]));

        const unsigned L = static_cast<unsigned>(t) * kRows + quarter * 32 + lane;
        const unsigned row = __umulhi(L, p.magic_pw), c = L - row * p.PW;
        const unsigned k = __umulhi(row, p.magic_rpp), i = row - k * p.RPP;
        if (c < 1u || c > static_cast<unsigned>(p.half_w) || i >= static_cast<unsigned>(rows_valid) || k >= static_cast<unsigned>(nbk))
          continue;
        __half* plane_out = p.out + (plane0 + k) * static_cast<size_t>(p.Pout) * 4;
        const ptrdiff_t res_minus_out = p.res - p.out;  // only used when there is a residual
        if (STRIDE == 1) {
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            __half* op = plane_out + (static_cast<size_t>(2 * (r0 + i) + g) * p.out_row_px + 2 * (c - 1)) * 4;
            uint4 q = make_uint4(0u, 0u, 0u, 0u);
            if (TAIL && p.has_res) q = __ldg(reinterpret_cast<const uint4*>(op + res_minus_out));
            const uint2 a = finish_px<ACT, TAIL>(r + 8 * g, blo, bhi, make_uint2(q.x, q.y), p.act_post);
            const uint2 b = finish_px<ACT, TAIL>(r + 8 * g + 4, blo, bhi, make_uint2(q.z, q.w), p.act_post);
            *reinterpret_cast<uint4*>(op) = make_uint4(a.x, a.y, b.x, b.y);
          }
        } else {
          __half* op = plane_out + (static_cast<size_t>(r0 + i) * p.out_row_px + (c - 1)) * 4;
          uint2 q = make_uint2(0u, 0u);
          if (TAIL && p.has_res) q = __ldg(reinterpret_cast<const uint2*>(op + res_minus_out));
          *reinterpret_cast<uint2*>(op) = finish_px<ACT, TAIL>(r, blo, bhi, q, p.act_post);
          // an odd plane carries one extra pixel: keep it zero
          if (last_band && p.Pout > p.out_plane_real && static_cast<int>(i) == rows_valid - 1 && static_cast<int>(c) == p.half_w)
            *reinterpret_cast<uint2*>(plane_out + static_cast<size_t>(p.out_plane_real) * 4) = make_uint2(0u, 0u);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kAcc * kAccCols);
  }
}

// ------------------------------------------------------------------ host side
// One K-chunk of 8: the pairs of staged row (parity `par`, offset `off` in double rows from the
// lane's own row) shifted by `dc` pairs.
struct Chunk {
  int par, off, dc;
};
struct Plan {
  int n_instr = 0;
  Chunk first[kMaxInstr], second[kMaxInstr];
  bool has_second[kMaxInstr];
  int first_row[2] = {0, 0};  // smallest `off` used per parity
  bool ok = false;
};

// tap (ky, kx) that links input (chunk, parity p) to output column n; false if there is none
bool tap_of(int stride, int pt, int pl, const Chunk& ch, int n, int p, int* ky, int* kx) {
  const int t = 2 * ch.off + ch.par;  // input row minus the lane's first output row (stride 1) / twice its output row
  if (stride == 1) {
    const int g = n >> 3, pp = (n >> 2) & 1;
    *ky = t - g + pt;
    *kx = 2 * ch.dc + p - pp + pl;
  } else {
    if (n >= 4) return false;
    *ky = t + pt;
    *kx = 2 * ch.dc + p + pl;
  }
  return *ky >= 0 && *ky < 3 && *kx >= 0 && *kx < 3;
}

Plan make_plan(int stride, int pt, int pl) {
  Plan plan;
  Chunk used[2][16];
  int n_used[2] = {0, 0};
  for (int par = 0; par < 2; ++par)
    for (int off = -1; off <= 2; ++off)
      for (int dc = -1; dc <= 1; ++dc) {
        const Chunk ch{par, off, dc};
        bool any = false;
        for (int n = 0; n < 16 && !any; ++n)
          for (int p = 0; p < 2 && !any; ++p) {
            int ky, kx;
            any = tap_of(stride, pt, pl, ch, n, p, &ky, &kx);
          }
        if (any) used[par][n_used[par]++] = ch;  // enumeration order = ascending address
      }
  for (int par = 0; par < 2; ++par) {
    if (n_used[par] == 0) continue;
    plan.first_row[par] = used[par][0].off;
    for (int i = 0; i < n_used[par]; ++i)
      if (used[par][i].off - plan.first_row[par] > 1) return plan;  // needs more than one extra staged row
    for (int i = 0; i < n_used[par]; i += 2) {
      if (plan.n_instr == kMaxInstr) return plan;
      plan.first[plan.n_instr] = used[par][i];
      plan.has_second[plan.n_instr] = i + 1 < n_used[par];
      if (i + 1 < n_used[par]) plan.second[plan.n_instr] = used[par][i + 1];
      ++plan.n_instr;
    }
  }
  plan.ok = plan.n_instr > 0;
  return plan;
}

struct Geometry {
  int PW, RB, RPP, NP, bands, pchunks, rows_total;
  unsigned region_bytes, region_stride, b_round, stage_bytes, tail;
  int stages;
  size_t smem;
};

Geometry make_geometry(int B, int H, int W, int Ho, int stride, int n_instr) {
  Geometry g;
  g.PW = W / 2 + 2;
  g.rows_total = stride == 1 ? H / 2 : Ho;
  const int row_bytes = g.PW * 16;
  int max_rows = kRegionTarget / row_bytes;  // staged rows per region
  if (max_rows < 3) max_rows = 3;
  if (g.rows_total + 1 <= max_rows) {
    g.RB = g.rows_total;
    g.bands = 1;
    g.NP = max_rows / (g.RB + 1);
    if (g.NP > B) g.NP = B;
    if (g.NP > 256) g.NP = 256;
  } else {
    g.NP = 1;
    g.bands = (g.rows_total + max_rows - 2) / (max_rows - 1);
    g.RB = (g.rows_total + g.bands - 1) / g.bands;
    g.bands = (g.rows_total + g.RB - 1) / g.RB;
  }
  g.RPP = g.RB + 1;
  g.pchunks = (B + g.NP - 1) / g.NP;
  g.region_bytes = static_cast<unsigned>(g.NP) * g.RPP * row_bytes;
  g.region_stride = (g.region_bytes + 127u) & ~127u;
  g.b_round = (static_cast<unsigned>(n_instr) * kBTile + 127u) & ~127u;
  g.stage_bytes = 2u * g.region_stride + g.b_round;
  g.tail = static_cast<unsigned>(kRows + 2 * g.PW + 8) * 16u;
  const long long room = static_cast<long long>(kSmemPerCta) - kHeader - kLead - g.tail;
  long long st = room / g.stage_bytes;
  if (st > kMaxStages) st = kMaxStages;
  if (st < 2) st = 2;
  g.stages = static_cast<int>(st);
  g.smem = static_cast<size_t>(kHeader) + kLead + static_cast<size_t>(g.stages) * g.stage_bytes + g.tail;
  return g;
}

unsigned magic_of(int d) { return static_cast<unsigned>((1ull << 32) / static_cast<unsigned>(d)) + 1u; }

int encode_rows_map(CUtensorMap* map, const void* base, int W, int H, int Pin, long long planes, const Geometry& g) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return static_cast<int>(cudaErrorNotSupported);
  const cuuint64_t gdim[4] = {static_cast<cuuint64_t>(W), 2, static_cast<cuuint64_t>(H / 2), static_cast<cuuint64_t>(planes)};
  const cuuint64_t gstride[3] = {static_cast<cuuint64_t>(W) * 8u, static_cast<cuuint64_t>(W) * 16u, static_cast<cuuint64_t>(Pin) * 8u};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(2 * g.PW), 1, static_cast<cuuint32_t>(g.RPP), static_cast<cuuint32_t>(g.NP)};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult cr = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 4, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return cr == CUDA_SUCCESS ? 0 : static_cast<int>(cudaErrorInvalidValue);
}

}  // namespace

bool depthwise_tc_supported(int H, int W, int Ho, int Wo, int kh, int kw, int sh, int sw, int dh, int dw, int pt, int pl) {
  if (kh != 3 || kw != 3 || sh != sw || (sh != 1 && sh != 2) || dh != 1 || dw != 1) return false;
  if (H < 2 || W < 2 || (H & 1) || (W & 1) || W > 252) return false;
  if (pt < 0 || pt > 1 || pl < 0 || pl > 1) return false;
  if (sh == 1 && (Ho != H || Wo != W || pt != 1 || pl != 1)) return false;
  if (sh == 2 && (Ho != H / 2 || Wo != W / 2)) return false;
  const Plan plan = make_plan(sh, pt, pl);
  if (!plan.ok) return false;
  const Geometry g = make_geometry(1, H, W, Ho, sh, plan.n_instr);
  return g.smem <= static_cast<size_t>(kSmemPerCta) + 8 * 1024 && g.RPP <= 256;
}

// Weight tiles per slice: n_instr x [2 K-chunks][2 column blocks][8 columns x 8 halves]; bias [C4] floats.
void depthwise_tc_pack(const float* w, const float* bias, int c, int stride, int pt, int pl, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Plan plan = make_plan(stride, pt, pl);
  const int S = slices(c);
  const size_t per_slice = static_cast<size_t>(plan.n_instr) * kBTile;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + per_slice * S, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(S) * 4 * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int ch = 0; ch < c; ++ch) bp[ch] = bias[ch];
  for (int s = 0; s < S; ++s)
    for (int q = 0; q < plan.n_instr; ++q) {
      uint16_t* tile = wp + (static_cast<size_t>(s) * per_slice + static_cast<size_t>(q) * kBTile) / 2;
      for (int u = 0; u < 2; ++u) {
        if (u == 1 && !plan.has_second[q]) continue;
        const Chunk& chk = u == 0 ? plan.first[q] : plan.second[q];
        for (int n = 0; n < 16; ++n)
          for (int kk = 0; kk < 8; ++kk) {
            const int p = kk >> 2, ci = kk & 3, ch = s * 4 + ci;
            if ((n & 3) != ci || ch >= c) continue;
            int ky, kx;
            if (!tap_of(stride, pt, pl, chk, n, p, &ky, &kx)) continue;
            // element (n, k = 8u + kk): K block u at 256 bytes, column block n / 8 at 128, column n % 8 at 16
            tile[(u * 256 + (n >> 3) * 128 + (n & 7) * 16) / 2 + kk] = f32_to_f16_rne(w[static_cast<size_t>(ky * 3 + kx) * c + ch]);
          }
      }
    }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = per_slice * S;
}

int launch_depthwise_tc(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream) {
  const Plan plan = make_plan(r.sh, r.pt, r.pl);
  if (!plan.ok) return static_cast<int>(cudaErrorInvalidConfiguration);
  const int S = slices(r.C);
  const Geometry g = make_geometry(r.B, r.H, r.W, r.Ho, r.sh, plan.n_instr);
  static int sms = 0;
  static bool attr_set = false;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    const int bytes = kSmemPerCta + 8 * 1024;
#define GI_DT_ATTR(ST, A, T) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(depthwise_tc_kernel<ST, A, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)
    GI_DT_ATTR(1, GI_ACT_NONE, false);
    GI_DT_ATTR(1, GI_ACT_RELU, false);
    GI_DT_ATTR(1, GI_ACT_RELU6, false);
    GI_DT_ATTR(1, GI_ACT_NONE, true);
    GI_DT_ATTR(1, GI_ACT_RELU, true);
    GI_DT_ATTR(1, GI_ACT_RELU6, true);
    GI_DT_ATTR(2, GI_ACT_NONE, false);
    GI_DT_ATTR(2, GI_ACT_RELU, false);
    GI_DT_ATTR(2, GI_ACT_RELU6, false);
    GI_DT_ATTR(2, GI_ACT_NONE, true);
    GI_DT_ATTR(2, GI_ACT_RELU, true);
    GI_DT_ATTR(2, GI_ACT_RELU6, true);
#undef GI_DT_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_set = true;
  }
  const int Pin = plane_pixels(r.H, r.W);
  MapEntry& me = map_cache_entry(state, launch_index);
  if (me.in != p.in0) {
    const int err = encode_rows_map(&me.map, p.in0, r.W, r.H, Pin, static_cast<long long>(S) * r.B, g);
    if (err != 0) return err;
    me.in = p.in0;
  }
  DtParams k;
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.bias = static_cast<const float*>(p.bias);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.B = r.B;
  k.W = r.W;
  k.Pout = plane_pixels(r.Ho, r.Wo);
  k.PW = g.PW;
  k.half_w = r.W / 2;
  k.RB = g.RB;
  k.RPP = g.RPP;
  k.NP = g.NP;
  k.bands = g.bands;
  k.pchunks = g.pchunks;
  const long long items = static_cast<long long>(S) * g.pchunks * g.bands;
  if (items > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  k.items = static_cast<int>(items);
  k.rows_total = g.rows_total;
  k.first_e = plan.first_row[0];
  k.first_o = plan.first_row[1];
  k.n_instr = plan.n_instr;
  for (int q = 0; q < plan.n_instr; ++q) {
    const Chunk& a = plan.first[q];
    const int rows_a = a.off - plan.first_row[a.par];
    k.a_off[q] = static_cast<int>(a.par ? g.region_stride : 0u) + (rows_a * g.PW + a.dc) * 16;
    if (plan.has_second[q]) {
      const Chunk& b = plan.second[q];
      k.lbo[q] = static_cast<unsigned>(((b.off - a.off) * g.PW + (b.dc - a.dc)) * 16);
    } else {
      k.lbo[q] = 16u;  // the second K-chunk meets an all-zero weight block
    }
  }
  k.region_stride = g.region_stride;
  k.region_bytes = g.region_bytes;
  k.b_bytes = static_cast<unsigned>(plan.n_instr) * kBTile;
  k.stage_bytes = g.stage_bytes;
  k.stages = g.stages;
  k.magic_pw = magic_of(g.PW);
  k.magic_rpp = magic_of(g.RPP);
  k.out_row_px = r.Wo;
  k.out_plane_real = r.Ho * r.Wo;
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  k.timeout_ns = 1000000000u;
  long long grid = static_cast<long long>(sms) * 2;
  if (grid > items) grid = items;
  const unsigned gr = static_cast<unsigned>(grid);
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
  const int act = r.ep.act_pre;
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
#define GI_DT_LAUNCH(ST, A, T) launch_pdl(depthwise_tc_kernel<ST, A, T>, gr, kThreads, g.smem, cu_stream, me.map, k)
#define GI_DT_LAUNCH_ACT(ST, T)                                   \
  do {                                                            \
    if (act == GI_ACT_RELU6) GI_DT_LAUNCH(ST, GI_ACT_RELU6, T);   \
    else if (act == GI_ACT_RELU) GI_DT_LAUNCH(ST, GI_ACT_RELU, T); \
    else GI_DT_LAUNCH(ST, GI_ACT_NONE, T);                        \
  } while (0)
  if (r.sh == 1) {
    if (tail) GI_DT_LAUNCH_ACT(1, true);
    else GI_DT_LAUNCH_ACT(1, false);
  } else {
    if (tail) GI_DT_LAUNCH_ACT(2, true);
    else GI_DT_LAUNCH_ACT(2, false);
  }
#undef GI_DT_LAUNCH_ACT
#undef GI_DT_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

unsigned int depthwise_tc_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_dwtc_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
