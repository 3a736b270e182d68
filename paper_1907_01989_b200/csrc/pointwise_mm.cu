// Pointwise (1x1) convolution for the shapes that are bound by the tensor pipe, not by HBM: many input AND
// output channels (512 -> 512, 960 -> 960, 1280 -> 1280 on 14x14 planes at batch 256).  The other two 1x1
// kernels give a CTA a tile of 128 pixels x 64-192 output channels; per byte fetched from L2 that is 64-77
// flops, and at the rate the tensor pipe could run L2 cannot deliver.  This kernel is built around flops per
// fetched byte and around keeping the pipe busy while a tile is written out:
//
//   CTA pair  a cluster of two CTAs on the two SMs that share a tensor-core pair works on one tile of 256 pixels
//             x up to 256 output channels with tcgen05.mma.cta_group::2 (M = 256): each CTA stages its own 128
//             pixels of the activations and its own half of the weight tile - 128 flops per fetched byte, the
//             hardware exchanges the weight halves - and receives its 128 rows of the accumulator in its own
//             tensor memory.  An accumulator is 256 of the 512 columns, so there are two: the twelve drain warps
//             of each CTA write tile t out while the MMAs of tile t+1 run.  (One CTA per tile with the same
//             fetch ratio needs a 256 x 256 accumulator that fills tensor memory; its drain, 5 us a tile, could
//             not be overlapped: 641 TFLOP/s on 512 -> 512 and 1147 on 1280 -> 1280 where the pair does 713 and 1274.)
//   A chunk   128 pixels x 64 channels per CTA: one tiled TMA copy lands the sixteen 4-channel slices as they lie in
//             memory ([slice][pixel] 8-byte pixel-slices); eight warps (of sixteen: eight for the even chunks, eight
//             for the odd ones) then interleave pairs of slices into the canonical K-major operand rows (16 bytes =
//             8 channels of one pixel) in place - a K group's 2 KB of operand rows lie exactly where its two slices
//             landed, so one warp owns a K group and needs no barrier but its own.  Exactly 2*M*N*K flops, nothing
//             padded or duplicated.  (Gathering the rows with 8-byte cp.async instead - every copy holds a
//             first-level cache line while in flight - fed a chunk in twice the time its MMAs take.)
//   B chunk   this CTA's half of up to 256 output channels x 64 input channels of the dense weight matrix, packed
//             at compile time, one bulk copy
//   MMA       4 tcgen05.mma (256 x N x 16) per chunk, issued by one thread of the pair's first CTA once its own
//             repack warps and the other CTA's - they arrive on a barrier of the first CTA - have finished the
//             chunk; a tcgen05.commit per CTA hands the stage back to both
//   drain     bias (fetched a tile ahead, kept in registers, broadcast by shuffle), activation, residual, fp16, 8-byte
//             stores (256 contiguous bytes per warp)
//
// Tiles are numbered so that pairs running at the same time work on the output-channel tiles of the same pixels:
// the activations come from HBM once, the re-reads hit L2.  Every copy goes to the one CTA that issued it; every wait
// is bounded, and both CTAs of a pair meet at a cluster barrier before either releases tensor memory or leaves.
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

constexpr int kPairRows = 256;    // pixels per tile of a CTA pair
constexpr int kRows = 128;        // pixels per CTA
constexpr int kKc = 16;           // input slices (64 channels) per chunk: the one MMA-issuing thread of a pair pays its waits
                                  // and commits per chunk, and has 128 cycles per MMA to do it in
constexpr int kRepackWarps = 16, kDrainWarps = 12;  // repack: eight warps (one per K group) on even chunks, eight on odd ones
constexpr int kMmaWarp = 1;       // first CTA: MMA issuer
constexpr int kTmaWarp = 2;       // activation copies
constexpr int kFirstRepack = 4, kFirstDrain = kFirstRepack + kRepackWarps;
static_assert(kFirstDrain % 4 == 0, "a drain warp's TMEM lane quarter is its warp index modulo 4");
constexpr int kThreads = 32 * (kFirstDrain + kDrainWarps);
constexpr int kMaxStages = 7;
constexpr int kHeader = 1024;
constexpr int kABytes = (kKc / 2) * kRows * 16;  // 16 KB
constexpr int kSmemMax = 227 * 1024;
constexpr unsigned kAccCols = 256;  // columns per accumulator buffer
constexpr int kGroupsPerWarp = (256 / 16 + kDrainWarps / 4 - 1) / (kDrainWarps / 4);  // 16-column groups a drain warp takes

__device__ unsigned int g_mm_error = 0;

enum : unsigned { kErrCopy = 1u, kErrMma = 2u, kErrLoad = 4u, kErrDrain = 8u, kErrRepack = 16u };

struct MmParams {
  const __half* res;
  __half* out;
  const unsigned char* wts;  // [n_tiles][n_chunks][2 halves] blocks of b_bytes
  const float* bias;
  unsigned int m_total;      // pixels (batch x stored plane)
  int s_out;
  int n_chunks, n_tile, n_tiles, m_tiles;
  int stages;
  unsigned b_bytes, stage_bytes;
  int act_pre, has_res, act_post;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long landed[kMaxStages];     // both copies of a stage (activations as they lie in memory, weights) have arrived
  unsigned long long full[kMaxStages];       // first CTA only: its eight repack warps of the chunk are done
  unsigned long long peer_full[kMaxStages];  // first CTA only: so are the second CTA's (they arrive from there)
  unsigned long long empty[kMaxStages];      // the pair's MMAs on the stage have completed (a commit from the first CTA)
  unsigned long long acc_full[2];            // an accumulator is complete (a commit from the first CTA)
  unsigned long long acc_empty[2];           // first CTA only: the drain warps of both CTAs have read an accumulator
  unsigned tmem_addr, abort_flag;
};
static_assert(sizeof(Header) <= kHeader, "header too large");

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}
// offset (in halves) of the 4 channels [4 so, 4 so + 4) of a pixel: slices of 4 channels, or - S8 - of 8
template <bool S8>
__device__ __forceinline__ size_t slice_offset(int so, unsigned m_total, unsigned pixel) {
  if (S8) return (static_cast<size_t>(so >> 1) * m_total + pixel) * 8 + static_cast<size_t>(so & 1) * 4;
  return (static_cast<size_t>(so) * m_total + pixel) * 4;
}
__device__ __forceinline__ void st_shared_v4(unsigned addr, unsigned a, unsigned b, unsigned c, unsigned d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow; S8: input and output
// are stored in slices of 8 channels (16 bytes per pixel-slice) instead of 4 - the layout experiment of
// gi_slice8_pointwise_*: a pixel-slice is then an operand row, the tiled copy lands the rows where the MMA reads
// them and nothing is rearranged
template <int ACT, bool TAIL, bool S8>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
    pointwise_mm_kernel(const __grid_constant__ CUtensorMap tmap_a, const MmParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned rank = cluster_ctarank();  // 0: issues the pair's MMAs
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned st0 = smem_u32(smem + kHeader);  // stage: A chunk (16 KB), then this CTA's half of the B chunk
  const int n_units = p.m_tiles * p.n_tiles;
  const int pair = static_cast<int>(blockIdx.x >> 1), n_pairs = static_cast<int>(gridDim.x >> 1);

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->landed[i]), 2);
      mbar_init(smem_u32(&hdr->full[i]), kRepackWarps / 2);
      mbar_init(smem_u32(&hdr->peer_full[i]), kRepackWarps / 2);
      mbar_init(smem_u32(&hdr->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), 2 * kDrainWarps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kMmaWarp) tmem_alloc_pair(smem_u32(&hdr->tmem_addr), 512u);
  if (warp == kTmaWarp && lane == 0) prefetch_tensormap(&tmap_a);
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // the other CTA's barriers exist before anything arrives on them
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------ weight chunks (never change: no wait for the previous kernel)
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      for (int u = pair; u < n_units && ok; u += n_pairs) {
        const int nt = u % p.n_tiles;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
          if (!mbar_wait_cluster(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_mm_error, kErrCopy)) {
            ok = false;
            break;
          }
          const unsigned landed = smem_u32(&hdr->landed[stage]);
          mbar_expect_tx(landed, p.b_bytes);
          bulk_load(st0 + stage * p.stage_bytes + kABytes,
                    p.wts + ((static_cast<size_t>(nt) * p.n_chunks + c) * 2 + rank) * p.b_bytes, p.b_bytes, landed);
        }
      }
      if (!ok) {
        // copies in flight must land before the CTA leaves
        const unsigned first = it > static_cast<unsigned>(p.stages) ? it - p.stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->landed[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_mm_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == kMmaWarp) {
    if (rank == 0) {
      // ------------------------------------------------------------ MMA issuer of the pair.  The whole warp runs the
      // loop - addresses, descriptors and barrier phases are then warp-uniform values the compiler keeps in uniform
      // registers, which is where tcgen05.mma takes its operands from - and one elected lane issues.
      const bool issuer = elect_one();
      const unsigned n_cols = static_cast<unsigned>(p.n_tile);
      const unsigned idesc = (1u << 4) | ((n_cols >> 3) << 17) | ((256u >> 4) << 24);
      const unsigned a_lbo = kRows * 16u, b_lbo = (n_cols >> 1) * 16u;
      const unsigned long long ad_step = static_cast<unsigned long long>((2u * a_lbo) >> 4);
      const unsigned long long bd_step = static_cast<unsigned long long>((2u * b_lbo) >> 4);
      // a shared-memory address of the second CTA is this CTA's address plus a constant
      const unsigned to_peer = mapa_shared(smem_u32(hdr), 1) - smem_u32(hdr);
      // The tensor pipe queues only an MMA or two: whatever this thread does between the last MMA of a chunk and the
      // first of the next is time the pipe may stand still.  So the barriers of chunk c+1 are polled before the MMAs of
      // chunk c are issued (a test that never suspends; the answer arrives while the MMAs run, and the copies are
      // usually that far ahead), the descriptors are one multiply-add per stage, and the other CTA's barriers are
      // this CTA's plus a constant.
      const unsigned long long ad0 = smem_desc(st0, a_lbo, 128), bd0 = smem_desc(st0 + kABytes, b_lbo, 128);
      const unsigned long long stage_step = static_cast<unsigned long long>(p.stage_bytes >> 4);
      const unsigned full0 = smem_u32(&hdr->full[0]), peer0 = smem_u32(&hdr->peer_full[0]), empty0 = smem_u32(&hdr->empty[0]);
      const unsigned n_stages = static_cast<unsigned>(p.stages);
      unsigned stage = 0, phase = 0, tile = 0;
      bool ok = true, ready = false;
      for (int u = pair; u < n_units && ok; u += n_pairs, ++tile) {
        const unsigned buf = tile & 1u, use = tile >> 1;
        // the first MMA of a tile overwrites the accumulator: both CTAs must have drained its previous tile
        if (!mbar_wait_cluster_warp(smem_u32(&hdr->acc_empty[buf]), (use & 1u) ^ 1u, abort_flag, p.timeout_ns, &g_mm_error, kErrMma)) break;
        const unsigned d_tmem = tmem_base + buf * kAccCols;
        for (int c = 0; c < p.n_chunks; ++c) {
          if (!ready && (!mbar_wait_warp(full0 + stage * 8u, phase, abort_flag, p.timeout_ns, &g_mm_error, kErrMma) ||
                         !mbar_wait_cluster_warp(peer0 + stage * 8u, phase, abort_flag, p.timeout_ns, &g_mm_error, kErrMma))) {
            ok = false;
            break;
          }
          tc_fence_after();
          // the next chunk of this CTA's sequence (it may belong to the next tile)
          unsigned nstage = stage + 1, nphase = phase;
          if (nstage == n_stages) {
            nstage = 0;
            nphase ^= 1u;
          }
          const bool next_full = mbar_test_wait(full0 + nstage * 8u, nphase);
          const bool next_peer = mbar_test_wait_cluster(peer0 + nstage * 8u, nphase);
          unsigned long long ad = ad0 + stage * stage_step, bd = bd0 + stage * stage_step;
          const unsigned e = empty0 + stage * 8u;
          if (issuer) {
#pragma unroll
            for (int ks = 0; ks < kKc / 4; ++ks) {
              umma_pair_f16(d_tmem, ad, bd, idesc, (c > 0 || ks > 0) ? 1u : 0u);
              ad += ad_step;
              bd += bd_step;
            }
            // the stage goes back to the copy threads of both CTAs
            umma_pair_commit(e);
            umma_pair_commit(e + to_peer);
          }
          __syncwarp();
          ready = __all_sync(0xffffffffu, next_full && next_peer) != 0;
          stage = nstage;
          phase = nphase;
        }
        if (ok && issuer) {
          const unsigned f = smem_u32(&hdr->acc_full[buf]);
          umma_pair_commit(f);
          umma_pair_commit(f + to_peer);
        }
        __syncwarp();
      }
    }
  } else if (warp == kTmaWarp) {
    // ------------------------------------------------------------ activation chunks: one tiled copy of 128 pixels x 8 slices
    // each; pixels beyond the tensor's end and slices beyond its last one read as zeros
    if (lane == 0) {
      pdl_wait();  // the activations are the previous kernel's output
      unsigned it = 0;
      bool ok = true;
      for (int u = pair; u < n_units && ok; u += n_pairs) {
        const int mt = u / p.n_tiles;
        const int px0 = mt * kPairRows + static_cast<int>(rank) * kRows;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
          if (!mbar_wait_cluster(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_mm_error, kErrLoad)) {
            ok = false;
            break;
          }
          const unsigned landed = smem_u32(&hdr->landed[stage]);
          mbar_expect_tx(landed, kABytes);
          // (8-channel slices: the map counts 8-byte halves of the 16-byte pixel-slices)
          if (S8) tma_load_2d(st0 + stage * p.stage_bytes, &tmap_a, 2 * px0, c * (kKc / 2), landed);
          else tma_load_2d(st0 + stage * p.stage_bytes, &tmap_a, px0, c * kKc, landed);
        }
      }
      if (!ok) {
        const unsigned first = it > static_cast<unsigned>(p.stages) ? it - p.stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->landed[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_mm_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp >= kFirstRepack && warp < kFirstDrain) {
    // ------------------------------------------------------------ landing layout -> operand layout, in place.  Landed:
    // [slice][pixel] 8-byte pixel-slices (1 KB per slice); operand: [K group of 8 channels][pixel] 16-byte rows (2 KB
    // per K group) - K group g takes the place of slices 2g and 2g+1.  A warp owns one K group of every second chunk:
    // it reads the group's 256 pixel-slices into registers, and only then writes its 128 rows.  It then counts itself
    // in on a barrier of the first CTA.  From the second CTA that arrival is a relaxed one: the proxy fence before it
    // has already made the rows visible to this SM's tensor core, which is the one that reads them, and a releasing
    // arrival across the pair (a full memory barrier on an SM with copies in flight) took a chunk's time by itself.
    const int rw = warp - kFirstRepack;
    const unsigned kg = static_cast<unsigned>(rw & 7), parity = static_cast<unsigned>(rw >> 3);
    const unsigned peer_full0 = mapa_shared(smem_u32(&hdr->peer_full[0]), 0);
    unsigned it = 0;
    bool ok = true;
    for (int u = pair; u < n_units && ok; u += n_pairs) {
      for (int c = 0; c < p.n_chunks; ++c, ++it) {
        if ((it & 1u) != parity) continue;
        const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
        if (!mbar_wait_warp(smem_u32(&hdr->landed[stage]), phase, abort_flag, p.timeout_ns, &g_mm_error, kErrRepack)) {
          ok = false;
          break;
        }
        if (!S8) {
          const unsigned base = st0 + stage * p.stage_bytes + kg * 2048u;
          unsigned lo[4][2], hi[4][2];  // pixel-slices of the even and of the odd slice, pixels lane, lane + 32, ...
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const unsigned px = static_cast<unsigned>(lane + 32 * j);
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(lo[j][0]), "=r"(lo[j][1]) : "r"(base + px * 8u) : "memory");
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(hi[j][0]), "=r"(hi[j][1]) : "r"(base + 1024u + px * 8u) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j)
            st_shared_v4(base + static_cast<unsigned>(lane + 32 * j) * 16u, lo[j][0], lo[j][1], hi[j][0], hi[j][1]);
          // visible to the tensor core's proxy, then count this warp in
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
        }  // with 8-channel slices the copy itself wrote the operand rows: the warp only passes the arrival on
        if (lane == 0) {
          if (rank == 0) mbar_arrive(smem_u32(&hdr->full[stage]));
          else asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(peer_full0 + stage * 8u) : "memory");
        }
      }
    }
  } else if (warp >= kFirstDrain) {
    // ------------------------------------------------------------ drain: this CTA's 128 rows of an accumulator -> global memory
    const int dw = warp - kFirstDrain;
    const int quarter = warp & 3, sub = dw >> 2;  // TMEM lane quarter; index among the warps sharing it
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int groups = p.n_tile >> 4;
    pdl_wait();  // the residual is read and the output written only below
    unsigned tile = 0;
    float bnext[kGroupsPerWarp];  // the first tile's bias values
#pragma unroll
    for (int k = 0; k < kGroupsPerWarp; ++k) {
      const int g = sub + k * (kDrainWarps / 4);
      bnext[k] = (g < groups && pair < n_units) ? __ldg(p.bias + (pair % p.n_tiles) * p.n_tile + g * 16 + (lane & 15)) : 0.f;
    }
    for (int u = pair; u < n_units; u += n_pairs, ++tile) {
      const int mt = u / p.n_tiles, nt = u - mt * p.n_tiles;
      const unsigned buf = tile & 1u, use = tile >> 1;
      // The tile's bias values were fetched during the tile before (the next tile's are fetched now): lane l keeps column l % 16 of each
      // of this warp's groups and the epilogue broadcasts from there.  (A load from global memory per slice inside
      // the epilogue - queued behind the barrier polls and shared-memory traffic of thirty other warps - took two
      // thirds of the drain.)
      float bpre[kGroupsPerWarp];
#pragma unroll
      for (int k = 0; k < kGroupsPerWarp; ++k) bpre[k] = bnext[k];
      const int un = u + n_pairs;
      const int ntn = un < n_units ? un % p.n_tiles : 0;
#pragma unroll
      for (int k = 0; k < kGroupsPerWarp; ++k) {
        const int g = sub + k * (kDrainWarps / 4);
        bnext[k] = g < groups ? __ldg(p.bias + ntn * p.n_tile + g * 16 + (lane & 15)) : 0.f;
      }
      if (!mbar_wait_cluster_parked_warp(smem_u32(&hdr->acc_full[buf]), use & 1u, abort_flag, p.timeout_ns, &g_mm_error, kErrDrain)) break;
      tc_fence_after();
      const unsigned pixel = static_cast<unsigned>(mt) * kPairRows + rank * kRows + static_cast<unsigned>(quarter * 32 + lane);
      const bool px_ok = pixel < p.m_total;
#pragma unroll
      for (int k = 0; k < kGroupsPerWarp; ++k) {  // 16-column groups of this lane quarter, dealt round-robin
        const int g = sub + k * (kDrainWarps / 4);
        if (g >= groups) break;
        unsigned r[16];
        tmem_ld16(tmem_base + lane_bits + buf * kAccCols + static_cast<unsigned>(g * 16), r);
        const int so0 = (nt * p.n_tile) / 4 + g * 4;
        uint2 rq[4];
        if (TAIL) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            rq[j] = make_uint2(0u, 0u);
            if (p.has_res && px_ok && so0 + j < p.s_out)
              rq[j] = __ldg(reinterpret_cast<const uint2*>(p.res + slice_offset<S8>(so0 + j, p.m_total, pixel)));
          }
        }
        tmem_ld_wait16(r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float4 b;
          b.x = __shfl_sync(0xffffffffu, bpre[k], 4 * j);
          b.y = __shfl_sync(0xffffffffu, bpre[k], 4 * j + 1);
          b.z = __shfl_sync(0xffffffffu, bpre[k], 4 * j + 2);
          b.w = __shfl_sync(0xffffffffu, bpre[k], 4 * j + 3);
          if (so0 + j >= p.s_out || !px_ok) continue;
          const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1])), make_float2(b.x, b.y));
          const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])), make_float2(b.z, b.w));
          uint2 o;
          if (!TAIL) {
            // the conversion clamps at zero itself; clamping at 6 after the rounding equals rounding after the clamp
            o.x = pack_f16x2<ACT != GI_ACT_NONE>(v0.x, v0.y);
            o.y = pack_f16x2<ACT != GI_ACT_NONE>(v1.x, v1.y);
            if (ACT == GI_ACT_RELU6) {
              const __half2 six = __float2half2_rn(6.f);
              const __half2 h0 = __hmin2(*reinterpret_cast<const __half2*>(&o.x), six), h1 = __hmin2(*reinterpret_cast<const __half2*>(&o.y), six);
              o.x = *reinterpret_cast<const unsigned*>(&h0);
              o.y = *reinterpret_cast<const unsigned*>(&h1);
            }
          } else {
            const float2 q0 = __half22float2(*reinterpret_cast<const __half2*>(&rq[j].x));
            const float2 q1 = __half22float2(*reinterpret_cast<const __half2*>(&rq[j].y));
            o.x = pack_f16x2<false>(act1(act1(v0.x, ACT) + q0.x, p.act_post), act1(act1(v0.y, ACT) + q0.y, p.act_post));
            o.y = pack_f16x2<false>(act1(act1(v1.x, ACT) + q1.x, p.act_post), act1(act1(v1.y, ACT) + q1.y, p.act_post));
          }
          *reinterpret_cast<uint2*>(p.out + slice_offset<S8>(so0 + j, p.m_total, pixel)) = o;
        }
      }
      // every tensor-memory load of this warp has completed (the wait above): a relaxed arrival is enough to let the
      // issuer overwrite the accumulator
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(smem_u32(&hdr->acc_empty[buf]));
        else asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(mapa_shared(smem_u32(&hdr->acc_empty[buf]), 0)) : "memory");
      }
    }
  }

  // Neither CTA may release tensor memory or leave while the other can still read its shared memory (the pair's
  // MMAs), write its tensor memory or arrive on its barriers: every role above ends after a bounded time, then both
  // CTAs meet here.
  tc_fence_before();
  __syncthreads();
  cluster_sync();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512u);
  }
}

struct Tiling {
  int s_in, s_out, n_chunks, n_tiles, n_tile, stages;
  unsigned b_bytes, stage_bytes;  // b_bytes: one CTA's half of a weight chunk
  size_t smem;
};

Tiling choose_tiling(int cin, int cout) {
  Tiling t;
  t.s_in = slices(cin);
  t.s_out = slices(cout);
  t.n_chunks = (t.s_in + kKc - 1) / kKc;
  const int n_pad = (cout + 15) / 16 * 16;
  t.n_tiles = (n_pad + 255) / 256;
  t.n_tile = ((n_pad + t.n_tiles - 1) / t.n_tiles + 15) / 16 * 16;
  t.b_bytes = static_cast<unsigned>(t.n_tile / 2) * kKc * 8u;  // n_tile / 2 rows x 32 channels x 2 bytes
  t.stage_bytes = kABytes + t.b_bytes;
  int stages = (kSmemMax - kHeader) / static_cast<int>(t.stage_bytes);
  t.stages = stages > kMaxStages ? kMaxStages : stages;
  t.smem = kHeader + static_cast<size_t>(t.stages) * t.stage_bytes;
  return t;
}

}  // namespace

bool pointwise_mm_supported(int cin, int cout) {
  if (cin <= 0 || cout <= 0) return false;
  return choose_tiling(cin, cout).stages >= 4;
}

// Where pointwise_mm_pack puts things in an empty blob: weights at 0, bias behind them; total size.
void pointwise_mm_blob_layout(int cin, int cout, uint64_t* bias_off, uint64_t* total) {
  const Tiling t = choose_tiling(cin, cout);
  const uint64_t wbytes = static_cast<uint64_t>(t.n_tiles) * t.n_chunks * 2 * t.b_bytes;
  *bias_off = round_up_u64(wbytes, 256);
  *total = *bias_off + static_cast<uint64_t>(t.n_tiles) * t.n_tile * sizeof(float);
}

// Dense weights as the B operand, per (output tile, K chunk, half of the tile's rows): [4 K groups][n_tile / 2 rows]
// [8 halves]; entries beyond the real channels are zero.
void pointwise_mm_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Tiling t = choose_tiling(cin, cout);
  const size_t wbytes = static_cast<size_t>(t.n_tiles) * t.n_chunks * 2 * t.b_bytes;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(t.n_tiles) * t.n_tile * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  const int half_rows = t.n_tile / 2;
  for (int co = 0; co < cout; ++co) {
    const int nt = co / t.n_tile, row = co % t.n_tile;
    const int half = row / half_rows, hr = row % half_rows;
    bp[co] = bias[co];
    for (int ci = 0; ci < cin; ++ci) {
      const int chunk = ci / (kKc * 4), k = ci % (kKc * 4);
      uint16_t* base = wp + ((static_cast<size_t>(nt) * t.n_chunks + chunk) * 2 + half) * (t.b_bytes / 2);
      base[(static_cast<size_t>(k / 8) * half_rows + hr) * 8 + k % 8] = f32_to_f16_rne(w[static_cast<size_t>(co) * cin + ci]);
    }
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = t.n_tile;
  r->tc_kc = kKc;
  r->tc_stages = t.stages;
}

int launch_pointwise_mm(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream) {
  const Tiling t = choose_tiling(r.C, r.Co);
  MmParams k{};
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.bias = static_cast<const float*>(p.bias);
  k.m_total = static_cast<unsigned>(r.B) * static_cast<unsigned>(plane_pixels(r.H, r.W));
  k.s_out = t.s_out;
  k.n_chunks = t.n_chunks;
  k.n_tile = t.n_tile;
  k.n_tiles = t.n_tiles;
  k.m_tiles = static_cast<int>((k.m_total + kPairRows - 1) / kPairRows);
  k.stages = t.stages;
  k.b_bytes = t.b_bytes;
  k.stage_bytes = t.stage_bytes;
  k.act_pre = r.ep.act_pre;
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  k.timeout_ns = 1000000000u;
  static bool attr_done_dev[kMaxDevices] = {};
  bool& attr_done = attr_done_dev[current_device_slot()];
  if (!attr_done) {
    cudaError_t e = cudaSuccess;
#define GI_MM_ATTR(A, T) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(pointwise_mm_kernel<A, T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax)
    GI_MM_ATTR(GI_ACT_NONE, false);
    GI_MM_ATTR(GI_ACT_RELU, false);
    GI_MM_ATTR(GI_ACT_RELU6, false);
    GI_MM_ATTR(GI_ACT_NONE, true);
    GI_MM_ATTR(GI_ACT_RELU, true);
    GI_MM_ATTR(GI_ACT_RELU6, true);
#undef GI_MM_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_done = true;
  }
  CUtensorMap tmap;
  {
    const int err = map_cache_lookup(state, launch_index, p.in0, &tmap, [&](CUtensorMap* m) {
      return encode_plane_map(m, p.in0, k.m_total, t.s_in, kRows, kKc);
    });
    if (err != 0) return err;
  }
  const long long units = static_cast<long long>(k.m_tiles) * k.n_tiles;
  const int pairs_max = device_sm_count() / 2;
  const unsigned grid = 2u * static_cast<unsigned>(units < pairs_max ? units : pairs_max);
  // the pair reserves all of tensor memory: ask for enough shared memory that no second CTA shares the SM
  size_t smem = t.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
#define GI_MM_LAUNCH(A, T) launch_pdl(pointwise_mm_kernel<A, T, false>, grid, kThreads, smem, st, tmap, k)
  if (tail) {
    if (k.act_pre == GI_ACT_RELU6) GI_MM_LAUNCH(GI_ACT_RELU6, true);
    else if (k.act_pre == GI_ACT_RELU) GI_MM_LAUNCH(GI_ACT_RELU, true);
    else GI_MM_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (k.act_pre == GI_ACT_RELU6) GI_MM_LAUNCH(GI_ACT_RELU6, false);
    else if (k.act_pre == GI_ACT_RELU) GI_MM_LAUNCH(GI_ACT_RELU, false);
    else GI_MM_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_MM_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

// The layout experiment: the same kernel on tensors stored in slices of 8 channels.  `wts` / `bias` are device copies of
// what pointwise_mm_pack wrote (the packed weights do not depend on the activations' slice width).
int launch_pointwise_mm_slice8(const void* in, void* out, const void* wts, const float* bias, unsigned m_total, int cin, int cout,
                               int act, void* stream) {
  const Tiling t = choose_tiling(cin, cout);
  MmParams k{};
  k.res = nullptr;
  k.out = static_cast<__half*>(out);
  k.wts = static_cast<const unsigned char*>(wts);
  k.bias = bias;
  k.m_total = m_total;
  k.s_out = 2 * ((cout + 7) / 8);  // in 4-channel groups: the whole last 8-channel slice is written (zeros beyond cout)
  k.n_chunks = t.n_chunks;
  k.n_tile = t.n_tile;
  k.n_tiles = t.n_tiles;
  k.m_tiles = static_cast<int>((m_total + kPairRows - 1) / kPairRows);
  k.stages = t.stages;
  k.b_bytes = t.b_bytes;
  k.stage_bytes = t.stage_bytes;
  k.act_pre = act;
  k.timeout_ns = 1000000000u;
  static bool attr_done_dev[kMaxDevices] = {};
  bool& attr_done = attr_done_dev[current_device_slot()];
  if (!attr_done) {
    cudaError_t e = cudaSuccess;
#define GI_MM_ATTR(A) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(pointwise_mm_kernel<A, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax)
    GI_MM_ATTR(GI_ACT_NONE);
    GI_MM_ATTR(GI_ACT_RELU);
    GI_MM_ATTR(GI_ACT_RELU6);
#undef GI_MM_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    attr_done = true;
  }
  CUtensorMap tmap;
  {
    // [slices of 8][pixels][16 bytes] as rows of 8-byte elements: a box of 128 pixels x 8 slices lands as 8 blocks of
    // 128 16-byte rows - the canonical K-major operand layout as it is
    const int err = encode_plane_map(&tmap, in, 2ull * m_total, (cin + 7) / 8, 2 * kRows, kKc / 2);
    if (err != 0) return err;
  }
  const long long units = static_cast<long long>(k.m_tiles) * k.n_tiles;
  const int pairs_max = device_sm_count() / 2;
  const unsigned grid = 2u * static_cast<unsigned>(units < pairs_max ? units : pairs_max);
  size_t smem = t.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (act == GI_ACT_RELU6) launch_pdl(pointwise_mm_kernel<GI_ACT_RELU6, false, true>, grid, kThreads, smem, st, tmap, k);
  else if (act == GI_ACT_RELU) launch_pdl(pointwise_mm_kernel<GI_ACT_RELU, false, true>, grid, kThreads, smem, st, tmap, k);
  else launch_pdl(pointwise_mm_kernel<GI_ACT_NONE, false, true>, grid, kThreads, smem, st, tmap, k);
  return static_cast<int>(cudaGetLastError());
}

unsigned int pointwise_mm_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_mm_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
