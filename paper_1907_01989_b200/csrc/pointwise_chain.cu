// Two consecutive 1x1 convolutions as ONE kernel (fp16 storage): the projection that ends an inverted-residual
// block (many channels -> few, + residual) and the expansion that opens the next block (few -> 6x as many).
// A 1x1 convolution has no spatial extent, so a tile of pixels can run through both operators without ever meeting
// another tile; the paper's cure for an engine bound by memory and dispatch is fewer, fatter programs (Section 3.2,
// "Shader Program Optimization").  The narrow tensor between the two is still written - the next block's residual
// sum reads it - but it is not read back: it goes from the first accumulator straight into the second MMA's operand.
// One launch, one fill and one drain replace two, and the second operator's input costs no memory traffic.
//
// Per tile of 128 pixels (row r of every MMA = pixel r of the tile):
//   G1   D1[128 x N1] = X[128 x K1] * W1^T       X streamed in 64-channel chunks: one TMA box (128 pixels x 16 slices) per
//                                                chunk lands in a deep ring; four warps rearrange it IN PLACE into the
//                                                canonical K-major operand layout (two 4-channel slices interleave into
//                                                one 16-byte operand row: every thread reads its pixel's sixteen pixel-slices,
//                                                the 128 threads meet at a named barrier, every thread writes its pixel's
//                                                eight rows); the chunk's W1 rows (bulk copy) have a ring of their own.  (8-byte
//                                                cp.async straight into the operand layout was the first version: each copy
//                                                holds an L1 line while in flight, and the little L1 left beside 200 KB of
//                                                shared memory capped a CTA at 14 GB/s.)
//   T1   bias, activation, residual, activation, fp16 -> global memory (the first operator's output) AND -> shared
//        memory in the operand layout (A2)
//   G2   D2[128 x n2_blk] = A2[128 x N1] * W2[block]^T     for each block of output channels; W2 blocks by bulk copy,
//                                                resident when all of them fit
//   T2   bias, activation, fp16 -> global memory (the second operator's output)
// D1 and A2 are double-buffered where tensor memory allows, D2 always: the MMA thread issues G1 of tile t+1 and keeps G2 of
// tile t as pending work that its waits poll for, so loads, both MMAs and both drains of neighbouring tiles overlap.
//
// Warps: 0 = X copies, 1 = MMA issuer and TMEM owner, 2..5 = X repack, 6..9 = T1, 10..21 = T2, 22 = W2 copies, 23 = W1 copies.
// All waits are bounded; a wait that runs out raises the abort flag and every role leaves its loop.
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

constexpr int kRows = 128;  // pixels per tile
constexpr int kKc = 16;     // input slices (64 channels) per chunk of G1
constexpr int kLoadWarps = 4, kT1Warps = 4, kT2Warps = 12;
constexpr int kFirstLoad = 2, kFirstT1 = kFirstLoad + kLoadWarps, kFirstT2 = kFirstT1 + kT1Warps;
constexpr int kW2Warp = kFirstT2 + kT2Warps, kW1Warp = kW2Warp + 1;
constexpr int kThreads = 32 * (kW1Warp + 1);
constexpr int kMaxLand = 16, kMaxW1 = 8, kMaxW2Slots = 12;
constexpr int kHeader = 1024;
constexpr int kABytes = (kKc / 2) * kRows * 16;  // 16 KB: one chunk of X
constexpr int kSmemMax = 227 * 1024;
constexpr int kMinLand = 3;  // landing stages: the launches this kernel is for are bound by bytes in flight per SM

__device__ unsigned int g_pc_error = 0;
enum : unsigned { kErrCopy = 1u, kErrMma = 2u, kErrLoad = 4u, kErrDrain = 8u };
#ifdef GI_TRACE
// debug builds: global-timer stamps of the first four tiles of every CTA (16 events per tile)
__device__ unsigned long long g_pc_trace[256 * 64];
#define PC_EV(tile, k)                                            \
  do {                                                            \
    if (blockIdx.x < 256 && (tile) < 4) {                         \
      unsigned long long t_;                                      \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));      \
      g_pc_trace[blockIdx.x * 64 + (tile) * 16 + (k)] = t_;       \
    }                                                             \
  } while (0)
#else
#define PC_EV(tile, k) ((void)0)
#endif

struct PcParams {
  const __half* in;
  const __half* res;
  __half* out1;
  __half* out2;
  const unsigned char* w1;  // n_chunks blocks of w1_bytes
  const unsigned char* w2;  // n2_blocks blocks of w2_bytes
  const float* bias;        // n1_pad floats of the first operator, then n2_blocks * n2_blk of the second
  unsigned int m_total;     // pixels (batch x stored plane)
  int m_tiles;
  int s_in, s_mid, s_out;
  int n_chunks, n1_pad, n2_blk, n2_blocks;
  int d_bufs;               // buffers of D1 and of A2 (1 or 2)
  int land, w1_stages, w2_slots, w2_resident, in_dead;
  unsigned w1_bytes, w2_bytes, w2_pitch, a2_bytes;
  unsigned off_res, off_a2, off_w2, off_w1, off_land;  // shared-memory offsets (the biases sit right behind the header)
  unsigned d2_col0;                    // first tensor-memory column of D2
  int act1_pre, has_res, act1_post;
  unsigned timeout_ns;
};

struct Header {
  unsigned long long land_full[kMaxLand], op_full[kMaxLand], land_empty[kMaxLand];  // an X box landed / rearranged / consumed
  unsigned long long w1_full[kMaxW1], w1_empty[kMaxW1];          // a chunk's W1 rows; freed by the MMA
  unsigned long long w2_full[kMaxW2Slots], w2_empty[kMaxW2Slots];
  unsigned long long d1_full[2], d1_empty[2], a2_full[2], a2_empty[2], d2_full[2], d2_empty[2];
  unsigned tmem_addr, abort_flag;
};
static_assert(sizeof(Header) <= kHeader, "header too large");

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}
// 8-byte asynchronous copy; with `bytes` = 0 nothing is read and the destination is filled with zeros
__device__ __forceinline__ void cp_async8_zfill(unsigned dst, const void* src, unsigned bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_pending() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void st_shared_v4(unsigned addr, unsigned a, unsigned b, unsigned c, unsigned d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// ACT2: the second operator's activation (it has neither a residual nor a second activation); LINEAR1: the first
// operator has no activation (the linear bottleneck of an inverted-residual block), only bias and residual
template <int ACT2, bool LINEAR1>
__global__ void __launch_bounds__(kThreads, 1) pointwise_chain_kernel(const __grid_constant__ CUtensorMap tmap_x, const PcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  float* sbias = reinterpret_cast<float*>(smem + kHeader);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned smem0 = smem_u32(smem);
  const unsigned land0 = smem0 + p.off_land, w1_0 = smem0 + p.off_w1, a2_0 = smem0 + p.off_a2, w2_0 = smem0 + p.off_w2;
  const int my_tiles = (p.m_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.land; ++i) {
      mbar_init(smem_u32(&hdr->land_full[i]), 1);
      mbar_init(smem_u32(&hdr->op_full[i]), kLoadWarps);
      mbar_init(smem_u32(&hdr->land_empty[i]), 1);
    }
    for (int i = 0; i < p.w1_stages; ++i) {
      mbar_init(smem_u32(&hdr->w1_full[i]), 1);
      mbar_init(smem_u32(&hdr->w1_empty[i]), 1);
    }
    prefetch_tensormap(&tmap_x);
    for (int i = 0; i < p.w2_slots; ++i) {
      mbar_init(smem_u32(&hdr->w2_full[i]), 1);
      mbar_init(smem_u32(&hdr->w2_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->d1_full[i]), 1);
      mbar_init(smem_u32(&hdr->d1_empty[i]), kT1Warps);
      mbar_init(smem_u32(&hdr->a2_full[i]), kT1Warps);
      mbar_init(smem_u32(&hdr->a2_empty[i]), 1);
      mbar_init(smem_u32(&hdr->d2_full[i]), 1);
      mbar_init(smem_u32(&hdr->d2_empty[i]), kT2Warps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), 512u);
  // biases never change: no wait for the previous kernel
  for (int i = threadIdx.x; i < p.n1_pad + p.n2_blocks * p.n2_blk; i += kThreads) sbias[i] = __ldg(p.bias + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  pdl_launch_dependents();
  if (threadIdx.x == 0) PC_EV(3, 15);

  if (warp == 0) {
    // ------------------------------------------------------------ X boxes into the landing ring
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      const unsigned long long evict_first = policy_evict_first();
      pdl_wait();  // the activations are the previous kernel's output
      for (int i = 0; i < my_tiles && ok; ++i) {
        const int px0 = static_cast<int>((blockIdx.x + static_cast<unsigned>(i) * gridDim.x) * kRows);
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned st = it % p.land, phase = (it / p.land) & 1u;
          if (!mbar_wait_parked(smem_u32(&hdr->land_empty[st]), phase ^ 1u, abort_flag, p.timeout_ns, &g_pc_error, kErrCopy)) {
            ok = false;
            break;
          }
          if (c == 0) PC_EV(i, 0);
          const unsigned full = smem_u32(&hdr->land_full[st]), dst = land0 + st * kABytes;
          mbar_expect_tx(full, kABytes);
          if (p.in_dead) tma_load_2d_hint(dst, &tmap_x, px0, c * kKc, full, evict_first);
          else tma_load_2d(dst, &tmap_x, px0, c * kKc, full);
          if (c == p.n_chunks - 1) PC_EV(i, 1);
        }
      }
      if (!ok) {
        // copies in flight must land before the CTA leaves
        const unsigned first = it > static_cast<unsigned>(p.land) ? it - p.land : 0u;
        for (unsigned j = first; j < it; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->land_full[j % p.land]), (j / p.land) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_pc_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == kW1Warp) {
    // ------------------------------------------------------------ W1 chunks (weights never change: no wait for the previous kernel)
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      for (int i = 0; i < my_tiles && ok; ++i) {
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned st = it % p.w1_stages, phase = (it / p.w1_stages) & 1u;
          if (!mbar_wait_parked(smem_u32(&hdr->w1_empty[st]), phase ^ 1u, abort_flag, p.timeout_ns, &g_pc_error, kErrCopy)) {
            ok = false;
            break;
          }
          const unsigned full = smem_u32(&hdr->w1_full[st]);
          mbar_expect_tx(full, p.w1_bytes);
          bulk_load(w1_0 + st * p.w1_bytes, p.w1 + static_cast<size_t>(c) * p.w1_bytes, p.w1_bytes, full);
        }
      }
      if (!ok) {
        const unsigned first = it > static_cast<unsigned>(p.w1_stages) ? it - p.w1_stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->w1_full[j % p.w1_stages]), (j / p.w1_stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_pc_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == kW2Warp) {
    // ------------------------------------------------------------ W2 blocks: once if they all fit, else a ring per tile
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      const int rounds = p.w2_resident ? (my_tiles > 0 ? 1 : 0) : my_tiles;
      for (int i = 0; i < rounds && ok; ++i) {
        for (int j = 0; j < p.n2_blocks; ++j, ++it) {
          const unsigned slot = it % p.w2_slots, phase = (it / p.w2_slots) & 1u;
          if (!p.w2_resident &&
              !mbar_wait_parked(smem_u32(&hdr->w2_empty[slot]), phase ^ 1u, abort_flag, p.timeout_ns, &g_pc_error, kErrCopy)) {
            ok = false;
            break;
          }
          const unsigned full = smem_u32(&hdr->w2_full[slot]);
          mbar_expect_tx(full, p.w2_bytes);
          bulk_load(w2_0 + slot * p.w2_pitch, p.w2 + static_cast<size_t>(j) * p.w2_bytes, p.w2_bytes, full);
        }
      }
      if (!ok) {
        const unsigned first = it > static_cast<unsigned>(p.w2_slots) ? it - p.w2_slots : 0u;
        for (unsigned j = first; j < it; ++j) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->w2_full[j % p.w2_slots]), (j / p.w2_slots) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_pc_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer.  G1 of a tile is paced by its loads; G2 of
    // the tile before becomes possible somewhere in the middle of it (when T1 has written A2 and a D2 buffer is free).
    // So G2 is kept as pending work that every wait of G1 polls for: it is issued the moment it can be, and T2 of a
    // tile overlaps the loads of the next.
    if (lane == 0) {
      const unsigned n1 = static_cast<unsigned>(p.n1_pad), n2 = static_cast<unsigned>(p.n2_blk);
      const unsigned idesc1 = (1u << 4) | ((n1 >> 3) << 17) | ((128u >> 4) << 24);
      const unsigned idesc2 = (1u << 4) | ((n2 >> 3) << 17) | ((128u >> 4) << 24);
      const unsigned a_lbo = kRows * 16u, b1_lbo = n1 * 16u, b2_lbo = n2 * 16u;
      const unsigned long long a_step = static_cast<unsigned long long>((2u * a_lbo) >> 4);
      const unsigned long long b1_step = static_cast<unsigned long long>((2u * b1_lbo) >> 4);
      const unsigned long long b2_step = static_cast<unsigned long long>((2u * b2_lbo) >> 4);
      const int k2_steps = p.n1_pad >> 4;
      unsigned it = 0, w2it = 0, jj = 0;
      int g2_tile = -1, g2_block = 0;  // pending G2: tile (or -1) and its next block
      bool g2_a2_ready = false;
      // issues the pending G2's blocks for as long as their operands and a D2 buffer are ready; never waits
      auto poll_g2 = [&]() {
        while (g2_tile >= 0) {
          const unsigned buf = static_cast<unsigned>(g2_tile % p.d_bufs), par = static_cast<unsigned>(g2_tile / p.d_bufs) & 1u;
          if (!g2_a2_ready) {
            if (!mbar_try_wait(smem_u32(&hdr->a2_full[buf]), par)) return;
            g2_a2_ready = true;
            PC_EV(g2_tile, 7);
          }
          const unsigned slot = p.w2_resident ? static_cast<unsigned>(g2_block) : w2it % p.w2_slots;
          const unsigned wpar = p.w2_resident ? 0u : (w2it / p.w2_slots) & 1u;
          if (!mbar_try_wait(smem_u32(&hdr->w2_full[slot]), wpar)) return;
          if (!mbar_try_wait(smem_u32(&hdr->d2_empty[jj & 1u]), ((jj >> 1) & 1u) ^ 1u)) return;
          tc_fence_after();
          unsigned long long ad = smem_desc(a2_0 + buf * p.a2_bytes, a_lbo, 128);
          unsigned long long bd = smem_desc(w2_0 + slot * p.w2_pitch, b2_lbo, 128);
          for (int ks = 0; ks < k2_steps; ++ks) {
            umma_f16(tmem_base + p.d2_col0 + (jj & 1u) * n2, ad, bd, idesc2, ks > 0 ? 1u : 0u);
            ad += a_step;
            bd += b2_step;
          }
          if (!p.w2_resident) {
            umma_commit(smem_u32(&hdr->w2_empty[slot]));
            ++w2it;
          }
          // the accumulator's commit comes last: T2 waits for it, so no arrival is pending when the CTA leaves
          if (g2_block == p.n2_blocks - 1) umma_commit(smem_u32(&hdr->a2_empty[buf]));
          umma_commit(smem_u32(&hdr->d2_full[jj & 1u]));
          ++jj;
          if (++g2_block == p.n2_blocks) {
            PC_EV(g2_tile, 8);
            g2_tile = -1;
          }
        }
      };
      // bounded wait that keeps issuing the pending G2 while it polls
      auto wait_polling = [&](unsigned bar, unsigned parity) -> bool {
        if (mbar_try_wait(bar, parity)) return true;
        const unsigned long long t0 = global_timer_ns();
        for (unsigned spin = 0;; ++spin) {
          poll_g2();
          if (mbar_try_wait(bar, parity)) return true;
          if ((spin & 63u) != 63u) continue;
          if (*abort_flag) return false;
          if (global_timer_ns() - t0 > p.timeout_ns) {
            atomicOr(&g_pc_error, kErrMma);
            *abort_flag = 1u;
            return false;
          }
        }
      };
      // the pending G2 to its end
      auto finish_g2 = [&]() -> bool {
        const unsigned long long t0 = global_timer_ns();
        for (unsigned spin = 0; g2_tile >= 0; ++spin) {
          poll_g2();
          if (g2_tile < 0) break;
          if ((spin & 63u) != 63u) continue;
          if (*abort_flag) return false;
          if (global_timer_ns() - t0 > p.timeout_ns) {
            atomicOr(&g_pc_error, kErrMma);
            *abort_flag = 1u;
            return false;
          }
        }
        return true;
      };
      bool ok = true;
      for (int i = 0; i < my_tiles && ok; ++i) {
        // G1 of tile i: its accumulator must have been read out by T1 (of tile i - d_bufs)
        const unsigned buf = static_cast<unsigned>(i % p.d_bufs), par = static_cast<unsigned>(i / p.d_bufs) & 1u;
        if (!wait_polling(smem_u32(&hdr->d1_empty[buf]), par ^ 1u)) break;
        tc_fence_after();
        PC_EV(i, 2);
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned st = it % p.land, ophase = (it / p.land) & 1u;
          const unsigned ws = it % p.w1_stages, wphase = (it / p.w1_stages) & 1u;
          // (polling the pending G2 here as well, chunk ready or not, starts T2 three microseconds earlier but gains
          // nothing: while T2's stores run, the rearranging warps' shared-memory traffic waits behind them and G1 of
          // the next tile takes that much longer - MobileNetV2 batch 256 1.5446 -> 1.5508 ms)
          if (!wait_polling(smem_u32(&hdr->op_full[st]), ophase) || !wait_polling(smem_u32(&hdr->w1_full[ws]), wphase)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (c == 0) PC_EV(i, 3);

          unsigned long long ad = smem_desc(land0 + st * kABytes, a_lbo, 128);
          unsigned long long bd = smem_desc(w1_0 + ws * p.w1_bytes, b1_lbo, 128);
#pragma unroll
          for (int ks = 0; ks < kKc / 4; ++ks) {
            umma_f16(tmem_base + buf * n1, ad, bd, idesc1, (c > 0 || ks > 0) ? 1u : 0u);
            ad += a_step;
            bd += b1_step;
          }
          umma_commit(smem_u32(&hdr->land_empty[st]));
          umma_commit(smem_u32(&hdr->w1_empty[ws]));

        }
        if (!ok) break;
        umma_commit(smem_u32(&hdr->d1_full[buf]));
        PC_EV(i, 4);
        // G2 of tile i becomes the pending work; the one before it must be through (it almost always is)
        if (!finish_g2()) break;
        g2_tile = i;
        g2_block = 0;
        g2_a2_ready = false;
      }
      if (ok) finish_g2();
    }
  } else if (warp < kFirstT1) {
    // ------------------------------------------------------------ X chunks: landing layout -> operand layout, in place
    // landed: [slice][pixel] 8-byte pixel-slices; operand: [K group of 8 channels][pixel] 16-byte rows.  Both are 16 KB;
    // a thread's four rows lie where other threads' pixel-slices landed, so all 128 threads read before any writes.
    const int row = threadIdx.x - 32 * kFirstLoad;  // 0 .. 127: row of the tile
    unsigned it = 0;
    bool ok = true;
    for (int i = 0; i < my_tiles && ok; ++i) {
      for (int c = 0; c < p.n_chunks; ++c, ++it) {
        const unsigned st = it % p.land, lphase = (it / p.land) & 1u;
        if (!mbar_wait_warp(smem_u32(&hdr->land_full[st]), lphase, abort_flag, p.timeout_ns, &g_pc_error, kErrLoad)) ok = false;
        const unsigned base = land0 + st * kABytes;
        unsigned v[kKc][2];
#pragma unroll
        for (int sl = 0; sl < kKc; ++sl)
          asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v[sl][0]), "=r"(v[sl][1]) : "r"(base + static_cast<unsigned>(sl) * (kRows * 8u) + static_cast<unsigned>(row) * 8u) : "memory");
        // the barrier also carries the outcome of the wait, so that all four warps leave together if one gave up
        unsigned all_ok;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(all_ok)
            : "r"(ok ? 1u : 0u), "n"(32 * kLoadWarps)
            : "memory");
        if (!all_ok) {
          ok = false;
          break;
        }

#pragma unroll
        for (int kg = 0; kg < kKc / 2; ++kg)
          st_shared_v4(base + static_cast<unsigned>(kg) * (kRows * 16u) + static_cast<unsigned>(row) * 16u, v[2 * kg][0], v[2 * kg][1], v[2 * kg + 1][0], v[2 * kg + 1][1]);
        // visible to the tensor core's proxy, then count this warp in
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->op_full[st]));

      }
    }
  } else if (warp < kFirstT2) {
    // ------------------------------------------------------------ T1: D1 -> first output (global) and A2 (shared)
    const int quarter = warp & 3;
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int row = quarter * 32 + lane;
    const int groups = p.n1_pad >> 4;
    const size_t slice_stride = static_cast<size_t>(p.m_total) * 4;
    // The residual of a tile does not depend on its MMAs: every thread copies its own pixel's residual (one 8-byte
    // pixel-slice per slice) into a private strip of shared memory while G1 of that tile runs, and reads it back
    // after its own copies have landed - no other thread touches the strip, so no barrier is needed.  Fetched
    // where it is used instead, the loads' latency (a microsecond and more each, one group after the other) was the
    // longest step of a tile.
    const unsigned res_row = smem0 + p.off_res + static_cast<unsigned>(row) * 8u;
    auto prefetch_residual = [&](int i) {
      const unsigned pixel = (blockIdx.x + static_cast<unsigned>(i) * gridDim.x) * kRows + static_cast<unsigned>(row);
      if (pixel < p.m_total)
        for (int s = 0; s < p.s_mid; ++s)
          cp_async8_zfill(res_row + static_cast<unsigned>(s) * (kRows * 8u), p.res + (static_cast<size_t>(s) * p.m_total + pixel) * 4, 8u);
      cp_async_commit();
    };
    pdl_wait();  // the residual is read and the output written only below
    if (p.has_res && my_tiles > 0) prefetch_residual(0);
    for (int i = 0; i < my_tiles; ++i) {
      const unsigned buf = static_cast<unsigned>(i % p.d_bufs), par = static_cast<unsigned>(i / p.d_bufs) & 1u;
      if (!mbar_wait_warp(smem_u32(&hdr->d1_full[buf]), par, abort_flag, p.timeout_ns, &g_pc_error, kErrDrain)) break;
      // A2[buf] is free once G2 of the tile that used it last has run
      if (!mbar_wait_warp(smem_u32(&hdr->a2_empty[buf]), par ^ 1u, abort_flag, p.timeout_ns, &g_pc_error, kErrDrain)) break;
      tc_fence_after();
      if (warp == kFirstT1 && lane == 0) PC_EV(i, 5);
      const unsigned tile = blockIdx.x + static_cast<unsigned>(i) * gridDim.x;
      const unsigned pixel = tile * kRows + static_cast<unsigned>(row);
      const bool px_ok = pixel < p.m_total;
      const unsigned a2_row = a2_0 + buf * p.a2_bytes + static_cast<unsigned>(row) * 16u;
      if (p.has_res) cp_async_wait_pending<0>();
      const unsigned d1_addr = tmem_base + lane_bits + buf * static_cast<unsigned>(p.n1_pad);
      // sixteen accumulator columns = four slices: bias, (activation,) residual, (activation,) fp16; stored as the first
      // operator's output and as two 16-byte rows of the second MMA's operand
      auto finish_group = [&](const unsigned (&r)[16], int g) {
        unsigned o[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint2 rq = make_uint2(0u, 0u);
          if (p.has_res && px_ok && g * 4 + j < p.s_mid)
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(rq.x), "=r"(rq.y) : "r"(res_row + static_cast<unsigned>(g * 4 + j) * (kRows * 8u)) : "memory");
          const float4 b = *reinterpret_cast<const float4*>(sbias + g * 16 + j * 4);
          const float2 q0 = __half22float2(*reinterpret_cast<const __half2*>(&rq.x));
          const float2 q1 = __half22float2(*reinterpret_cast<const __half2*>(&rq.y));
          if (LINEAR1) {
            const float2 v0 = __fadd2_rn(__fadd2_rn(make_float2(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1])), make_float2(b.x, b.y)), q0);
            const float2 v1 = __fadd2_rn(__fadd2_rn(make_float2(__uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])), make_float2(b.z, b.w)), q1);
            o[2 * j] = pack_f16x2<false>(v0.x, v0.y);
            o[2 * j + 1] = pack_f16x2<false>(v1.x, v1.y);
          } else {
            const float v0 = act1(act1(__uint_as_float(r[4 * j]) + b.x, p.act1_pre) + q0.x, p.act1_post);
            const float v1 = act1(act1(__uint_as_float(r[4 * j + 1]) + b.y, p.act1_pre) + q0.y, p.act1_post);
            const float v2 = act1(act1(__uint_as_float(r[4 * j + 2]) + b.z, p.act1_pre) + q1.x, p.act1_post);
            const float v3 = act1(act1(__uint_as_float(r[4 * j + 3]) + b.w, p.act1_pre) + q1.y, p.act1_post);
            o[2 * j] = pack_f16x2<false>(v0, v1);
            o[2 * j + 1] = pack_f16x2<false>(v2, v3);
          }
          if (px_ok && g * 4 + j < p.s_mid)
            *reinterpret_cast<uint2*>(p.out1 + static_cast<size_t>(g * 4 + j) * slice_stride + static_cast<size_t>(pixel) * 4) =
                make_uint2(o[2 * j], o[2 * j + 1]);
        }
        st_shared_v4(a2_row + static_cast<unsigned>(2 * g) * (kRows * 16u), o[0], o[1], o[2], o[3]);
        st_shared_v4(a2_row + static_cast<unsigned>(2 * g + 1) * (kRows * 16u), o[4], o[5], o[6], o[7]);
      };
      // the next group's tensor-memory load is in flight while this group is finished
      unsigned ra[16], rb[16];
      tmem_ld16(d1_addr, ra);
      for (int g = 0; g < groups; g += 2) {
        tmem_ld_wait16(ra);
        if (g + 1 < groups) tmem_ld16(d1_addr + static_cast<unsigned>((g + 1) * 16), rb);
        finish_group(ra, g);
        if (g + 1 >= groups) break;
        tmem_ld_wait16(rb);
        if (g + 2 < groups) tmem_ld16(d1_addr + static_cast<unsigned>((g + 2) * 16), ra);
        finish_group(rb, g + 1);
      }
      tc_fence_before();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&hdr->d1_empty[buf]));
        mbar_arrive(smem_u32(&hdr->a2_full[buf]));
        if (warp == kFirstT1) PC_EV(i, 6);
        PC_EV(i, 11 + (warp - kFirstT1));
      }
      // the strip has been read: the next tile's residual may overwrite it
      if (p.has_res && i + 1 < my_tiles) prefetch_residual(i + 1);
    }
  } else {
    // ------------------------------------------------------------ T2: D2 blocks -> second output
    const int dw = warp - kFirstT2;
    const int quarter = warp & 3, sub = dw >> 2;  // TMEM lane quarter; index among the three warps sharing it
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int groups = p.n2_blk >> 4;
    const float* sb2 = sbias + p.n1_pad;
    const size_t slice_stride = static_cast<size_t>(p.m_total) * 4;
    pdl_wait();
    unsigned jj = 0;
    bool ok = true;
    for (int i = 0; i < my_tiles && ok; ++i) {
      const unsigned tile = blockIdx.x + static_cast<unsigned>(i) * gridDim.x;
      const unsigned pixel = tile * kRows + static_cast<unsigned>(quarter * 32 + lane);
      const bool px_ok = pixel < p.m_total;
      for (int j = 0; j < p.n2_blocks; ++j, ++jj) {
        const unsigned b = jj & 1u;
        if (!mbar_wait_warp(smem_u32(&hdr->d2_full[b]), (jj >> 1) & 1u, abort_flag, p.timeout_ns, &g_pc_error, kErrDrain)) {
          ok = false;
          break;
        }
        tc_fence_after();
        if (warp == kFirstT2 && lane == 0 && j == 0) PC_EV(i, 9);
        const unsigned d2_addr = tmem_base + lane_bits + p.d2_col0 + b * static_cast<unsigned>(p.n2_blk);
        auto finish_group = [&](const unsigned (&r)[16], int g) {
          const int ch0 = j * p.n2_blk + g * 16;
          const int so0 = ch0 >> 2;
          __half* dst = p.out2 + static_cast<size_t>(so0) * slice_stride + static_cast<size_t>(pixel) * 4;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (so0 + q >= p.s_out || !px_ok) continue;
            const float4 bb = *reinterpret_cast<const float4*>(sb2 + ch0 + q * 4);
            const float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1])), make_float2(bb.x, bb.y));
            const float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3])), make_float2(bb.z, bb.w));
            uint2 o;
            // the conversion clamps at zero itself; clamping at 6 after the rounding equals rounding after the clamp
            o.x = pack_f16x2<ACT2 != GI_ACT_NONE>(v0.x, v0.y);
            o.y = pack_f16x2<ACT2 != GI_ACT_NONE>(v1.x, v1.y);
            if (ACT2 == GI_ACT_RELU6) {
              const __half2 six = __float2half2_rn(6.f);
              const __half2 h0 = __hmin2(*reinterpret_cast<const __half2*>(&o.x), six), h1 = __hmin2(*reinterpret_cast<const __half2*>(&o.y), six);
              o.x = *reinterpret_cast<const unsigned*>(&h0);
              o.y = *reinterpret_cast<const unsigned*>(&h1);
            }
            *reinterpret_cast<uint2*>(dst + q * slice_stride) = o;
          }
        };
        // the next group's tensor-memory load is in flight while this group is finished
        constexpr int kStep = kT2Warps / 4;
        unsigned ra[16], rb[16];
        if (sub < groups) tmem_ld16(d2_addr + static_cast<unsigned>(sub * 16), ra);
        for (int g = sub; g < groups; g += 2 * kStep) {
          tmem_ld_wait16(ra);
          if (g + kStep < groups) tmem_ld16(d2_addr + static_cast<unsigned>((g + kStep) * 16), rb);
          finish_group(ra, g);
          if (g + kStep >= groups) break;
          tmem_ld_wait16(rb);
          if (g + 2 * kStep < groups) tmem_ld16(d2_addr + static_cast<unsigned>((g + 2 * kStep) * 16), ra);
          finish_group(rb, g + kStep);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->d2_empty[b]));
        if (warp == kFirstT2 && lane == 0 && j == p.n2_blocks - 1) PC_EV(i, 10);
      }
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

struct Tiling {
  int s_in, s_mid, s_out, n_chunks, n1_pad, n2_blk, n2_blocks, d_bufs, land, w1_stages, w2_slots, w2_resident;
  unsigned w1_bytes, w2_bytes, w2_pitch, a2_bytes, off_res, off_a2, off_w2, off_w1, off_land, d2_col0;
  size_t smem;
  bool ok;
};

// One tiling attempt with `d_bufs` buffers of D1 / A2; `has_res`: the first operator has a residual input (its strips
// take shared memory).
Tiling try_tiling(int cin, int cmid, int cout, bool has_res, int d_bufs) {
  Tiling t{};
  t.ok = false;
  if (cin <= 0 || cmid <= 0 || cout <= 0) return t;
  t.s_in = slices(cin);
  t.s_mid = slices(cmid);
  t.s_out = slices(cout);
  t.n_chunks = (t.s_in + kKc - 1) / kKc;
  t.n1_pad = (cmid + 15) / 16 * 16;
  if (t.n1_pad > 256) return t;
  // tensor memory: D1 (one or two buffers of n1_pad columns) and two D2 buffers of n2_blk columns
  t.d_bufs = d_bufs;
  int max_blk = (512 - d_bufs * t.n1_pad) / 2 / 16 * 16;
  if (max_blk > 256) max_blk = 256;
  if (max_blk < (d_bufs == 2 ? 96 : 16)) return t;
  const int n2_pad = (cout + 15) / 16 * 16;
  t.n2_blocks = (n2_pad + max_blk - 1) / max_blk;
  t.n2_blk = ((n2_pad + t.n2_blocks - 1) / t.n2_blocks + 15) / 16 * 16;
  t.d2_col0 = static_cast<unsigned>(t.d_bufs * t.n1_pad);
  t.w1_bytes = static_cast<unsigned>(t.n1_pad) * kKc * 8u;  // n1_pad rows x 64 channels x 2 bytes
  t.w2_bytes = static_cast<unsigned>(t.n2_blk) * static_cast<unsigned>(t.n1_pad) * 2u;
  t.w2_pitch = (t.w2_bytes + 1023u) / 1024u * 1024u;
  t.a2_bytes = static_cast<unsigned>(kRows) * static_cast<unsigned>(t.n1_pad) * 2u;
  const unsigned bias_bytes = (static_cast<unsigned>(t.n1_pad + t.n2_blocks * t.n2_blk) * 4u + 1023u) / 1024u * 1024u;
  t.off_res = kHeader + bias_bytes;  // the residual strips: one 8-byte pixel-slice per slice and row
  t.off_a2 = t.off_res + (has_res ? static_cast<unsigned>(t.s_mid) * kRows * 8u : 0u);
  t.off_w2 = t.off_a2 + static_cast<unsigned>(t.d_bufs) * t.a2_bytes;
  const long long avail = static_cast<long long>(kSmemMax) - t.off_w2;
  // the least the two G1 rings need: two W1 stages and kMinLand landing stages
  const long long min_rings = 2LL * t.w1_bytes + static_cast<long long>(kMinLand) * kABytes;
  // all W2 blocks resident if that still leaves rings of some depth, else two slots that follow the tiles
  if (t.n2_blocks <= kMaxW2Slots && avail - static_cast<long long>(t.n2_blocks) * t.w2_pitch >= 2 * min_rings) {
    t.w2_resident = 1;
    t.w2_slots = t.n2_blocks;
  } else {
    t.w2_resident = 0;
    t.w2_slots = 2;
    if (avail - 2LL * t.w2_pitch < min_rings) return t;
  }
  t.off_w1 = t.off_w2 + static_cast<unsigned>(t.w2_slots) * t.w2_pitch;
  long long left = static_cast<long long>(kSmemMax) - t.off_w1;
  // W1 ring: up to four stages first, then the landing ring, then what is left goes to W1 again
  int w1 = static_cast<int>((left - static_cast<long long>(kMinLand) * kABytes) / t.w1_bytes);
  if (w1 > 4) w1 = 4;
  if (w1 > t.n_chunks) w1 = t.n_chunks < 2 ? 2 : t.n_chunks;
  if (w1 < 2) return t;
  long long land = (left - static_cast<long long>(w1) * t.w1_bytes) / kABytes;
  if (land > kMaxLand) land = kMaxLand;
  left -= land * kABytes;
  while (w1 < kMaxW1 && w1 < t.n_chunks && left - static_cast<long long>(w1 + 1) * t.w1_bytes >= 0) ++w1;
  t.w1_stages = w1;
  t.land = static_cast<int>(land);
  t.off_land = t.off_w1 + static_cast<unsigned>(w1) * t.w1_bytes;
  t.smem = t.off_land + static_cast<size_t>(t.land) * kABytes;
  t.ok = t.land >= kMinLand;
  return t;
}

Tiling choose_tiling(int cin, int cmid, int cout, bool has_res) {
  const Tiling t = try_tiling(cin, cmid, cout, has_res, 2);
  return t.ok ? t : try_tiling(cin, cmid, cout, has_res, 1);
}

}  // namespace

bool pointwise_chain_supported(int cin, int cmid, int cout, bool has_res) { return choose_tiling(cin, cmid, cout, has_res).ok; }

// First operator: dense weights as the B operand per K chunk, [8 K groups][n1_pad rows][8 halves].  Second operator:
// per block of output channels [n1_pad / 8 K groups][n2_blk rows][8 halves].  Entries beyond the real channels are
// zero, and so are the padded biases, so padded columns of both accumulators hold exact zeros.
void pointwise_chain_pack(const float* w1, const float* b1, const float* w2, const float* b2, int cin, int cmid, int cout,
                          std::vector<uint8_t>* blob, LaunchRec* r) {
  const Tiling t = choose_tiling(cin, cmid, cout, r->ep.has_res != 0);
  const size_t w1_total = static_cast<size_t>(t.n_chunks) * t.w1_bytes, w2_total = static_cast<size_t>(t.n2_blocks) * t.w2_bytes;
  const uint64_t off1 = round_up_u64(blob->size(), 256);
  blob->resize(off1 + w1_total, 0);
  const uint64_t off2 = round_up_u64(blob->size(), 256);
  blob->resize(off2 + w2_total, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(t.n1_pad + t.n2_blocks * t.n2_blk) * sizeof(float), 0);
  uint16_t* p1 = reinterpret_cast<uint16_t*>(blob->data() + off1);
  uint16_t* p2 = reinterpret_cast<uint16_t*>(blob->data() + off2);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cmid; ++co) {
    bp[co] = b1[co];
    for (int ci = 0; ci < cin; ++ci) {
      const int chunk = ci / (kKc * 4), k = ci % (kKc * 4);
      uint16_t* base = p1 + static_cast<size_t>(chunk) * (t.w1_bytes / 2);
      base[(static_cast<size_t>(k / 8) * t.n1_pad + co) * 8 + k % 8] = f32_to_f16_rne(w1[static_cast<size_t>(co) * cin + ci]);
    }
  }
  for (int co = 0; co < cout; ++co) {
    const int blk = co / t.n2_blk, row = co % t.n2_blk;
    bp[t.n1_pad + co] = b2[co];
    uint16_t* base = p2 + static_cast<size_t>(blk) * (t.w2_bytes / 2);
    for (int ci = 0; ci < cmid; ++ci)
      base[(static_cast<size_t>(ci / 8) * t.n2_blk + row) * 8 + ci % 8] = f32_to_f16_rne(w2[static_cast<size_t>(co) * cmid + ci]);
  }
  r->wts = Loc{W_WEIGHTS, 0, off1};
  r->wts2 = Loc{W_WEIGHTS, 0, off2};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = w1_total + w2_total;
  r->tc_nt = t.n2_blk;
  r->tc_kc = kKc;
  r->tc_stages = t.land;
}

int launch_pointwise_chain(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream) {
  const Tiling t = choose_tiling(r.C, r.Cmid, r.Co2, r.ep.has_res != 0);
  if (!t.ok || !p.out2) return static_cast<int>(cudaErrorInvalidValue);
  PcParams k{};
  k.in = static_cast<const __half*>(p.in0);
  k.res = static_cast<const __half*>(p.res);
  k.out1 = static_cast<__half*>(p.out);
  k.out2 = static_cast<__half*>(p.out2);
  k.w1 = static_cast<const unsigned char*>(p.wts);
  k.w2 = static_cast<const unsigned char*>(p.wts2);
  k.bias = static_cast<const float*>(p.bias);
  k.m_total = static_cast<unsigned>(r.B) * static_cast<unsigned>(plane_pixels(r.H, r.W));
  k.m_tiles = static_cast<int>((k.m_total + kRows - 1) / kRows);
  k.s_in = t.s_in;
  k.s_mid = t.s_mid;
  k.s_out = t.s_out;
  k.n_chunks = t.n_chunks;
  k.n1_pad = t.n1_pad;
  k.n2_blk = t.n2_blk;
  k.n2_blocks = t.n2_blocks;
  k.d_bufs = t.d_bufs;
  k.land = t.land;
  k.w1_stages = t.w1_stages;
  k.in_dead = r.in0_dead;
  k.w2_slots = t.w2_slots;
  k.w2_resident = t.w2_resident;
  k.w1_bytes = t.w1_bytes;
  k.w2_bytes = t.w2_bytes;
  k.w2_pitch = t.w2_pitch;
  k.a2_bytes = t.a2_bytes;
  k.off_res = t.off_res;
  k.off_a2 = t.off_a2;
  k.off_w2 = t.off_w2;
  k.off_w1 = t.off_w1;
  k.off_land = t.off_land;
  k.d2_col0 = t.d2_col0;
  k.act1_pre = r.ep.act_pre;
  k.has_res = r.ep.has_res;
  k.act1_post = r.ep.act_post;
  k.timeout_ns = 1000000000u;
  static bool attr_done_dev[kMaxDevices] = {};
  bool& attr_done = attr_done_dev[current_device_slot()];
  if (!attr_done) {
    cudaError_t e = cudaSuccess;
#define GI_PC_ATTR(A, L) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(pointwise_chain_kernel<A, L>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax)
    GI_PC_ATTR(GI_ACT_NONE, false);
    GI_PC_ATTR(GI_ACT_RELU, false);
    GI_PC_ATTR(GI_ACT_RELU6, false);
    GI_PC_ATTR(GI_ACT_NONE, true);
    GI_PC_ATTR(GI_ACT_RELU, true);
    GI_PC_ATTR(GI_ACT_RELU6, true);
#undef GI_PC_ATTR
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
  const int sms = device_sm_count();
  const unsigned grid = static_cast<unsigned>(k.m_tiles < sms ? k.m_tiles : sms);
  // the kernel reserves all of tensor memory: ask for enough shared memory that no second CTA shares the SM
  size_t smem = t.smem;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int act2 = r.ep2.act_pre;
  const bool linear1 = k.act1_pre == GI_ACT_NONE && k.act1_post == GI_ACT_NONE;
#define GI_PC_LAUNCH(A, L) launch_pdl(pointwise_chain_kernel<A, L>, grid, kThreads, smem, st, tmap, k)
  if (linear1) {
    if (act2 == GI_ACT_RELU6) GI_PC_LAUNCH(GI_ACT_RELU6, true);
    else if (act2 == GI_ACT_RELU) GI_PC_LAUNCH(GI_ACT_RELU, true);
    else GI_PC_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (act2 == GI_ACT_RELU6) GI_PC_LAUNCH(GI_ACT_RELU6, false);
    else if (act2 == GI_ACT_RELU) GI_PC_LAUNCH(GI_ACT_RELU, false);
    else GI_PC_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_PC_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

#ifdef GI_TRACE
int pointwise_chain_trace(unsigned long long* dst, int n) {
  const size_t bytes = sizeof(unsigned long long) * (n < 256 * 64 ? n : 256 * 64);
  return static_cast<int>(cudaMemcpyFromSymbol(dst, g_pc_trace, bytes));
}
#endif

unsigned int pointwise_chain_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_pc_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
