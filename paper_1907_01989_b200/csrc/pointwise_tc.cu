// Pointwise (1x1) convolution on the 5th-generation tensor cores: tcgen05.mma with the
// accumulator in tensor memory, operands fed by TMA, fused bias / activation / residual
// epilogue.  This is the "specialised 1x1 convolution" of Section 3.2, rebuilt for sm_100a.
//
// The channel-sliced layout stores 4 channels (8 bytes) per pixel-slice, while the tensor
// core wants 16 contiguous bytes along K.  Two neighbouring pixels of one slice are 16
// contiguous bytes, so a plane is read as rows of "pixel pairs":
//     A'[r][s*8 + p*4 + c] = x[pixel 2r+p][channel 4s+c]           (r: pair, p: parity)
// which is exactly the canonical K-major, no-swizzle operand layout (8 rows x 16 bytes per core
// matrix) and can be copied by TMA with no repacking.  The weights are expanded at compile
// time into B'[so*8 + p'*4 + j][s*8 + p*4 + c] = (p == p') ? w[4so+j][4s+c] : 0, so that
//     D'[r][so*8 + p'*4 + j] = y[pixel 2r+p'][channel 4so+j],
// i.e. 8 consecutive fp32 accumulator columns of one lane are the 16 output bytes of a pixel
// pair in one output slice.  Half of the multiplies hit structural zeros; these layers are
// bound by HBM bandwidth, not by the tensor pipe, so the pipe has the slack.
//
// Two CTAs per SM, persistent over (pixel tile, output-channel tile) units; warp 0 issues TMA,
// warp 1 issues MMAs and owns tensor memory, warps 2-9 run the epilogue: two warps per TMEM
// lane quarter, each taking every second 16-column chunk and loading the next chunk from tensor
// memory while it converts and stores the current one.  Two accumulators per CTA live in tensor
// memory, so the epilogue of a tile overlaps the loads and MMAs of the next one.  (One layer
// shape - very few input channels, 17-32 output slices - runs as one wide CTA per SM with four
// epilogue warps per quarter instead.)  Every wait is bounded: after about a second it raises an
// error word the host can read, drains the copies in flight and leaves, so the context stays usable.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>
#include <vector>

#include "kernels.h"
#include "pdl.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace gi {
namespace {

constexpr int kTileRows = 128;               // pixel pairs (TMEM lanes) per tile
constexpr int kTilePx = 2 * kTileRows;       // pixels per tile
constexpr int kSliceBytes = kTileRows * 16;  // one input slice of a tile in shared memory
constexpr int kCoreBytes = 128;              // one 8x8 fp16 core matrix
constexpr int kMaxStages = 8;
constexpr int kMaxAcc = 8;                   // narrow tiles are short: more of them must be in flight
constexpr int kMaxNts = 16;                  // output slices per tile: 16 * 8 = 128 accumulator columns, two
                                             // buffers per CTA, two CTAs per SM = all 512 TMEM columns
constexpr int kSmemHeader = 1024;            // barriers, TMEM address, abort flag
constexpr int kSmemBudget = 200 * 1024;
constexpr int kEpiWarpsPerQuarter = 4;       // epilogue warps sharing one TMEM lane quarter (at most)
constexpr int kEpiWarps = 4 * kEpiWarpsPerQuarter;
constexpr int kThreads = 64 + 32 * kEpiWarps;

__device__ unsigned int g_tc_error = 0;  // sticky: non-zero once any wait in this module timed out

struct TcParams {
  const __half* res;
  __half* out;
  const float* bias;
  const unsigned char* wts;
  unsigned int m_total_px;  // batch * pixels per stored plane (even)
  int s_out;                // real output slices
  int nts, n_tiles;         // output slices per tile (even), number of such tiles
  int kc, k_chunks;         // input slices per pipeline stage (even), stages per tile
  int stages;
  int m_tiles, groups;      // pixel tiles; each pixel tile is split over `groups` CTAs along n_tiles
  int act_pre, has_res, act_post;
  int in_dead;              // the input is not read again: its TMA loads carry the evict-first L2 hint
  unsigned int tmem_cols;   // power of two >= n_acc * nts * 8
  unsigned int n_acc;       // accumulator buffers in tensor memory (power of two, 2..8): tiles in flight
  int epq;                  // epilogue warps per TMEM lane quarter (1, 2 or 4); blockDim = 64 + 128 * epq
  unsigned int timeout_ns;
};

using namespace ptx;

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

struct SmemHeader {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long acc_full[kMaxAcc];
  unsigned long long acc_empty[kMaxAcc];
  unsigned tmem_addr;
  unsigned abort_flag;
};
static_assert(sizeof(SmemHeader) <= kSmemHeader, "header too large");

enum : unsigned { kErrProducer = 1u, kErrMma = 2u, kErrEpilogue = 4u, kErrDrain = 8u };

// ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow
template <int ACT, bool TAIL>
__global__ void __launch_bounds__(kThreads, 1) pointwise_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned stage_a_bytes = static_cast<unsigned>(p.kc) * kSliceBytes;
  const unsigned stage_b_bytes = static_cast<unsigned>(p.kc) * p.nts * kCoreBytes;
  const unsigned stage_bytes = stage_a_bytes + stage_b_bytes;
  const unsigned data0 = smem_u32(smem + kSmemHeader);
  volatile unsigned* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_a);
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->full[i]), 1);
      mbar_init(smem_u32(&hdr->empty[i]), 1);
    }
    for (unsigned i = 0; i < p.n_acc; ++i) {
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), 4 * p.epq);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // the prologue above touched only on-chip state; activations are read and written after the wait
  pdl_launch_dependents();
  pdl_wait();
  const unsigned tmem_base = hdr->tmem_addr;
  const int n_units = p.m_tiles * p.groups;
  const unsigned acc_cols = static_cast<unsigned>(p.nts) * 8u;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      const unsigned long long evict_first = policy_evict_first();
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const int m_tile = u / p.groups, grp = u - m_tile * p.groups;
        for (int nt = grp; nt < p.n_tiles && ok; nt += p.groups) {
          for (int kc_i = 0; kc_i < p.k_chunks; ++kc_i, ++it) {
            const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
            if (!mbar_wait(smem_u32(&hdr->empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_tc_error, kErrProducer)) {
              ok = false;
              break;
            }
            const unsigned full = smem_u32(&hdr->full[stage]);
            mbar_expect_tx(full, stage_bytes);
            const unsigned dst = data0 + stage * stage_bytes;
            // pixels outside the tensor and slices beyond the last one arrive as zeros
            if (p.in_dead) tma_load_2d_hint(dst, &tmap_a, m_tile * kTilePx, kc_i * p.kc, full, evict_first);
            else tma_load_2d(dst, &tmap_a, m_tile * kTilePx, kc_i * p.kc, full);
            bulk_load(dst + stage_a_bytes, p.wts + (static_cast<size_t>(nt) * p.k_chunks + kc_i) * stage_b_bytes, stage_b_bytes,
                      full);
          }
        }
      }
      if (!ok) {
        // copies already issued still land in shared memory: wait for them (bounded) before leaving
        const unsigned first = it > static_cast<unsigned>(p.stages) ? it - p.stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->full[j % p.stages]), (j / p.stages) & 1u)) {
            if (global_timer_ns() - t0 > p.timeout_ns) {
              atomicOr(&g_tc_error, kErrDrain);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = nts * 8
      const unsigned idesc = (1u << 4) | ((acc_cols >> 3) << 17) | ((kTileRows >> 4) << 24);
      const unsigned b_lbo = static_cast<unsigned>(p.nts) * kCoreBytes;
      unsigned it = 0, tile = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const int m_tile = u / p.groups, grp = u - m_tile * p.groups;
        for (int nt = grp; nt < p.n_tiles && ok; nt += p.groups, ++tile) {
          const unsigned acc = tile % p.n_acc, acc_phase = (tile / p.n_acc) & 1u;
          if (!mbar_wait(smem_u32(&hdr->acc_empty[acc]), acc_phase ^ 1u, abort_flag, p.timeout_ns, &g_tc_error, kErrMma)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const unsigned d_tmem = tmem_base + acc * acc_cols;
          for (int kc_i = 0; kc_i < p.k_chunks; ++kc_i, ++it) {
            const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
            if (!mbar_wait(smem_u32(&hdr->full[stage]), phase, abort_flag, p.timeout_ns, &g_tc_error, kErrMma)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const unsigned a_base = data0 + stage * stage_bytes, b_base = a_base + stage_a_bytes;
            // descriptors built once per stage and advanced by adds: the issuing thread's own
            // instruction stream is what bounds short tiles
            unsigned long long ad = smem_desc(a_base, kSliceBytes, kCoreBytes), bd = smem_desc(b_base, b_lbo, kCoreBytes);
            const unsigned long long ad_step = static_cast<unsigned long long>((2u * kSliceBytes) >> 4);
            const unsigned long long bd_step = static_cast<unsigned long long>((2u * b_lbo) >> 4);
            umma_f16(d_tmem, ad, bd, idesc, kc_i > 0 ? 1u : 0u);
            for (int ks = 1; ks < p.kc / 2; ++ks) {
              ad += ad_step;
              bd += bd_step;
              umma_f16(d_tmem, ad, bd, idesc, 1u);
            }
            umma_commit(smem_u32(&hdr->empty[stage]));  // the stage is free once these MMAs have read it
          }
          if (ok) umma_commit(smem_u32(&hdr->acc_full[acc]));
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2 .. 1 + 4 * epq)
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int sub = (warp - 2) >> 2;
    const unsigned rows_total = p.m_total_px >> 1;
    const int n_chunks = p.nts >> 1;  // 2 output slices = 16 accumulator columns per chunk
    unsigned tile = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
      const int m_tile = u / p.groups, grp = u - m_tile * p.groups;
      const unsigned row = static_cast<unsigned>(m_tile) * kTileRows + quarter * 32 + lane;
      const bool row_ok = row < rows_total;
      for (int nt = grp; nt < p.n_tiles && ok; nt += p.groups, ++tile) {
        const unsigned acc = tile % p.n_acc, acc_phase = (tile / p.n_acc) & 1u;
        if (!mbar_wait_warp(smem_u32(&hdr->acc_full[acc]), acc_phase, abort_flag, p.timeout_ns, &g_tc_error, kErrEpilogue)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const unsigned t_addr = tmem_base + acc * acc_cols + (static_cast<unsigned>(quarter * 32) << 16);
        const float4* bias4 = reinterpret_cast<const float4*>(p.bias) + static_cast<size_t>(nt) * p.nts;

        // the chunk's bias and residual are fetched together with its accumulator columns, one chunk ahead
        auto issue = [&](unsigned* r, float4* b, uint4* q, int c) {
          tmem_ld16(t_addr + static_cast<unsigned>(c) * 16u, r);
          b[0] = __ldg(bias4 + 2 * c);
          b[1] = __ldg(bias4 + 2 * c + 1);
          if (TAIL) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const int so = nt * p.nts + 2 * c + j;
              q[j] = make_uint4(0u, 0u, 0u, 0u);
              if (p.has_res && so < p.s_out && row_ok)
                q[j] = __ldg(reinterpret_cast<const uint4*>(p.res + (static_cast<size_t>(so) * p.m_total_px + 2u * row) * 4u));
            }
          }
        };
        auto finish = [&](const unsigned* r, const float4* b, const uint4* q, int c) {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int so = nt * p.nts + 2 * c + j;
            if (so >= p.s_out || !row_ok) continue;
            const size_t off = (static_cast<size_t>(so) * p.m_total_px + 2u * row) * 4u;  // in halves
            // columns 8j..8j+7: channels 0-3 of the even pixel, then of the odd pixel; bias per channel
            const float2 b01 = make_float2(b[j].x, b[j].y), b23 = make_float2(b[j].z, b[j].w);
            float2 v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              v[i] = __fadd2_rn(make_float2(__uint_as_float(r[8 * j + 2 * i]), __uint_as_float(r[8 * j + 2 * i + 1])),
                                (i & 1) ? b23 : b01);
            uint4 o;
            __half2* oh = reinterpret_cast<__half2*>(&o);
            if (!TAIL) {
              // the conversion instruction clamps at 0 itself; clamping at 6 after the rounding
              // equals rounding after the clamp because 6 is an fp16 value
              unsigned* ow = reinterpret_cast<unsigned*>(&o);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                ow[i] = pack_f16x2<ACT != GI_ACT_NONE>(v[i].x, v[i].y);
                if (ACT == GI_ACT_RELU6) ow[i] = __vmins2(ow[i], 0x46004600u);  // non-negative fp16 order like integers
              }
            } else {
              const __half2* rh = reinterpret_cast<const __half2*>(&q[j]);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(rh[i]);  // zero when there is no residual
                // the usual tail is the residual sum of a linear projection: no activation on either side of it
                float2 s2 = __fadd2_rn(make_float2(act1(v[i].x, ACT), act1(v[i].y, ACT)), f);
                if (p.act_post != GI_ACT_NONE) {
                  s2.x = act1(s2.x, p.act_post);
                  s2.y = act1(s2.y, p.act_post);
                }
                oh[i] = __floats2half2_rn(s2.x, s2.y);
              }
            }
            *reinterpret_cast<uint4*>(p.out + off) = o;
          }
        };

        unsigned ra[16], rb[16];
        float4 ba[2], bb[2];
        uint4 qa[2], qb[2];
        int c = sub;
        if (c < n_chunks) issue(ra, ba, qa, c);
        for (; c < n_chunks; c += 2 * p.epq) {
          const int c1 = c + p.epq, c2 = c + 2 * p.epq;
          tmem_ld_wait16(ra);
          if (c1 < n_chunks) issue(rb, bb, qb, c1);
          finish(ra, ba, qa, c);
          if (c1 < n_chunks) {
            tmem_ld_wait16(rb);
            if (c2 < n_chunks) issue(ra, ba, qa, c2);
            finish(rb, bb, qb, c1);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[acc]));
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// ------------------------------------------------------------------ host side
struct Tiling {
  int s_in, s_out, kc, k_chunks, nts, n_tiles, stages;
};

Tiling choose_tiling(int cin, int cout) {
  Tiling t;
  t.s_in = slices(cin);
  t.s_out = slices(cout);
  const int s_in_even = (t.s_in + 1) / 2 * 2;
  t.kc = s_in_even < 8 ? s_in_even : 8;
  t.k_chunks = (s_in_even + t.kc - 1) / t.kc;
  // very few input channels and 17-32 output slices (16 -> 96): one wide tile per pixel tile beats
  // two narrow ones (measured 0.131 vs 0.157 ms at 112x112, batch 256); then one CTA per SM
  const int max_nts = (t.s_in <= 4 && t.s_out > kMaxNts && t.s_out <= 2 * kMaxNts) ? 2 * kMaxNts : kMaxNts;
  t.n_tiles = (t.s_out + max_nts - 1) / max_nts;
  t.nts = (t.s_out + t.n_tiles - 1) / t.n_tiles;
  t.nts = (t.nts + 1) / 2 * 2;  // N = nts * 8 must be a multiple of 16
  const int stage_bytes = t.kc * (kSliceBytes + t.nts * kCoreBytes);
  t.stages = kSmemBudget / stage_bytes;
  if (t.stages > kMaxStages) t.stages = kMaxStages;
  if (t.stages < 2) t.stages = 2;
  return t;
}

struct DeviceInfo {
  int sms = 0;
  bool attr_set = false;
};
DeviceInfo& device_info() {
  static DeviceInfo info[64];
  int dev = 0;
  cudaGetDevice(&dev);
  return info[dev & 63];
}

}  // namespace

bool pointwise_tc_supported(int cin, int cout) { return cin > 0 && cout > 0; }

// Expanded weights, per (output tile, K chunk): [kc input slices][nts output slices][8 rows x 8 halves],
// row = parity' * 4 + output channel in slice, column = parity * 4 + input channel in slice.
void pointwise_tc_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Tiling t = choose_tiling(cin, cout);
  const size_t chunk_bytes = static_cast<size_t>(t.kc) * t.nts * kCoreBytes;
  const size_t wbytes = static_cast<size_t>(t.n_tiles) * t.k_chunks * chunk_bytes;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(t.n_tiles) * t.nts * 4 * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int nt = 0; nt < t.n_tiles; ++nt)
    for (int kc_i = 0; kc_i < t.k_chunks; ++kc_i)
      for (int sl = 0; sl < t.kc; ++sl)
        for (int ol = 0; ol < t.nts; ++ol) {
          const int s = kc_i * t.kc + sl, so = nt * t.nts + ol;
          uint16_t* core = wp + ((static_cast<size_t>(nt) * t.k_chunks + kc_i) * chunk_bytes +
                                 (static_cast<size_t>(sl) * t.nts + ol) * kCoreBytes) / 2;
          if (s >= t.s_in || so >= t.s_out) continue;
          for (int j = 0; j < 4; ++j) {
            const int co = so * 4 + j;
            if (co >= cout) continue;
            for (int c = 0; c < 4; ++c) {
              const int ci = s * 4 + c;
              if (ci >= cin) continue;
              const uint16_t h = f32_to_f16_rne(w[static_cast<size_t>(co) * cin + ci]);
              core[(0 * 4 + j) * 8 + 0 * 4 + c] = h;  // parity 0 block
              core[(1 * 4 + j) * 8 + 1 * 4 + c] = h;  // parity 1 block
            }
          }
        }
  for (int co = 0; co < cout; ++co) bp[co] = bias[co];
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = t.nts;
  r->tc_kc = t.kc;
  r->tc_stages = t.stages;
}

int launch_pointwise_tc(const LaunchRec& r, const Ptrs& p, void** state, int launch_index, void* stream) {
  const Tiling t = choose_tiling(r.C, r.Co);
  const unsigned m_total = static_cast<unsigned>(r.B) * static_cast<unsigned>(plane_pixels(r.H, r.W));
  DeviceInfo& di = device_info();
  if (di.sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || di.sms <= 0)
      return static_cast<int>(cudaErrorInvalidDevice);
  }
  if (!di.attr_set) {
    cudaError_t e = cudaSuccess;
    const int bytes = kSmemHeader + kSmemBudget;
#define GI_TC_ATTR(A, T) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(pointwise_tc_kernel<A, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)
    GI_TC_ATTR(GI_ACT_NONE, false);
    GI_TC_ATTR(GI_ACT_RELU, false);
    GI_TC_ATTR(GI_ACT_RELU6, false);
    GI_TC_ATTR(GI_ACT_NONE, true);
    GI_TC_ATTR(GI_ACT_RELU, true);
    GI_TC_ATTR(GI_ACT_RELU6, true);
#undef GI_TC_ATTR
    if (e != cudaSuccess) return static_cast<int>(e);
    di.attr_set = true;
  }
  // tensor map over the input: pixels (8-byte elements) x slices; cached per launch and input address
  CUtensorMap tmap;
  {
    const int err = map_cache_lookup(state, launch_index, p.in0, &tmap, [&](CUtensorMap* m) {
      return encode_plane_map(m, p.in0, m_total, t.s_in, kTilePx, t.kc);
    });
    if (err != 0) return err;
  }
  TcParams k;
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.bias = static_cast<const float*>(p.bias);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.m_total_px = m_total;
  k.s_out = t.s_out;
  k.nts = t.nts;
  k.n_tiles = t.n_tiles;
  k.kc = t.kc;
  k.k_chunks = t.k_chunks;
  k.stages = t.stages;
  k.m_tiles = static_cast<int>((m_total / 2 + kTileRows - 1) / kTileRows);
  // split the output tiles of one pixel tile over `groups` CTAs so that the busiest SM runs
  // as few tiles as possible; ties go to fewer groups (the input tile is then re-read less)
  const bool wide = t.nts > kMaxNts;
  const long long cta_slots = static_cast<long long>(di.sms) * (wide ? 1 : 2);
  int groups = 1;
  long long best_rounds = -1;
  for (int g = 1; g <= t.n_tiles; ++g) {
    const long long units_g = static_cast<long long>(k.m_tiles) * g;
    const long long rounds = ((units_g + cta_slots - 1) / cta_slots) * ((t.n_tiles + g - 1) / g);
    if (best_rounds < 0 || rounds < best_rounds) {
      best_rounds = rounds;
      groups = g;
    }
  }
  k.groups = groups;
  k.act_pre = r.ep.act_pre;
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  k.in_dead = r.in0_dead;
  // two buffers measured best on MobileNetV2 (four or eight were 4-8 % slower on the narrow layers)
  const unsigned n_acc = 2;
  k.n_acc = n_acc;
  unsigned cols = 32;
  while (cols < n_acc * static_cast<unsigned>(t.nts) * 8) cols <<= 1;
  k.tmem_cols = cols;
  k.timeout_ns = 1000000000u;
  // two slim CTAs per SM (each its own producer / MMA / epilogue pipeline) hide the latency chain
  // of short tiles better than one wide CTA: measured +20-50 % on the narrow layers
  const int n_chunks = t.nts / 2;
  k.epq = wide ? 4 : n_chunks >= 2 ? 2 : 1;
  int ctas_per_sm = wide ? 1 : 2;
  const size_t stage_bytes = static_cast<size_t>(t.kc) * (kSliceBytes + t.nts * kCoreBytes);
  const long long units = static_cast<long long>(k.m_tiles) * groups;
  // no more work units than SMs: a second CTA per SM would stay empty, so the one CTA keeps
  // all of shared memory for stages in flight
  if (units <= di.sms) ctas_per_sm = 1;
  if (ctas_per_sm == 2) {
    const int st2 = static_cast<int>((108 * 1024 - kSmemHeader) / stage_bytes);
    if (st2 < 2) ctas_per_sm = 1;
    else if (st2 < k.stages) k.stages = st2;
  }
  const long long slots = static_cast<long long>(di.sms) * ctas_per_sm;
  const unsigned grid = static_cast<unsigned>(units < slots ? units : slots);
  const size_t smem = kSmemHeader + static_cast<size_t>(k.stages) * stage_bytes;
  const unsigned threads = 64u + 128u * k.epq;
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
#define GI_TC_LAUNCH(A, T) launch_pdl(pointwise_tc_kernel<A, T>, grid, threads, smem, cu_stream, tmap, k)
  if (tail) {
    if (k.act_pre == GI_ACT_RELU6) GI_TC_LAUNCH(GI_ACT_RELU6, true);
    else if (k.act_pre == GI_ACT_RELU) GI_TC_LAUNCH(GI_ACT_RELU, true);
    else GI_TC_LAUNCH(GI_ACT_NONE, true);
  } else {
    if (k.act_pre == GI_ACT_RELU6) GI_TC_LAUNCH(GI_ACT_RELU6, false);
    else if (k.act_pre == GI_ACT_RELU) GI_TC_LAUNCH(GI_ACT_RELU, false);
    else GI_TC_LAUNCH(GI_ACT_NONE, false);
  }
#undef GI_TC_LAUNCH
  return static_cast<int>(cudaGetLastError());
}

void pointwise_tc_release(void* state) { map_cache_release(state); }

unsigned int pointwise_tc_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_tc_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
