// Pointwise (1x1) convolution, second tensor-core variant: the activation operand goes through
// registers into TENSOR MEMORY and the MMA reads it from there (tcgen05.mma with A in TMEM), the
// weights come from shared memory, filled by bulk TMA copies.
//
// Why a second variant: a pixel-slice is 4 fp16 = two 32-bit words, and a TMEM lane holds the K
// axis of an fp16 A operand two elements per 32-bit column - so "lane = pixel, columns 2s, 2s+1 =
// slice s" IS the operand layout.  A thread loads the 8 bytes of its pixel for a run of slices
// (coalesced: a warp reads 256 contiguous bytes per slice) and writes them to its lane with
// tcgen05.st.  Nothing is padded or duplicated, so the tensor pipe does exactly 2*M*N*K flops and
// the weight operand is the dense [Cout][Cin] matrix.  The pixel-pair variant (pointwise_tc.cu)
// keeps its place for small Cin, where its fully asynchronous TMA feed wins; this one takes the
// layers with many input channels, where the pair variant's 4x larger expanded weight tile made
// the shared-memory fill, not HBM, the bound.
//
// CTA = 10 warps: warp 0 streams weight chunks (TMA, mbarrier ring), warp 1 issues MMAs and owns
// tensor memory, warps 2-9 are the data warps: two per TMEM lane quarter, each loading half of a
// K chunk of the next tile and then draining half of the accumulator columns of the previous
// tile (bias, activation, residual, fp16 pack, 8-byte stores: 256 contiguous bytes per warp).
// Accumulators and A chunks are double-buffered in the 512 TMEM columns.  Waits are bounded.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "sm100_ptx.cuh"

namespace gi {
namespace {

using namespace ptx;

constexpr int kRows = 128;
constexpr int kDataWarps = 8;
constexpr int kThreads = 64 + 32 * kDataWarps;
constexpr int kMaxStages = 4;
constexpr int kSmemHeader = 1024;
constexpr int kSmemBudget = 200 * 1024;
constexpr int kMaxNt = 192;

__device__ unsigned int g_ts_error = 0;

struct TsParams {
  const __half* in;
  const __half* res;
  __half* out;
  const float* bias;
  const unsigned char* wts;
  unsigned int m_total_px;
  int s_in, s_out;
  int ks, n_chunks;      // input slices per K chunk (multiple of 4), chunks per tile
  int n_t, n_tiles;      // output channels per tile (multiple of 16), tiles along N
  int stages;
  int m_tiles;
  int has_res, act_post;
  unsigned int timeout_ns;
};

struct Header {
  unsigned long long b_full[kMaxStages];
  unsigned long long b_empty[kMaxStages];
  unsigned long long a_full[2];
  unsigned long long a_empty[2];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned tmem_addr;
  unsigned abort_flag;
};

__device__ __forceinline__ void tmem_st16(unsigned taddr, const unsigned* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
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

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

enum : unsigned { kErrProducer = 1u, kErrMma = 2u, kErrData = 4u, kErrDrain = 8u };

// ACT: activation right after the bias; TAIL: a residual add and / or a second activation follow
template <int ACT, bool TAIL>
__global__ void __launch_bounds__(kThreads, 1) pointwise_ts_kernel(const TsParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Header* hdr = reinterpret_cast<Header*>(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile unsigned* abort_flag = &hdr->abort_flag;
  const unsigned chunk_bytes = static_cast<unsigned>(p.ks) * p.n_t * 8u;  // ks/2 K units x n_t rows x 16 bytes
  const unsigned data0 = smem_u32(smem + kSmemHeader);
  const unsigned a_cols = static_cast<unsigned>(p.ks) * 2u;
  const unsigned acc_cols = static_cast<unsigned>(p.n_t);
  const int n_units = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&hdr->b_full[i]), 1);
      mbar_init(smem_u32(&hdr->b_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&hdr->a_full[i]), kDataWarps);
      mbar_init(smem_u32(&hdr->a_empty[i]), 1);
      mbar_init(smem_u32(&hdr->acc_full[i]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[i]), kDataWarps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&hdr->tmem_addr), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = hdr->tmem_addr;
  // TMEM columns: [0, 2*n_t) two accumulators, then two A chunk buffers of 2*ks columns
  const unsigned a_col0 = 2u * acc_cols;

  if (warp == 0) {
    // ------------------------------------------------------------ weight producer
    if (lane == 0) {
      unsigned it = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const int n_tile = u % p.n_tiles;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, phase = (it / p.stages) & 1u;
          if (!mbar_wait(smem_u32(&hdr->b_empty[stage]), phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrProducer)) {
            ok = false;
            break;
          }
          const unsigned full = smem_u32(&hdr->b_full[stage]);
          mbar_expect_tx(full, chunk_bytes);
          bulk_load(data0 + stage * chunk_bytes, p.wts + (static_cast<size_t>(n_tile) * p.n_chunks + c) * chunk_bytes, chunk_bytes,
                    full);
        }
      }
      if (!ok) {
        const unsigned first = it > static_cast<unsigned>(p.stages) ? it - p.stages : 0u;
        for (unsigned j = first; j < it; ++j) {
          unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&hdr->b_full[j % p.stages]), (j / p.stages) & 1u)) {
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
      // instruction descriptor: fp32 accumulator, fp16 A and B, B K-major, M = 128, N = n_t
      const unsigned idesc = (1u << 4) | ((acc_cols >> 3) << 17) | ((kRows >> 4) << 24);
      const unsigned b_lbo = acc_cols * 16u;  // distance between consecutive 8-element K units of the weight tile
      unsigned it = 0, tile = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x, ++tile) {
        const unsigned acc = tile & 1u, acc_phase = (tile >> 1) & 1u;
        if (!mbar_wait(smem_u32(&hdr->acc_empty[acc]), acc_phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrMma)) break;
        const unsigned d_tmem = tmem_base + acc * acc_cols;
        for (int c = 0; c < p.n_chunks; ++c, ++it) {
          const unsigned stage = it % p.stages, b_phase = (it / p.stages) & 1u;
          const unsigned abuf = it & 1u, a_phase = (it >> 1) & 1u;
          if (!mbar_wait(smem_u32(&hdr->a_full[abuf]), a_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrMma) ||
              !mbar_wait(smem_u32(&hdr->b_full[stage]), b_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrMma)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const unsigned a_tmem = tmem_base + a_col0 + abuf * a_cols;
          const unsigned b_base = data0 + stage * chunk_bytes;
          for (int ks = 0; ks < p.ks / 4; ++ks) {  // 16 channels = 4 slices = 8 TMEM columns = 2 K units per MMA
            const unsigned long long bd = smem_desc(b_base + ks * 2 * b_lbo, b_lbo, 128);
            umma_f16_ts(d_tmem, a_tmem + ks * 8, bd, idesc, (c > 0 || ks > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&hdr->a_empty[abuf]));
          umma_commit(smem_u32(&hdr->b_empty[stage]));
        }
        if (ok) umma_commit(smem_u32(&hdr->acc_full[acc]));
      }
    }
  } else {
    // ------------------------------------------------------------ data warps: load A, drain D
    const int quarter = warp & 3;          // TMEM lanes [32*quarter, +32)
    const int half_id = (warp - 2) >> 2;   // which half of the chunk's slices / of the accumulator columns
    const unsigned lane_bits = static_cast<unsigned>(quarter * 32) << 16;
    const int row_in_tile = quarter * 32 + lane;
    const int ks_half = p.ks >> 1;         // slices this warp loads per chunk (multiple of 8)
    unsigned it = 0;
    bool ok = true;

    auto load_unit = [&](int u) -> bool {
      const int m_tile = u / p.n_tiles;
      const unsigned pixel = static_cast<unsigned>(m_tile) * kRows + row_in_tile;
      const bool px_ok = pixel < p.m_total_px;
      for (int c = 0; c < p.n_chunks; ++c, ++it) {
        const unsigned abuf = it & 1u, a_phase = (it >> 1) & 1u;
        if (!mbar_wait(smem_u32(&hdr->a_empty[abuf]), a_phase ^ 1u, abort_flag, p.timeout_ns, &g_ts_error, kErrData)) return false;
        tc_fence_after();
        const int s0 = c * p.ks + half_id * ks_half;
        const unsigned t_addr = tmem_base + lane_bits + a_col0 + abuf * a_cols + static_cast<unsigned>(half_id * ks_half) * 2u;
        const __half* src = p.in + (static_cast<size_t>(s0) * p.m_total_px + pixel) * 4;
        const size_t slice_stride = static_cast<size_t>(p.m_total_px) * 4;
        for (int j = 0; j < ks_half; j += 8) {
          // up to 8 slices = 16 columns per store; all loads of a batch are issued before the store
          unsigned r[16];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            uint2 v = make_uint2(0u, 0u);
            if (px_ok && j + q < ks_half && s0 + j + q < p.s_in) v = __ldg(reinterpret_cast<const uint2*>(src + (j + q) * slice_stride));
            r[2 * q] = v.x;
            r[2 * q + 1] = v.y;
          }
          tmem_st16(t_addr + j * 2, r);  // ks_half is a multiple of 8: always whole 16-column stores
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->a_full[abuf]));
      }
      return true;
    };

    auto drain_unit = [&](int u, unsigned tile) -> bool {
      const int m_tile = u / p.n_tiles, n_tile = u - m_tile * p.n_tiles;
      const unsigned acc = tile & 1u, acc_phase = (tile >> 1) & 1u;
      if (!mbar_wait(smem_u32(&hdr->acc_full[acc]), acc_phase, abort_flag, p.timeout_ns, &g_ts_error, kErrData)) return false;
      tc_fence_after();
      const unsigned pixel = static_cast<unsigned>(m_tile) * kRows + row_in_tile;
      const bool px_ok = pixel < p.m_total_px;
      const int groups = p.n_t >> 4;                       // 16-column groups in the accumulator
      const int g0 = half_id == 0 ? 0 : (groups + 1) >> 1; // first half takes the extra group
      const int g1 = half_id == 0 ? (groups + 1) >> 1 : groups;
      const unsigned t_addr = tmem_base + lane_bits + acc * acc_cols;
      for (int g = g0; g < g1; ++g) {
        unsigned r[16];
        tmem_ld16(t_addr + g * 16, r);
        tmem_ld_wait16(r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int so = (n_tile * p.n_t) / 4 + g * 4 + j;
          if (so >= p.s_out || !px_ok) continue;
          const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias) + so);
          const size_t off = (static_cast<size_t>(so) * p.m_total_px + pixel) * 4;  // in halves
          float2 v0 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1])), make_float2(b.x, b.y));
          float2 v1 = __fadd2_rn(make_float2(__uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])), make_float2(b.z, b.w));
          __half2 h0, h1;
          if (!TAIL) {
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
            uint2 q = make_uint2(0u, 0u);
            if (p.has_res) q = __ldg(reinterpret_cast<const uint2*>(p.res + off));
            const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
            const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
            h0 = __floats2half2_rn(act1(act1(v0.x, ACT) + r0.x, p.act_post), act1(act1(v0.y, ACT) + r0.y, p.act_post));
            h1 = __floats2half2_rn(act1(act1(v1.x, ACT) + r1.x, p.act_post), act1(act1(v1.y, ACT) + r1.y, p.act_post));
          }
          uint2 o;
          o.x = *reinterpret_cast<const unsigned*>(&h0);
          o.y = *reinterpret_cast<const unsigned*>(&h1);
          *reinterpret_cast<uint2*>(p.out + off) = o;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[acc]));
      return true;
    };

    // software pipeline: the operand of unit i+1 is loaded before the accumulator of unit i is drained
    int prev = -1;
    unsigned tile = 0;
    for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
      ok = load_unit(u);
      if (ok && prev >= 0) {
        ok = drain_unit(prev, tile);
        ++tile;
      }
      prev = u;
    }
    if (ok && prev >= 0) drain_unit(prev, tile);
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
  int s_in, s_out, ks, n_chunks, n_t, n_tiles, stages;
};

Tiling choose_tiling(int cin, int cout) {
  Tiling t;
  t.s_in = slices(cin);
  t.s_out = slices(cout);
  const int n_pad = (cout + 15) / 16 * 16;
  t.n_tiles = (n_pad + kMaxNt - 1) / kMaxNt;
  t.n_t = ((n_pad + t.n_tiles - 1) / t.n_tiles + 15) / 16 * 16;
  // TMEM: 2 accumulators of n_t columns, 2 A buffers of 2*ks columns, 512 in all
  int ks_max = (512 - 2 * t.n_t) / 4;
  ks_max = ks_max / 16 * 16;  // whole 16-column stores for both halves of a chunk
  if (ks_max > 64) ks_max = 64;
  const int s_pad = (t.s_in + 15) / 16 * 16;
  t.n_chunks = (s_pad + ks_max - 1) / ks_max;
  t.ks = ((s_pad + t.n_chunks - 1) / t.n_chunks + 15) / 16 * 16;
  const int chunk_bytes = t.ks * t.n_t * 8;
  t.stages = kSmemBudget / chunk_bytes;
  if (t.stages > kMaxStages) t.stages = kMaxStages;
  if (t.stages < 2) t.stages = 2;
  return t;
}

}  // namespace

bool pointwise_ts_supported(int cin, int cout) { return cin > 0 && cout > 0; }

// Dense weights as the B operand, per (output tile, K chunk): [ks/2 K units][n_t rows][8 halves].
void pointwise_ts_pack(const float* w, const float* bias, int cin, int cout, std::vector<uint8_t>* blob, LaunchRec* r) {
  const Tiling t = choose_tiling(cin, cout);
  const size_t chunk_bytes = static_cast<size_t>(t.ks) * t.n_t * 8;
  const size_t wbytes = static_cast<size_t>(t.n_tiles) * t.n_chunks * chunk_bytes;
  const uint64_t woff = round_up_u64(blob->size(), 256);
  blob->resize(woff + wbytes, 0);
  const uint64_t boff = round_up_u64(blob->size(), 256);
  blob->resize(boff + static_cast<size_t>(t.n_tiles) * t.n_t * sizeof(float), 0);
  uint16_t* wp = reinterpret_cast<uint16_t*>(blob->data() + woff);
  float* bp = reinterpret_cast<float*>(blob->data() + boff);
  for (int co = 0; co < cout; ++co) {
    const int nt = co / t.n_t, row = co % t.n_t;
    bp[co] = bias[co];
    for (int ci = 0; ci < cin; ++ci) {
      const int chunk = ci / (t.ks * 4), k = ci % (t.ks * 4);
      uint16_t* base = wp + (static_cast<size_t>(nt) * t.n_chunks + chunk) * (chunk_bytes / 2);
      base[(static_cast<size_t>(k / 8) * t.n_t + row) * 8 + k % 8] = f32_to_f16_rne(w[static_cast<size_t>(co) * cin + ci]);
    }
  }
  r->wts = Loc{W_WEIGHTS, 0, woff};
  r->bias = Loc{W_WEIGHTS, 0, boff};
  r->wts_bytes = wbytes;
  r->tc_nt = t.n_t;
  r->tc_kc = t.ks;
  r->tc_stages = t.stages;
}

int launch_pointwise_ts(const LaunchRec& r, const Ptrs& p, void* stream) {
  const Tiling t = choose_tiling(r.C, r.Co);
  TsParams k;
  k.in = static_cast<const __half*>(p.in0);
  k.res = static_cast<const __half*>(p.res);
  k.out = static_cast<__half*>(p.out);
  k.bias = static_cast<const float*>(p.bias);
  k.wts = static_cast<const unsigned char*>(p.wts);
  k.m_total_px = static_cast<unsigned>(r.B) * static_cast<unsigned>(plane_pixels(r.H, r.W));
  k.s_in = t.s_in;
  k.s_out = t.s_out;
  k.ks = t.ks;
  k.n_chunks = t.n_chunks;
  k.n_t = t.n_t;
  k.n_tiles = t.n_tiles;
  k.stages = t.stages;
  k.m_tiles = static_cast<int>((k.m_total_px + kRows - 1) / kRows);
  k.has_res = r.ep.has_res;
  k.act_post = r.ep.act_post;
  k.timeout_ns = 1000000000u;
  static int sms = 0;
  static bool attr_set = false;
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const bool tail = k.has_res || k.act_post != GI_ACT_NONE;
  if (!attr_set) {
    cudaError_t e = cudaSuccess;
    const int bytes = kSmemHeader + kSmemBudget;
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
  const long long units = static_cast<long long>(k.m_tiles) * k.n_tiles;
  const unsigned grid = static_cast<unsigned>(units < sms ? units : sms);
  // the kernel reserves all of tensor memory, so exactly one CTA may live on an SM: ask for enough
  // shared memory that a second one cannot be co-resident
  size_t smem = kSmemHeader + static_cast<size_t>(t.stages) * t.ks * t.n_t * 8;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaStream_t cu_stream = static_cast<cudaStream_t>(stream);
  const int act = r.ep.act_pre;
#define GI_TS_LAUNCH(A, T) pointwise_ts_kernel<A, T><<<grid, kThreads, smem, cu_stream>>>(k)
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

unsigned int pointwise_ts_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_ts_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
