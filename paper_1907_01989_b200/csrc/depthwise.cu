// Depthwise 3x3 convolution for fp16 storage: a bandwidth-bound stencil.
//
// A work item is a band of output rows in a few planes (plane = one 4-channel slice of one
// image; the planes of one slice are adjacent in memory, so they share the slice's 36 weights).
// The input rows a band needs - its halo included - are one contiguous run per plane and are
// staged into shared memory by bulk asynchronous copies (16-byte aligned, one mbarrier per
// buffer).  CTAs are persistent over a contiguous range of items and stage into a ring of two to
// four buffers: the copies for the next one to three items are in flight while the current one is
// computed (bytes in flight are what hides the HBM latency).  Each thread walks
// down one output column; every input row it reads feeds three running accumulators (packed
// two-wide fp32 FMAs), so an input pixel-slice is read from HBM once and from shared memory
// three times; stores are 8 bytes per lane, contiguous across the warp.  Zero padding: zero rows
// staged above / below the band and a zero pixel that out-of-image columns point at (no tests in
// the loop); the packed small-plane mode tests row validity instead.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "pdl.cuh"

namespace gi {
namespace {

__device__ unsigned int g_dw_error = 0;  // sticky: set if the staging copy did not arrive in time

struct DwGeom {
  int B, H, W, Pin, Ho, Wo, Pout, S;
  int stride, dil, pt, pl;
  int nb;       // planes per work item
  int sub;      // sub-bands per band (thread groups walking different rows of one plane)
  int tr;       // output rows walked by one thread
  int bands;    // bands per plane
  int bchunks;  // ceil(B / nb)
  int head_px;  // zeroed pixels in front of each plane's staged rows (even, >= W + 2)
  int plane_stride_px;  // pixels reserved per plane in one staging buffer (even)
  int items;            // S * bchunks * bands
  int packed;           // 1: whole small planes, staged back to back by one copy per item
  int in_dead;          // 1: the input tensor is not read again after this kernel
  int nbuf;             // staging buffers per CTA (2..4): nbuf - 1 items are in flight ahead of the one computed
  unsigned timeout_ns;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ float act1(float v, int kind) {
  if (kind == GI_ACT_RELU) return fmaxf(v, 0.0f);
  if (kind == GI_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

// three taps of one input row, 4 channels each, as packed pairs for the two-wide fp32 FMA
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
// start of an accumulation: the bias is the addend of the first FMA
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
__device__ __forceinline__ Row widen(const uint2* u) {
  Row r;
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    r.lo[k] = __half22float2(*reinterpret_cast<const __half2*>(&u[k].x));
    r.hi[k] = __half22float2(*reinterpret_cast<const __half2*>(&u[k].y));
  }
  return r;
}

// Staging buffer of one plane: [head_px zeros][rows of the band, copied][W+1 zeros when the band
// touches the bottom edge].  Row -1 and row H therefore read as zeros with no test in the loop.
//
// MODE 0: stride 1, dilation 1, at most one padding row above and below - every input row feeds
//         three running accumulators
// MODE 1: stride 2, dilation 1, same padding limit - the last row of an output is the first row
//         of the next
// MODE 2: anything else - three rows fetched per output row, each tap tested
// MODE 3: stride 1, dilation d > 1, padding d on every side (the dilated blocks of a segmentation backbone), whole planes
//         staged by one copy: the rows of one residue class modulo d form an ordinary 3-row stencil among themselves
//         (output row y reads rows y - d, y, y + d), so a thread owns (plane, residue, column) and walks its class
//         with the three running accumulators of mode 0 - every staged pixel is fetched and widened three times, as in
//         mode 0, instead of nine times as in mode 2
// PACKED (modes 0/1, small planes): a work item is a run of whole planes, which are contiguous in
//         memory, so ONE bulk copy stages them back to back (many small copies are slow); the
//         rows above and below a plane are then its neighbours' rows, so row validity is tested
//         (one compare per row) instead of relying on zero rows.
// ACT: activation applied right after the bias (the common fused case); TAIL: a residual add
// and / or a second activation follow.
// PAIR (mode 0, even W): a thread owns TWO adjacent output columns.  The four input pixels a row of the pair
// needs are fetched with three loads and converted once (16 conversions for two outputs instead of 24), and
// the pair is stored with one 16-byte store: the kernel is bound by the FMA pipe (packed FMAs, the fp16 ->
// fp32 conversions and integer multiply-adds all issue there) as much as by HBM.
// PLANE (0 = none; mode 0: 14 / 7 whole packed planes, 28 in bands of 14 rows, 112 / 56 with PAIR in sub-bands of 14 rows; mode 1:
// 112 / 56 / 28 wide planes in bands of 8 / 7 / 7 output rows, 14 whole packed planes).  For the packed case: the planes are PLANE x PLANE with one padding row and
// column on every side, and a thread walks a whole column.  With the trip count and the row pitch known at compile
// time the walk is straight-line code: the three running accumulators rotate without register moves, every address is
// an immediate offset from one base and the tests for rows outside the plane disappear (measured in the kernel that
// runs a whole inverted-residual block: 36 % less time in the same stencil).
template <int MODE, int ACT, bool TAIL, bool PACKED, bool PAIR, int PLANE>
__global__ void __launch_bounds__(256, (PLANE > 0 && !PAIR) ? 3 : 2) depthwise_f16_kernel(const __half* __restrict__ in, const float* __restrict__ w,
                                                                const float* __restrict__ bias, const __half* __restrict__ res,
                                                                __half* __restrict__ out, const DwGeom g, const Epilogue ep) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[4];
  __shared__ unsigned timed_out;
  const unsigned buf_bytes = PACKED ? static_cast<unsigned>(g.Pin) * 8u * g.nb + 16u : static_cast<unsigned>(g.plane_stride_px) * 8u * g.nb;
  const int W = g.W, H = g.H, Wo = g.Wo, stride = g.stride, pt = g.pt;

  // contiguous, balanced range of work items for this CTA: items of one slice stay together
  const int per = g.items / gridDim.x, extra = g.items % gridDim.x;
  const int first = blockIdx.x * per + min(static_cast<int>(blockIdx.x), extra);
  const int count = per + (static_cast<int>(blockIdx.x) < extra ? 1 : 0);
  const int th = g.sub * g.tr;

  // work items are numbered band-fastest, then batch chunk, then slice; a CTA walks a contiguous
  // range, so the triple is decoded once and then advanced without divisions
  struct Item {
    int s, bc, band;
  };
  auto advance = [&](Item it) {
    if (++it.band == g.bands) {
      it.band = 0;
      if (++it.bc == g.bchunks) {
        it.bc = 0;
        ++it.s;
      }
    }
    return it;
  };
  auto item_rows = [&](const Item& it, int& s, int& b0, int& nbk, int& oy0, int& oy1, int& start_px, unsigned& bytes, bool& last_band) {
    const int band = it.band, bc = it.bc;
    s = it.s;
    b0 = bc * g.nb;
    nbk = min(g.nb, g.B - b0);
    oy0 = band * th;
    oy1 = min(g.Ho, oy0 + th);
    const int in_y0 = max(0, oy0 * stride - pt);
    const int in_y1 = min(H, (oy1 - 1) * stride - pt + 2 * g.dil + 1);
    start_px = in_y0 * W;
    start_px -= start_px & 1;  // copies start on a 16-byte boundary: at most one pixel early
    const int end_px = min((in_y1 * W + 1) & ~1, g.Pin);
    bytes = static_cast<unsigned>(end_px - start_px) * 8u;
    last_band = band == g.bands - 1;
  };
  auto issue = [&](const Item& item, int buf) {  // the 32 threads of warp 0: lane l copies planes l, l+32, ...
    int s, b0, nbk, oy0, oy1, start_px;
    unsigned bytes;
    bool lb;
    item_rows(item, s, b0, nbk, oy0, oy1, start_px, bytes, lb);
    const unsigned bar = smem_u32(&bars[buf]);
    // an input nobody reads again leaves L2 first, so that the output written here stays for the next kernel
    unsigned long long pol;
    if (g.in_dead) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    // earlier generic-proxy writes to this buffer (the zeroed bottom row) precede the async writes
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // the phase cannot complete before this arrival, whatever order the copies land in
    if (threadIdx.x == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes * nbk) : "memory");
    if (PACKED) {
      if (threadIdx.x == 0) {
        const __half* src = in + (static_cast<size_t>(s) * g.B + b0) * g.Pin * 4;
        const unsigned dst = smem_u32(smem_raw) + buf * buf_bytes + 16u;  // one zero pixel pair in front
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                     "l"(src), "r"(bytes * nbk), "r"(bar), "l"(pol)
                     : "memory");
      }
      return;
    }
    for (int pi = threadIdx.x; pi < nbk; pi += 32) {
      const __half* src = in + ((static_cast<size_t>(s) * g.B + b0 + pi) * g.Pin + start_px) * 4;
      const unsigned dst =
          smem_u32(smem_raw) + buf * buf_bytes + (static_cast<unsigned>(pi) * g.plane_stride_px + g.head_px) * 8u;
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst), "l"(src),
                   "r"(bytes), "r"(bar), "l"(pol)
                   : "memory");
    }
  };

  pdl_launch_dependents();
  // the zero heads are written once; copies never touch them
  if (PACKED) {
    if (static_cast<int>(threadIdx.x) < 2 * g.nbuf)
      *reinterpret_cast<uint2*>(smem_raw + (threadIdx.x >> 1) * buf_bytes + (threadIdx.x & 1) * 8) = make_uint2(0u, 0u);
  } else {
    for (int i = threadIdx.x; i < g.nbuf * g.nb * g.head_px; i += blockDim.x) {
      const int plane = i / g.head_px, px = i - plane * g.head_px;
      *reinterpret_cast<uint2*>(smem_raw + (static_cast<size_t>(plane) * g.plane_stride_px + px) * 8) = make_uint2(0u, 0u);
    }
  }
  pdl_wait();  // the first staging copy below reads the previous kernel's output
  if (threadIdx.x == 0) {
    for (int b = 0; b < g.nbuf; ++b) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[b])) : "memory");
    timed_out = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // column (pair of columns) owned by this thread in the first pass over an item's columns: (plane, sub-band, x)
  const int wcols = PAIR ? Wo >> 1 : Wo;
  const int vp_first = static_cast<int>(threadIdx.x) / wcols;
  const int x_first = static_cast<int>(threadIdx.x) - vp_first * wcols;
  const int pi_first = vp_first / g.sub, sb_first = vp_first - pi_first * g.sub;
  Item cur = {first / (g.bands * g.bchunks), (first / g.bands) % g.bchunks, first % g.bands};
  // the first nbuf - 1 items are requested up front; `ahead` is the next item to request
  Item ahead = cur;
  for (int j = 0; j < g.nbuf - 1 && j < count; ++j) {
    if (threadIdx.x < 32) issue(ahead, j);
    ahead = advance(ahead);
  }

  float2 wlo[9], whi[9];  // 9 taps x (channels 0-1, channels 2-3) of the current slice
  float2 blo = make_float2(0.f, 0.f), bhi = blo;
  int cur_s = -1;
  const int C4 = g.S * 4;

  int buf = 0, ahead_buf = g.nbuf - 1;
  unsigned round = 0;  // how often the ring of buffers has wrapped: the parity of the wait
  for (int i = 0; i < count; ++i) {
    int s, b0, nbk, oy0, oy1, start_px;
    unsigned bytes;
    bool last_band;
    item_rows(cur, s, b0, nbk, oy0, oy1, start_px, bytes, last_band);
    cur = advance(cur);
    // the buffer nbuf - 1 ahead was last read in iteration i-1, which ended with a barrier: refill it now
    if (i + g.nbuf - 1 < count) {
      if (threadIdx.x < 32) issue(ahead, ahead_buf);
      ahead = advance(ahead);
    }
    if (s != cur_s) {
      cur_s = s;
#pragma unroll
      for (int t = 0; t < 9; ++t) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(w + t * C4 + s * 4));
        wlo[t] = make_float2(v.x, v.y);
        whi[t] = make_float2(v.z, v.w);
      }
      const float4 v = __ldg(reinterpret_cast<const float4*>(bias + s * 4));
      blo = make_float2(v.x, v.y);
      bhi = make_float2(v.z, v.w);
    }
    {  // bounded wait for this item's rows
      const unsigned bar = smem_u32(&bars[buf]), parity = round & 1u;
      unsigned ok = 0;
      unsigned long long t0 = 0;
      for (unsigned spin = 0; !ok; ++spin) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (!ok && (spin & 255u) == 255u) {
          unsigned long long now;
          asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
          if (t0 == 0) {
            t0 = now;
          } else if (now - t0 > g.timeout_ns || *reinterpret_cast<volatile unsigned*>(&timed_out)) {
            timed_out = 1;
            atomicOr(&g_dw_error, 1u);
            break;
          }
        }
      }
    }
    if (*reinterpret_cast<volatile unsigned*>(&timed_out)) break;  // give up; results of this launch are invalid

    unsigned char* buf_base = smem_raw + buf * buf_bytes;
    if (MODE != 2 && !PACKED && (oy1 - 1) * stride - pt + 2 >= H) {
      // this band reads row H: W+1 zero pixels right after the last image row (they replace the
      // plane's own padding pixel and whatever an earlier item left there)
      const int z0 = H * W - start_px;
      for (int j = threadIdx.x; j < nbk * (W + 1); j += blockDim.x) {
        const int pi = j / (W + 1), px = j - pi * (W + 1);
        *reinterpret_cast<uint2*>(buf_base + (static_cast<size_t>(pi) * g.plane_stride_px + g.head_px + z0 + px) * 8) =
            make_uint2(0u, 0u);
      }
      __syncthreads();
    }

    const unsigned buf_addr = smem_u32(buf_base);
    const int cols = nbk * g.sub * wcols;
    for (int c = threadIdx.x; c < cols; c += blockDim.x) {
      int x = x_first, sb = sb_first, pi = pi_first;  // the first pass uses the decomposition made once per CTA
      if (c != static_cast<int>(threadIdx.x)) {
        const int vp = c / wcols;
        x = c - vp * wcols;
        pi = vp / g.sub;
        sb = vp - pi * g.sub;
      }
      if (PAIR) x *= 2;
      // (mode 3: `sb` is the residue class, whose first row is row sb)
      const int ya = MODE == 3 ? sb : oy0 + sb * g.tr, yb = MODE == 3 ? H : min(oy1, ya + g.tr);
      if (ya >= yb) continue;
      // plane_zero: a pixel of the zero head; data: where pixel (0,0) of the plane would be staged
      const unsigned plane_zero = PACKED ? buf_addr : buf_addr + static_cast<unsigned>(pi) * g.plane_stride_px * 8u;
      const unsigned data = PACKED ? buf_addr + 16u + static_cast<unsigned>(pi) * g.Pin * 8u
                                   : plane_zero + static_cast<unsigned>(g.head_px - start_px) * 8u;
      const size_t out_off = ((static_cast<size_t>(s) * g.B + b0 + pi) * g.Pout + static_cast<size_t>(ya) * Wo + x) * 4;
      __half* op = out + out_off;
      const ptrdiff_t res_minus_out = res - out;  // only used when TAIL
      const int out_stride = MODE == 3 ? g.dil * Wo * 4 : Wo * 4;  // halves from one output row of this thread to its next
      auto emit = [&](const Acc& a) {
        uint2 u;
        if (!TAIL) {
          // clamping after the rounding equals rounding after the clamp: 0 and 6 are fp16 values
          const __half2 lo = __floats2half2_rn(a.lo.x, a.lo.y), hi = __floats2half2_rn(a.hi.x, a.hi.y);
          u.x = *reinterpret_cast<const unsigned*>(&lo);
          u.y = *reinterpret_cast<const unsigned*>(&hi);
          // the clamps as signed 16-bit integer min / max on the fp16 bit patterns (negative
          // values have the sign bit set, non-negative ones order like integers): these run on
          // the integer pipe, which this kernel leaves idle, instead of the busy fp16 / FMA pipe
          if (ACT != GI_ACT_NONE) {
            u.x = __vmaxs2(u.x, 0u);
            u.y = __vmaxs2(u.y, 0u);
          }
          if (ACT == GI_ACT_RELU6) {
            u.x = __vmins2(u.x, 0x46004600u);
            u.y = __vmins2(u.y, 0x46004600u);
          }
        } else {
          float v[4] = {a.lo.x, a.lo.y, a.hi.x, a.hi.y};
#pragma unroll
          for (int e = 0; e < 4; ++e) v[e] = act1(v[e], ACT);
          if (ep.has_res) {
            const uint2 q = *reinterpret_cast<const uint2*>(op + res_minus_out);
            const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
            const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
            v[0] += r0.x;
            v[1] += r0.y;
            v[2] += r1.x;
            v[3] += r1.y;
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) v[e] = act1(v[e], ep.act_post);
          const __half2 lo = __floats2half2_rn(v[0], v[1]), hi = __floats2half2_rn(v[2], v[3]);
          u.x = *reinterpret_cast<const unsigned*>(&lo);
          u.y = *reinterpret_cast<const unsigned*>(&hi);
        }
        *reinterpret_cast<uint2*>(op) = u;
        op += out_stride;
      };
      const Acc bias_acc = {blo, bhi};

      if (MODE == 0 && PAIR) {
        // pixels x-1 | x, x+1 | x+2 of every input row: the outer two may lie outside the image (zero pixel)
        const int iy_first = ya - pt;
        const bool vl = x - g.pl >= 0, vr = x - g.pl + 3 < W;
        const unsigned mid0 = data + static_cast<unsigned>((iy_first * W + x - g.pl + 1) * 8);
        unsigned pm = mid0, pl_ = vl ? mid0 - 8u : plane_zero, pr_ = vr ? mid0 + 16u : plane_zero;
        const unsigned row_step = static_cast<unsigned>(W) * 8u, sl = vl ? row_step : 0u, sr = vr ? row_step : 0u;
        float2 plo[4], phi[4];  // the row's four pixels, widened
        auto next4 = [&]() {
          // (never with PACKED staging: the rows above and below the image are staged zeros)
          uint4 m;
          const uint2 a = lds64(pl_);
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w) : "r"(pm));
          const uint2 d = lds64(pr_);
          pl_ += sl;
          pm += row_step;
          pr_ += sr;
          plo[0] = __half22float2(*reinterpret_cast<const __half2*>(&a.x));
          phi[0] = __half22float2(*reinterpret_cast<const __half2*>(&a.y));
          plo[1] = __half22float2(*reinterpret_cast<const __half2*>(&m.x));
          phi[1] = __half22float2(*reinterpret_cast<const __half2*>(&m.y));
          plo[2] = __half22float2(*reinterpret_cast<const __half2*>(&m.z));
          phi[2] = __half22float2(*reinterpret_cast<const __half2*>(&m.w));
          plo[3] = __half22float2(*reinterpret_cast<const __half2*>(&d.x));
          phi[3] = __half22float2(*reinterpret_cast<const __half2*>(&d.y));
        };
        // kernel row `kr` of the current input row into the accumulators of both columns
        auto fma2 = [&](Acc* a, int kr) {
#pragma unroll
          for (int k = 0; k < 3; ++k) {
            a[0].lo = __ffma2_rn(plo[k], wlo[kr * 3 + k], a[0].lo);
            a[0].hi = __ffma2_rn(phi[k], whi[kr * 3 + k], a[0].hi);
            a[1].lo = __ffma2_rn(plo[k + 1], wlo[kr * 3 + k], a[1].lo);
            a[1].hi = __ffma2_rn(phi[k + 1], whi[kr * 3 + k], a[1].hi);
          }
        };
        auto start2 = [&](Acc* a) {  // a new output row: bias, then kernel row 0
          a[0] = bias_acc;
          a[1] = bias_acc;
          fma2(a, 0);
        };
        auto finish1 = [&](const Acc& a, const __half* rp) {
          uint2 u;
          if (!TAIL) {
            const __half2 lo = __floats2half2_rn(a.lo.x, a.lo.y), hi = __floats2half2_rn(a.hi.x, a.hi.y);
            u.x = *reinterpret_cast<const unsigned*>(&lo);
            u.y = *reinterpret_cast<const unsigned*>(&hi);
            if (ACT != GI_ACT_NONE) {
              u.x = __vmaxs2(u.x, 0u);
              u.y = __vmaxs2(u.y, 0u);
            }
            if (ACT == GI_ACT_RELU6) {
              u.x = __vmins2(u.x, 0x46004600u);
              u.y = __vmins2(u.y, 0x46004600u);
            }
          } else {
            float v[4] = {a.lo.x, a.lo.y, a.hi.x, a.hi.y};
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = act1(v[e], ACT);
            if (ep.has_res) {
              const uint2 q = *reinterpret_cast<const uint2*>(rp);
              const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
              const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
              v[0] += r0.x;
              v[1] += r0.y;
              v[2] += r1.x;
              v[3] += r1.y;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = act1(v[e], ep.act_post);
            const __half2 lo = __floats2half2_rn(v[0], v[1]), hi = __floats2half2_rn(v[2], v[3]);
            u.x = *reinterpret_cast<const unsigned*>(&lo);
            u.y = *reinterpret_cast<const unsigned*>(&hi);
          }
          return u;
        };
        auto emit2 = [&](const Acc* a) {  // two adjacent pixels: one 16-byte store (x even, rows of even length)
          const uint2 u0 = finish1(a[0], op + res_minus_out), u1 = finish1(a[1], op + res_minus_out + 4);
          *reinterpret_cast<uint4*>(op) = make_uint4(u0.x, u0.y, u1.x, u1.y);
          op += out_stride;
        };
        if (PLANE == 112 || PLANE == 56) {
          // sub-bands of exactly 14 output rows of a PLANE-wide image: the 16 staged rows as straight-line code (the
          // accumulators rotate at compile time, the row offsets are immediates, columns outside the image are predicated)
          constexpr int kRowsOut = 14;
          Acc acc[3][2];
#pragma unroll
          for (int j = 0; j < kRowsOut + 2; ++j) {
            uint4 m;
            uint2 a = make_uint2(0u, 0u), d = make_uint2(0u, 0u);
            if (vl) a = lds64(mid0 + static_cast<unsigned>(j * PLANE * 8 - 8));
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w) : "r"(mid0 + static_cast<unsigned>(j * PLANE * 8)));
            if (vr) d = lds64(mid0 + static_cast<unsigned>(j * PLANE * 8 + 16));
            plo[0] = __half22float2(*reinterpret_cast<const __half2*>(&a.x));
            phi[0] = __half22float2(*reinterpret_cast<const __half2*>(&a.y));
            plo[1] = __half22float2(*reinterpret_cast<const __half2*>(&m.x));
            phi[1] = __half22float2(*reinterpret_cast<const __half2*>(&m.y));
            plo[2] = __half22float2(*reinterpret_cast<const __half2*>(&m.z));
            phi[2] = __half22float2(*reinterpret_cast<const __half2*>(&m.w));
            plo[3] = __half22float2(*reinterpret_cast<const __half2*>(&d.x));
            phi[3] = __half22float2(*reinterpret_cast<const __half2*>(&d.y));
            if (j >= 2) {
              fma2(acc[(j + 1) % 3], 2);
              emit2(acc[(j + 1) % 3]);
            }
            if (j >= 1 && j <= kRowsOut) fma2(acc[(j + 2) % 3], 1);
            if (j < kRowsOut) start2(acc[j % 3]);
          }
          continue;
        }
        Acc a0[2], a1[2], a2[2];
        next4();
        start2(a0);
        next4();
        fma2(a0, 1);
        start2(a1);
        for (int oy = ya; oy < yb; oy += 3) {
          next4();
          fma2(a0, 2);
          emit2(a0);
          fma2(a1, 1);
          start2(a2);
          if (oy + 1 >= yb) break;
          next4();
          fma2(a1, 2);
          emit2(a1);
          fma2(a2, 1);
          start2(a0);
          if (oy + 2 >= yb) break;
          next4();
          fma2(a2, 2);
          emit2(a2);
          fma2(a0, 1);
          start2(a1);
        }
      } else if (MODE == 0 && PACKED && PLANE > 0) {
        const unsigned col = data + static_cast<unsigned>(x) * 8u;
        const bool vl = x >= 1, vr = x + 1 < PLANE;
        Acc acc[3];
        acc[0] = bias_acc;
#pragma unroll
        for (int iy = 0; iy < PLANE; ++iy) {
          // input row iy is kernel row 2 of output row iy - 1 (now complete), row 1 of output row iy, row 0 of iy + 1
          uint2 u[3];
          u[0] = make_uint2(0u, 0u);
          u[2] = make_uint2(0u, 0u);
          if (vl) u[0] = lds64(col + static_cast<unsigned>((iy * PLANE - 1) * 8));
          u[1] = lds64(col + static_cast<unsigned>(iy * PLANE * 8));
          if (vr) u[2] = lds64(col + static_cast<unsigned>((iy * PLANE + 1) * 8));
          const Row r = widen(u);
          if (iy >= 1) {
            fma_row(acc[(iy + 2) % 3], r, wlo + 6, whi + 6);
            emit(acc[(iy + 2) % 3]);
          }
          fma_row(acc[iy % 3], r, wlo + 3, whi + 3);
          if (iy + 1 < PLANE) acc[(iy + 1) % 3] = fma_row_from(bias_acc, r, wlo, whi);
        }
        emit(acc[(PLANE - 1) % 3]);
      } else if (MODE == 0 && !PACKED && PLANE == 28) {
        // the same straight-line walk for 28-wide planes cut into bands of 14 output rows: the band's 16 input rows are
        // staged with zero rows above the first and below the last row of the image, so every row is simply read
        constexpr int kRowsOut = 14, kW = 28;
        const unsigned col = data + static_cast<unsigned>(((ya - 1) * kW + x) * 8);
        const bool vl = x >= 1, vr = x + 1 < kW;
        Acc acc[3];
#pragma unroll
        for (int j = 0; j < kRowsOut + 2; ++j) {
          // staged row j of the band is kernel row 2 of output row j - 2 (now complete), row 1 of j - 1, row 0 of j
          uint2 u[3];
          u[0] = make_uint2(0u, 0u);
          u[2] = make_uint2(0u, 0u);
          if (vl) u[0] = lds64(col + static_cast<unsigned>((j * kW - 1) * 8));
          u[1] = lds64(col + static_cast<unsigned>(j * kW * 8));
          if (vr) u[2] = lds64(col + static_cast<unsigned>((j * kW + 1) * 8));
          const Row r = widen(u);
          if (j >= 2) {
            fma_row(acc[(j + 1) % 3], r, wlo + 6, whi + 6);
            emit(acc[(j + 1) % 3]);
          }
          if (j >= 1 && j <= kRowsOut) fma_row(acc[(j + 2) % 3], r, wlo + 3, whi + 3);
          if (j < kRowsOut) acc[j % 3] = fma_row_from(bias_acc, r, wlo, whi);
        }
      } else if (MODE == 3) {
        const int d = g.dil;
        const bool vl = x - d >= 0, vr = x + d < W;
        unsigned at = data + static_cast<unsigned>((ya * W + x) * 8);
        const unsigned row_step = static_cast<unsigned>(d * W) * 8u, dx = static_cast<unsigned>(d) * 8u;
        auto next_row = [&]() {
          uint2 u[3];
          u[0] = make_uint2(0u, 0u);
          u[2] = make_uint2(0u, 0u);
          if (vl) u[0] = lds64(at - dx);
          u[1] = lds64(at);
          if (vr) u[2] = lds64(at + dx);
          at += row_step;
          return widen(u);
        };
        const int n = (H - ya + d - 1) / d;  // rows of this residue class
        // class row k is kernel row 2 of the class's output row k - 1, row 1 of output row k, row 0 of output row k + 1
        Acc a0 = bias_acc, a1, a2;
        Row r = next_row();
        fma_row(a0, r, wlo + 3, whi + 3);
        a1 = fma_row_from(bias_acc, r, wlo, whi);
        for (int k = 1;; k += 3) {
          if (k >= n) {
            emit(a0);
            break;
          }
          r = next_row();
          fma_row(a0, r, wlo + 6, whi + 6);
          emit(a0);
          fma_row(a1, r, wlo + 3, whi + 3);
          a2 = fma_row_from(bias_acc, r, wlo, whi);
          if (k + 1 >= n) {
            emit(a1);
            break;
          }
          r = next_row();
          fma_row(a1, r, wlo + 6, whi + 6);
          emit(a1);
          fma_row(a2, r, wlo + 3, whi + 3);
          a0 = fma_row_from(bias_acc, r, wlo, whi);
          if (k + 2 >= n) {
            emit(a2);
            break;
          }
          r = next_row();
          fma_row(a2, r, wlo + 6, whi + 6);
          emit(a2);
          fma_row(a0, r, wlo + 3, whi + 3);
          a1 = fma_row_from(bias_acc, r, wlo, whi);
        }
      } else if (MODE == 1 && !PACKED && PLANE > 0) {
        // stride 2 without padding above / left on PLANE-wide planes, bands of exactly kRowsOut output rows: the band's
        // 2 * kRowsOut + 1 staged rows as straight-line code.  Window columns 2x and 2x + 1 are one aligned 16-byte
        // load; column 2x + 2 lies outside the image only for the last output column.  An even staged row is kernel
        // row 2 of the output row above it and row 0 of the one below; an odd one is kernel row 1.
        constexpr int kRowsOut = PLANE == 112 ? 8 : 7, kW = PLANE;
        const unsigned col = data + static_cast<unsigned>((2 * ya * kW + 2 * x) * 8);
        const bool vr = 2 * x + 2 < kW;
        Acc cur = bias_acc;
#pragma unroll
        for (int j = 0; j <= 2 * kRowsOut; ++j) {
          uint4 m;
          uint2 u[3];
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w) : "r"(col + static_cast<unsigned>(j * kW * 8)));
          u[0] = make_uint2(m.x, m.y);
          u[1] = make_uint2(m.z, m.w);
          u[2] = make_uint2(0u, 0u);
          if (vr) u[2] = lds64(col + static_cast<unsigned>((j * kW + 2) * 8));
          const Row r = widen(u);
          if (j & 1) {
            fma_row(cur, r, wlo + 3, whi + 3);
          } else {
            if (j > 0) {
              fma_row(cur, r, wlo + 6, whi + 6);
              emit(cur);
            }
            if (j < 2 * kRowsOut) cur = fma_row_from(bias_acc, r, wlo, whi);
          }
        }
      } else if (MODE == 1 && PACKED && PLANE == 14) {
        // the same for whole 14 x 14 planes staged back to back (7 output rows): row 14 lies outside the plane and
        // contributes nothing, so the last output row is complete after row 13
        constexpr int kW = 14;
        const unsigned col = data + static_cast<unsigned>(2 * x * 8);
        const bool vr = 2 * x + 2 < kW;
        Acc cur = bias_acc;
#pragma unroll
        for (int j = 0; j < kW; ++j) {
          uint4 m;
          uint2 u[3];
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w) : "r"(col + static_cast<unsigned>(j * kW * 8)));
          u[0] = make_uint2(m.x, m.y);
          u[1] = make_uint2(m.z, m.w);
          u[2] = make_uint2(0u, 0u);
          if (vr) u[2] = lds64(col + static_cast<unsigned>((j * kW + 2) * 8));
          const Row r = widen(u);
          if (j & 1) {
            fma_row(cur, r, wlo + 3, whi + 3);
            if (j == kW - 1) emit(cur);
          } else {
            if (j > 0) {
              fma_row(cur, r, wlo + 6, whi + 6);
              emit(cur);
            }
            cur = fma_row_from(bias_acc, r, wlo, whi);
          }
        }
      } else if (MODE != 2) {
        // one pointer per tap column, walking down the staged rows; a column outside the image
        // stays on a zero pixel
        unsigned tp[3], step[3];
        const int iy_first = ya * stride - pt;
        int iy_cur = iy_first;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          const int ix = x * stride - g.pl + k;
          const bool v = ix >= 0 && ix < W;
          tp[k] = v ? data + static_cast<unsigned>((iy_first * W + ix) * 8) : plane_zero;
          step[k] = v ? static_cast<unsigned>(W) * 8u : 0u;
        }
        auto next_row = [&]() {
          uint2 u[3];
          if (PACKED) {
            const bool vy = iy_cur >= 0 && iy_cur < H;  // outside the plane lie the neighbours' rows, not zeros
            ++iy_cur;
#pragma unroll
            for (int k = 0; k < 3; ++k) {
              u[k] = make_uint2(0u, 0u);
              if (vy) u[k] = lds64(tp[k]);
              tp[k] += step[k];
            }
          } else {
#pragma unroll
            for (int k = 0; k < 3; ++k) {
              u[k] = lds64(tp[k]);
              tp[k] += step[k];
            }
          }
          return widen(u);
        };
        if (MODE == 0) {
          Acc a0, a1, a2;
          Row r = next_row();
          a0 = fma_row_from(bias_acc, r, wlo, whi);  // output ya, kernel row 0
          r = next_row();
          fma_row(a0, r, wlo + 3, whi + 3);          // output ya, kernel row 1
          a1 = fma_row_from(bias_acc, r, wlo, whi);  // output ya+1, kernel row 0
          for (int oy = ya; oy < yb; oy += 3) {
            r = next_row();
            fma_row(a0, r, wlo + 6, whi + 6);
            emit(a0);
            fma_row(a1, r, wlo + 3, whi + 3);
            a2 = fma_row_from(bias_acc, r, wlo, whi);
            if (oy + 1 >= yb) break;
            r = next_row();
            fma_row(a1, r, wlo + 6, whi + 6);
            emit(a1);
            fma_row(a2, r, wlo + 3, whi + 3);
            a0 = fma_row_from(bias_acc, r, wlo, whi);
            if (oy + 2 >= yb) break;
            r = next_row();
            fma_row(a2, r, wlo + 6, whi + 6);
            emit(a2);
            fma_row(a0, r, wlo + 3, whi + 3);
            a1 = fma_row_from(bias_acc, r, wlo, whi);
          }
        } else {
          Acc carry = fma_row_from(bias_acc, next_row(), wlo, whi);
          for (int oy = ya; oy < yb; ++oy) {
            fma_row(carry, next_row(), wlo + 3, whi + 3);
            const Row r2 = next_row();
            fma_row(carry, r2, wlo + 6, whi + 6);
            emit(carry);
            carry = fma_row_from(bias_acc, r2, wlo, whi);
          }
        }
      } else {
        int ix[3];
        bool vx[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          ix[k] = x * stride - g.pl + k * g.dil;
          vx[k] = ix[k] >= 0 && ix[k] < W;
        }
        auto fetch = [&](int iy) {
          uint2 u[3];
          const bool vy = iy >= 0 && iy < H;
#pragma unroll
          for (int k = 0; k < 3; ++k)
            u[k] = (vy && vx[k]) ? lds64(data + static_cast<unsigned>((iy * W + ix[k]) * 8)) : make_uint2(0u, 0u);
          return widen(u);
        };
        for (int oy = ya; oy < yb; ++oy) {
          const int iy = oy * stride - pt;
          Acc a = bias_acc;
          fma_row(a, fetch(iy), wlo, whi);
          fma_row(a, fetch(iy + g.dil), wlo + 3, whi + 3);
          fma_row(a, fetch(iy + 2 * g.dil), wlo + 6, whi + 6);
          emit(a);
        }
      }
    }
    // an odd plane carries one extra pixel: keep it zero
    if (last_band && g.Pout > g.Ho * Wo && static_cast<int>(threadIdx.x) < nbk) {
      const size_t off = ((static_cast<size_t>(s) * g.B + b0 + threadIdx.x) * g.Pout + g.Ho * Wo) * 4;
      *reinterpret_cast<uint2*>(out + off) = make_uint2(0u, 0u);
    }
    __syncthreads();  // everyone is done with this buffer before it is refilled
    if (++buf == g.nbuf) {
      buf = 0;
      ++round;
    }
    if (++ahead_buf == g.nbuf) ahead_buf = 0;
  }
  if (*reinterpret_cast<volatile unsigned*>(&timed_out) && threadIdx.x == 0) {
    // copies already issued may still land: give them the same bounded grace before leaving
    unsigned long long t0, now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    do {
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
    } while (now - t0 < g.timeout_ns);
  }
}

constexpr int kMaxSmem = 200 * 1024;    // all staging buffers of one CTA
constexpr int kSmemPerCta = 110 * 1024; // target: two CTAs per SM
constexpr int kSmemPerSm = 226 * 1024;

}  // namespace

// `dry_run`: stop after the geometry has been derived and checked, before anything that touches the device
static int depthwise_f16_impl(const LaunchRec& r, const Ptrs& p, void* stream, bool dry_run) {
  DwGeom g;
  g.B = r.B;
  g.H = r.H;
  g.W = r.W;
  g.Pin = plane_pixels(r.H, r.W);
  g.Ho = r.Ho;
  g.Wo = r.Wo;
  g.Pout = plane_pixels(r.Ho, r.Wo);
  g.S = slices(r.C);
  g.stride = r.sh;
  g.dil = r.dh;
  g.pt = r.pt;
  g.pl = r.pl;
  g.timeout_ns = 1000000000u;
  g.in_dead = r.in0_dead;
  g.head_px = (g.W + 3) & ~1;
  // two output columns per thread: stride 1, one padding column, rows of even length (16-byte aligned pixel
  // pairs), planes at least 56 wide.  Measured at batch 256 against one column per thread: 112x112x32
  // 0.1055 -> 0.0901 ms, 112x112x96 (batch 128) 0.1393 -> 0.1290 ms, 56x56x144 0.1208 -> 0.1024 ms; 28x28 and
  // smaller planes are 2-12 % slower that way and keep one column per thread.
  const bool pair = g.stride == 1 && g.dil == 1 && g.pl == 1 && g.pt <= 1 && g.W % 2 == 0 && g.Wo == g.W && g.W >= 56;
  const int wcols = pair ? g.Wo / 2 : g.Wo;
  // thread groups: as many "virtual planes" (plane x sub-band) as fit in ~256 threads
  int vp = 256 / wcols;
  if (vp < 1) vp = 1;
  g.nb = vp < g.B ? vp : g.B;
  g.sub = vp / g.nb;
  if (g.sub < 1) g.sub = 1;
  // rows walked by a thread: 16 (stride 1) or 8; pairs: 14, which divides the usual plane heights - bands of
  // equal height measured better than taller ones with a short last band (16 rows: 10-20 % slower on 112 / 56)
  // planes of up to about 33 x 33 pixels are walked whole as well (28 or 33 rows per thread): whole planes are contiguous,
  // so one copy stages an item instead of one per plane, and no halo row is read twice (28 x 28, batch 256, 192 channels:
  // 0.0430 -> 0.0389 ms)
  // - where that still leaves at least one work item per SM (at batch 1 the bands are the parallelism)
  const int whole_nb = g.nb < 1 ? 1 : g.nb;
  const bool whole = g.H > 16 && g.H * g.W <= 1100 && static_cast<long long>(g.S) * ((g.B + whole_nb - 1) / whole_nb) >= 148;
  const int tr_target = g.stride == 1 ? (pair ? 14 : (whole ? g.H : 16)) : 8;
  int total_sub = (g.Ho + tr_target - 1) / tr_target;
  if (pair) {
    // up to four sub-bands of one plane (they share halo rows), two passes of the threads per item; the
    // staging budget below then decides how many planes go with them (56 rows of 112: one; of 56: two)
    g.sub = total_sub < 4 ? total_sub : 4;
    const int planes = 512 / (wcols * g.sub);
    g.nb = planes < 1 ? 1 : planes < g.B ? planes : g.B;
  }
  if (total_sub < g.sub) g.sub = total_sub;
  g.tr = (g.Ho + total_sub - 1) / total_sub;
  g.bands = (total_sub + g.sub - 1) / g.sub;
  auto smem_for = [&](const DwGeom& q) {
    const int th = q.sub * q.tr;
    const int rows_in = (th - 1) * q.stride + 2 * q.dil + 1;
    int px = (rows_in < q.H ? rows_in : q.H) * q.W + 2;  // + alignment pixel in front, rounding pixel behind
    if (px > q.Pin) px = q.Pin;
    return q.head_px + ((px + 1) & ~1) + ((q.W + 3) & ~1);  // zero head, staged rows, zero row behind
  };
  g.plane_stride_px = smem_for(g);
  // per staging buffer: two buffers per CTA, two or three CTAs per SM - unless the measured table says otherwise
  const long long budget = (r.dw_buf_kb > 0 ? r.dw_buf_kb : 64) * 1024LL;
  while (static_cast<long long>(g.plane_stride_px) * 8 * g.nb > budget && (g.nb > 1 || g.sub > 1 || g.tr > 1)) {
    if (g.nb > 1) {
      g.nb = (g.nb + 1) / 2;
    } else if (g.sub > 1) {
      g.sub = (g.sub + 1) / 2;
    } else {
      g.tr = (g.tr + 1) / 2;
    }
    total_sub = (g.Ho + g.tr - 1) / g.tr;
    g.bands = (total_sub + g.sub - 1) / g.sub;
    g.plane_stride_px = smem_for(g);
  }
  // dilated, stride 1, padded by the dilation, planes small enough to stage a few whole: the residue-class walk
  const bool dilated = g.stride == 1 && g.dil > 1 && g.pt == g.dil && g.pl == g.dil && g.Ho == g.H && g.Wo == g.W && g.dil <= g.H &&
                       static_cast<long long>(g.Pin) * 8 <= budget;
  if (dilated) {
    g.sub = g.dil;                          // residue classes
    g.tr = (g.H + g.dil - 1) / g.dil;       // rows of the longest class
    g.bands = 1;
    long long planes = budget / (static_cast<long long>(g.Pin) * 8);
    if (planes > 8) planes = 8;
    g.nb = planes < g.B ? static_cast<int>(planes) : g.B;
    g.plane_stride_px = smem_for(g);
  }
  // the fast paths need the rows above and below the image to be at most one (zero rows in the buffer)
  const int overshoot = (g.Ho - 1) * g.stride - g.pt + 2 - (g.H - 1);
  const bool edge_ok = g.dil == 1 && g.pt <= 1 && overshoot <= 1;
  const int mode = dilated ? 3 : (edge_ok && g.stride == 1) ? 0 : (edge_ok && g.stride == 2) ? 1 : 2;
  // small planes, several per item, each walked top to bottom by its threads: stage them with one copy
  const bool packed = mode == 3 || (mode != 2 && g.bands == 1 && g.sub == 1 && g.nb > 4 && !pair);
  g.packed = packed ? 1 : 0;
  const size_t buf_bytes = packed ? static_cast<size_t>(g.Pin) * 8 * g.nb + 16 : static_cast<size_t>(g.plane_stride_px) * 8 * g.nb;
  // bytes in flight hide the HBM latency: two CTAs per SM (the register file allows no more),
  // each with up to three items requested ahead of the one it computes
  // small square planes, stride 1, one padding row / column on every side, a thread per whole column: straight-line stencil
  const bool whole_plane = packed && mode == 0 && !pair && g.H == g.W && g.pt == 1 && g.pl == 1 && g.Ho == g.H && g.Wo == g.W;
  // ... and 28-wide planes in bands of 14 rows per thread (staged with zero rows: not the one-copy mode)
  const bool band28 = !packed && mode == 0 && !pair && g.W == 28 && g.Wo == 28 && g.Ho == g.H && g.H % 14 == 0 && g.tr == 14 && g.pt == 1 && g.pl == 1;
  // ... and the two-columns-per-thread mode on 112- and 56-wide planes whose sub-bands are exactly 14 rows
  const bool pair14 = pair && mode == 0 && g.pt == 1 && g.tr == 14 && g.Ho % 14 == 0 && (g.W == 112 || g.W == 56);
  // ... and stride 2 without padding above / left on 112-, 56- and 28-wide planes whose bands are exactly 8 / 7 / 7 output rows
  const bool down = !packed && mode == 1 && g.pt == 0 && g.pl == 0 && (g.W == 112 || g.W == 56 || g.W == 28) && g.Wo == g.W / 2 &&
                    g.Ho == g.H / 2 && g.H % 2 == 0 && g.sub == 1 && g.tr == (g.W == 112 ? 8 : 7) && g.Ho % g.tr == 0;
  // ... and on whole 14 x 14 planes staged by one copy
  const bool down14 = packed && mode == 1 && g.pt == 0 && g.pl == 0 && g.W == 14 && g.H == 14 && g.Wo == 7 && g.Ho == 7;
  const int plane = whole_plane && g.H == 28 ? 28 : whole_plane && g.H == 14 ? 14 : whole_plane && g.H == 7 ? 7 : band28 ? 28 : pair14 ? g.W : down ? g.W : down14 ? 14 : 0;
  // the one-column straight-line variants need 80 registers: three CTAs per SM, so each gets a third of the shared memory
  const bool three_ctas = plane > 0 && !pair;
  const size_t per_cta = r.dw_cta_kb > 0 ? static_cast<size_t>(r.dw_cta_kb) * 1024
                                          : three_ctas ? static_cast<size_t>(73 * 1024) : static_cast<size_t>(kSmemPerCta);
  int nbuf = static_cast<int>(per_cta / buf_bytes);
  g.nbuf = nbuf > 4 ? 4 : nbuf < 2 ? 2 : nbuf;
  const size_t smem = buf_bytes * g.nbuf;
  if (smem > static_cast<size_t>(kMaxSmem)) return static_cast<int>(cudaErrorInvalidConfiguration);
  g.bchunks = (g.B + g.nb - 1) / g.nb;
  const long long items = static_cast<long long>(g.S) * g.bchunks * g.bands;
  if (items > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  g.items = static_cast<int>(items);
  if (dry_run) return 0;
  int threads = (g.nb * g.sub * wcols + 31) / 32 * 32;
  if (threads > 256) threads = 256;
  if (threads < 32) threads = 32;
  const int sms = device_sm_count();
  // persistent CTAs, a few per SM so that one CTA's copies overlap another's arithmetic
  long long ctas_per_sm = static_cast<long long>(kSmemPerSm) / static_cast<long long>(smem + 1024);
  if (ctas_per_sm > 2048 / threads) ctas_per_sm = 2048 / threads;
  // the grid is oversubscribed 2x: the block scheduler then evens out the tail
  ctas_per_sm *= 2;
  if (ctas_per_sm > 6) ctas_per_sm = 6;
  if (ctas_per_sm < 1) ctas_per_sm = 1;
  long long grid = static_cast<long long>(sms) * ctas_per_sm;
  if (grid > items) grid = items;
  const int act = r.ep.act_pre;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* in = static_cast<const __half*>(p.in0);
  const float* w = static_cast<const float*>(p.wts);
  const float* b = static_cast<const float*>(p.bias);
  const __half* res = static_cast<const __half*>(p.res);
  __half* out = static_cast<__half*>(p.out);
  static bool attr_done_dev[kMaxDevices][4][3][2][2][2][11] = {};
  bool(&attr_done)[4][3][2][2][2][11] = attr_done_dev[current_device_slot()];
  const bool tail = r.ep.has_res || r.ep.act_post != GI_ACT_NONE;
#define GI_DW_LAUNCH3(M, A, T, P, Q, PL, PLI)                                                                                 \
  do {                                                                                                                        \
    if (!attr_done[M][A][T][P][Q][PLI]) {                                                                                     \
      const cudaError_t e =                                                                                                   \
          cudaFuncSetAttribute(depthwise_f16_kernel<M, A, T, P, Q, PL>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem); \
      if (e != cudaSuccess) return static_cast<int>(e);                                                                       \
      attr_done[M][A][T][P][Q][PLI] = true;                                                                                   \
    }                                                                                                                         \
    launch_pdl(depthwise_f16_kernel<M, A, T, P, Q, PL>, static_cast<unsigned>(grid), threads, smem, st, in, w, b, res, out, g, r.ep); \
  } while (0)
#define GI_DW_LAUNCH2(M, A, T, P, Q)                  \
  do {                                                \
    if (M == 0 && P == 0 && Q == 1 && plane == 112) { \
      GI_DW_LAUNCH3(0, A, T, 0, 1, 112, 4);           \
    } else if (M == 0 && P == 0 && Q == 1 && plane == 56) { \
      GI_DW_LAUNCH3(0, A, T, 0, 1, 56, 5);            \
    } else if (M == 0 && P == 1 && Q == 0 && plane == 14) {  \
      GI_DW_LAUNCH3(0, A, T, 1, 0, 14, 1);            \
    } else if (M == 0 && P == 1 && Q == 0 && plane == 7) { \
      GI_DW_LAUNCH3(0, A, T, 1, 0, 7, 2);             \
    } else if (M == 0 && P == 1 && Q == 0 && plane == 28) { \
      GI_DW_LAUNCH3(0, A, T, 1, 0, 28, 10);           \
    } else if (M == 0 && P == 0 && Q == 0 && plane == 28) { \
      GI_DW_LAUNCH3(0, A, T, 0, 0, 28, 3);            \
    } else if (M == 1 && P == 0 && Q == 0 && plane == 112) { \
      GI_DW_LAUNCH3(1, A, T, 0, 0, 112, 6);           \
    } else if (M == 1 && P == 0 && Q == 0 && plane == 56) { \
      GI_DW_LAUNCH3(1, A, T, 0, 0, 56, 7);            \
    } else if (M == 1 && P == 0 && Q == 0 && plane == 28) { \
      GI_DW_LAUNCH3(1, A, T, 0, 0, 28, 8);            \
    } else if (M == 1 && P == 1 && Q == 0 && plane == 14) { \
      GI_DW_LAUNCH3(1, A, T, 1, 0, 14, 9);            \
    } else {                                          \
      GI_DW_LAUNCH3(M, A, T, P, Q, 0, 0);             \
    }                                                 \
  } while (0)
#define GI_DW_LAUNCH(M, A, T, P)            \
  do {                                      \
    if (M == 0 && P == 0 && pair) {         \
      GI_DW_LAUNCH2(0, A, T, 0, 1);         \
    } else {                                \
      GI_DW_LAUNCH2(M, A, T, P, 0);         \
    }                                       \
  } while (0)
#define GI_DW_ACT(M, A)       \
  do {                        \
    if (tail && packed) {        \
      GI_DW_LAUNCH(M, A, 1, 1);  \
    } else if (tail) {           \
      GI_DW_LAUNCH(M, A, 1, 0);  \
    } else if (packed) {         \
      GI_DW_LAUNCH(M, A, 0, 1);  \
    } else {                     \
      GI_DW_LAUNCH(M, A, 0, 0);  \
    }                            \
  } while (0)
#define GI_DW_MODE(M)              \
  do {                             \
    if (act == GI_ACT_RELU6) {     \
      GI_DW_ACT(M, GI_ACT_RELU6);  \
    } else if (act == GI_ACT_RELU) { \
      GI_DW_ACT(M, GI_ACT_RELU);   \
    } else {                       \
      GI_DW_ACT(M, GI_ACT_NONE);   \
    }                              \
  } while (0)
  if (mode == 0) {
    GI_DW_MODE(0);
  } else if (mode == 1) {
    GI_DW_MODE(1);
  } else if (mode == 3) {
    GI_DW_MODE(3);
  } else {
    GI_DW_MODE(2);
  }
#undef GI_DW_MODE
#undef GI_DW_ACT
#undef GI_DW_LAUNCH
#undef GI_DW_LAUNCH2
#undef GI_DW_LAUNCH3
  return static_cast<int>(cudaGetLastError());
}

int launch_depthwise_f16(const LaunchRec& r, const Ptrs& p, void* stream) { return depthwise_f16_impl(r, p, stream, false); }

// Host-only: the staged stencil can run this shape (its staging buffers fit shared memory, its work items an
// int).  Decided once at compile time; shapes it cannot run (rows thousands of pixels wide) take the plain
// one-thread-per-pixel kernel instead of failing in the middle of a run.
bool depthwise_f16_supported(const LaunchRec& r) {
  if (r.sh != r.sw || r.dh != r.dw) return false;
  return depthwise_f16_impl(r, Ptrs{}, nullptr, true) == 0;
}

unsigned int depthwise_error_word(int* cuda_err) {
  unsigned int v = 0;
  const cudaError_t e = cudaMemcpyFromSymbol(&v, g_dw_error, sizeof v);
  if (cuda_err) *cuda_err = static_cast<int>(e);
  return v;
}

}  // namespace gi
