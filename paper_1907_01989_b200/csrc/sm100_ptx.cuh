// Thin wrappers over the sm_100a PTX used by the tensor-core kernels: mbarriers with bounded
// waits, TMA (tiled and untiled bulk copies), tcgen05 MMA / commit / tensor-memory management.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

namespace gi {
namespace ptx {

__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false if the CTA is aborting or the limit ran out (then it raises the
// abort flag and sets `code` in the sticky device error word itself).
static __device__ __noinline__ bool mbar_wait_slow(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                            unsigned* error_word, unsigned code) {
  unsigned long long t0 = 0;
  for (unsigned spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 255u) == 255u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > timeout_ns) {
        *abort_flag = 1;
        atomicOr(error_word, code);
        return false;
      }
    }
  }
}

// The wait every role uses: a phase that has already completed - the common case for a consumer that runs behind its
// producer - is recognised by one inline poll; only a real wait pays for the call into the polling routine.  (The
// single MMA-issuing thread of a kernel executes its instructions one dependent step at a time: shortening its path
// per chunk took the wide-tile 1x1 kernel from 622 to 728 TFLOP/s.)
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                          unsigned* error_word, unsigned code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, timeout_ns, error_word, code);
}

// The same bounded wait for a single thread that waits most of the time (a copy or MMA-issuing thread): each
// poll may sleep in hardware for up to a microsecond and returns as soon as the phase completes, so the
// waiting thread takes no issue slots from the warps that compute.  Used where the compute warps are bound by
// instruction issue (the depthwise + 1x1 kernel); in the other tensor-core kernels it measured 0.3-0.7 %
// slower than the plain poll on every network, so they keep mbar_wait.
static __device__ __noinline__ bool mbar_wait_parked(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                              unsigned* error_word, unsigned code) {
  unsigned long long t0 = 0;
  for (unsigned spin = 0;; ++spin) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000u)
        : "memory");
    if (ok) return true;
    if ((spin & 15u) == 15u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > timeout_ns) {
        *abort_flag = 1;
        atomicOr(error_word, code);
        return false;
      }
    }
  }
}
// The same wait for a whole warp that goes on to warp-collective instructions (tcgen05.ld / .st / .wait are
// .sync.aligned: all 32 lanes must execute them together).  Lanes leave the polling loop at different
// iterations; the vote brings them back together and gives every lane the same answer, so that the warp
// also gives up as one.  A phase that has already completed - the common case for a consumer that runs behind
// its producer - is recognised by one inline poll, without the call into the bounded-wait routine.
// (Letting one lane poll for the warp, with a warp barrier and a shuffle behind it, measured slower: +1 us per
// kernel at batch 1.)
__device__ __forceinline__ bool mbar_wait_warp(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                               unsigned* error_word, unsigned code) {
  const bool ok = mbar_wait(bar, parity, abort_flag, timeout_ns, error_word, code);
  return __all_sync(0xffffffffu, ok) != 0;
}

__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
// start fetching a tensor map (a kernel parameter) so that the first tiled copy does not wait for it
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(map)) : "memory");
}
// L2 eviction policy "evict first": for tensors nobody reads again, so that the lines this kernel
// writes (the next kernel's input) are the ones that stay in L2
__device__ __forceinline__ unsigned long long policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar, unsigned long long pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
               "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(unsigned smem_dst, unsigned cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, 128 x N x 16, fp16 operands, fp32 accumulate
__device__ __forceinline__ void umma_f16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned idesc,
                                         unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on an mbarrier once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory operand descriptor: K-major, no swizzle.  Core matrices are 8 rows x 16 bytes,
// stored as 128 contiguous bytes; `lbo` is the byte distance between the two core matrices
// an MMA reads along K, `sbo` the distance between consecutive 8-row groups.
__device__ __forceinline__ unsigned long long smem_desc(unsigned addr, unsigned lbo, unsigned sbo) {
  unsigned long long d = 0;
  d |= static_cast<unsigned long long>((addr & 0x3ffffu) >> 4);
  d |= static_cast<unsigned long long>((lbo >> 4) & 0x3fffu) << 16;
  d |= static_cast<unsigned long long>((sbo >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  return d;         // base offset 0, layout type 0 (no swizzle)
}

// two floats -> packed fp16 (x in the low half), round to nearest even; RELU folds max(., 0) into
// the conversion instruction
template <bool RELU>
__device__ __forceinline__ unsigned pack_f16x2(float x, float y) {
  unsigned d;
  if (RELU) asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(y), "f"(x));
  else asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(y), "f"(x));
  return d;
}

// 32 lanes x 16 consecutive 32-bit columns: thread t of the warp receives lane (quarter*32 + t)
__device__ __forceinline__ void tmem_ld16(unsigned taddr, unsigned* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// wait for every tensor-memory load issued so far; the registers of the chunk about to be used
// are operands so that no use of them can be scheduled above the wait
__device__ __forceinline__ void tmem_ld_wait16(unsigned* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}

// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
  unsigned pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- CTA pairs (a cluster of two CTAs on the two SMs that share one tensor-core pair) -------------------------
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// hardware barrier over all threads of the cluster; every thread of both CTAs must reach it
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the address of `addr` (a shared-memory address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ unsigned mapa_shared(unsigned addr, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// arrive on an mbarrier of any CTA of the cluster; what this thread wrote before is visible to the waiter
__device__ __forceinline__ void mbar_arrive_cluster(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// poll an mbarrier of this CTA that the other CTA of the pair arrives on
__device__ __forceinline__ bool mbar_try_wait_cluster(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking tests of a phase (try_wait may suspend the thread for a while when the phase is not complete):
// for a thread that has other work to issue first and looks at the answer later.
__device__ __forceinline__ bool mbar_test_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait_cluster(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait on such a barrier (same contract as mbar_wait)
static __device__ __noinline__ bool mbar_wait_cluster_slow(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                                    unsigned* error_word, unsigned code) {
  unsigned long long t0 = 0;
  for (unsigned spin = 0;; ++spin) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((spin & 255u) == 255u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > timeout_ns) {
        *abort_flag = 1;
        atomicOr(error_word, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait_cluster(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                                  unsigned* error_word, unsigned code) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  return mbar_wait_cluster_slow(bar, parity, abort_flag, timeout_ns, error_word, code);
}
__device__ __forceinline__ bool mbar_wait_cluster_warp(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                                       unsigned* error_word, unsigned code) {
  const bool ok = mbar_wait_cluster(bar, parity, abort_flag, timeout_ns, error_word, code);
  return __all_sync(0xffffffffu, ok) != 0;
}
// The parked form of that wait (see mbar_wait_parked): each poll may sleep in hardware for up to a microsecond
// and returns as soon as the phase completes.  For roles that wait most of the time - a warp that spins on a
// barrier floods the shared-memory pipeline that also feeds the tensor core its operands.
static __device__ __noinline__ bool mbar_wait_cluster_parked(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                                      unsigned* error_word, unsigned code) {
  unsigned long long t0 = 0;
  for (unsigned spin = 0;; ++spin) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000u)
        : "memory");
    if (ok) return true;
    if ((spin & 15u) == 15u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > timeout_ns) {
        *abort_flag = 1;
        atomicOr(error_word, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait_cluster_parked_warp(unsigned bar, unsigned parity, volatile unsigned* abort_flag,
                                                              unsigned timeout_ns, unsigned* error_word, unsigned code) {
  const bool ok = mbar_wait_cluster_parked(bar, parity, abort_flag, timeout_ns, error_word, code);
  return __all_sync(0xffffffffu, ok) != 0;
}
__device__ __forceinline__ bool mbar_wait_parked_warp(unsigned bar, unsigned parity, volatile unsigned* abort_flag, unsigned timeout_ns,
                                                      unsigned* error_word, unsigned code) {
  const bool ok = mbar_wait_parked(bar, parity, abort_flag, timeout_ns, error_word, code);
  return __all_sync(0xffffffffu, ok) != 0;
}
// Tensor memory of both CTAs of a pair, same columns in each: one warp of EACH CTA executes these
__device__ __forceinline__ void tmem_alloc_pair(unsigned smem_dst, unsigned cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(unsigned taddr, unsigned cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D (+)= A * B^T over the pair, 256 x N x 16: each CTA supplies 128 rows of A and N/2 rows of B from its own shared
// memory (same offsets in both) and receives its 128 rows of D in its own tensor memory.  Issued by one thread of
// the pair's first CTA.
__device__ __forceinline__ void umma_pair_f16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned idesc,
                                              unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on an mbarrier of either CTA (cluster address) once every pair MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_pair_commit(unsigned cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr) : "memory");
}

}  // namespace ptx
}  // namespace gi
