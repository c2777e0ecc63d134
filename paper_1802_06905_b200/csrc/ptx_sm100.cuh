// PTX wrappers for sm_100a (mbarrier, TMA, tcgen05 / TMEM) shared by the tensor-core kernels.
// Everything here is a thin inline wrapper; waits are bounded (see mbar_wait*).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.h"

namespace cconv {
namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P1;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, P1;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up when another role raised the CTA's abort flag or when the time limit
// passes; on expiry it records `code` in the global status word and raises the abort flag.
// The polling loop is kept out of line so that the callers' loop bodies stay small.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            int* status, int code, uint64_t limit_ns) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((i & 63u) == 63u) {
      const uint64_t t = globaltimer_ns();
      if (t0 == 0) {
        t0 = t;
      } else if (t - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(status, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int code, uint64_t limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, code, limit_ns);
}
// Wait used by warps whose 32 lanes walk a loop together (the MMA issuer, the epilogue).
// Two measured rules shape it (each cost almost 2x in tcgen05 issue rate when broken):
//  * EVERY lane polls the barrier itself -- no "lane 0 polls, then warp sync";
//  * nothing is called: a function call anywhere in the issuing loop, even on a path that never
//    runs, slows the whole loop, so the time-limit check is inline and rare.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity,
                                               volatile int* abort_flag, int* status, int code,
                                               uint64_t limit_ns) {
  uint64_t t0 = 0;
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 0x3FFFu) == 0u) {
      if (*abort_flag) return false;
      const uint64_t t = globaltimer_ns();
      if (t0 == 0) {
        t0 = t;
      } else if (t - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(status, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                            int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                            int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
// Tensor store shared -> global (bulk async-group completion): the box at `src` in shared memory
// goes to coordinates (c0..c3) of the tensor; elements outside the tensor's extents are not written.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1,
                                             int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
          reinterpret_cast<uint64_t>(tm)),
      "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void bulk_commit_group() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Waits until all but the latest N bulk groups of this thread have read their shared-memory source
// (`_read`) or are complete (their writes performed).
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_group() {
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// Orders this thread's earlier shared-memory writes before later asynchronous-proxy reads of them.
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem], executed only where `issue` is true (the warp stays converged).
__device__ __forceinline__ void umma_bf16_if(bool issue, uint32_t d_tmem, uint64_t a_desc,
                                             uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.ne.b32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(uint32_t(issue))
      : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
// ---- straight-line groups of MMAs: two adds per instruction instead of rebuilding both descriptors ----
// Nine taps of one 16-channel step of a 3x3 filter in one instruction block: Filter blocks
// a_lo + t*4 KB, Image views b_lo + off[t].  a_lo / b_lo are descriptor low words (address >> 4 already merged
// with the constant fields); only lane `issue` issues; `accumulate` applies to tap 0, the rest add.
__device__ __forceinline__ void umma_taps9_bh1(
    bool issue, uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
    uint32_t idesc, uint32_t accumulate, const uint32_t (&off)[9]) {
  asm volatile(
      "{\n\t.reg .pred p, q, pt;\n\t.reg .b64 ad, bd;\n\t.reg .b32 a, b, d2;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "setp.ne.b32 q, %7, 0;\n\t"
      "setp.eq.b32 pt, %5, %5;\n\t"
      "mov.b64 ad, {%1, %2};\n\t"
      "mov.b64 bd, {%3, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t"
      "add.u32 a, %1, 256;\n\t"
      "add.u32 b, %3, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 512;\n\t"
      "add.u32 b, %3, %9;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 768;\n\t"
      "add.u32 b, %3, %10;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1024;\n\t"
      "add.u32 b, %3, %11;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1280;\n\t"
      "add.u32 b, %3, %12;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1536;\n\t"
      "add.u32 b, %3, %13;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1792;\n\t"
      "add.u32 b, %3, %14;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 2048;\n\t"
      "add.u32 b, %3, %15;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "}"
      ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
      "r"(uint32_t(issue)), "r"(off[1]), "r"(off[2]), "r"(off[3]), "r"(off[4]), "r"(off[5]), "r"(off[6]),
      "r"(off[7]), "r"(off[8])
      : "memory");
}

// Nine taps of one 16-channel step of a 3x3 filter in one instruction block: Filter blocks
// a_lo + t*4 KB, Image views b_lo + off[t] and b_lo + off[t] + hstep (second output row, accumulator
// d + n_mma).  a_lo / b_lo are descriptor low words (address >> 4 already merged
// with the constant fields); only lane `issue` issues; `accumulate` applies to tap 0, the rest add.
__device__ __forceinline__ void umma_taps9_bh2(
    bool issue, uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
    uint32_t idesc, uint32_t accumulate, const uint32_t (&off)[9], uint32_t hstep, uint32_t n_mma) {
  asm volatile(
      "{\n\t.reg .pred p, q, pt;\n\t.reg .b64 ad, bd;\n\t.reg .b32 a, b, d2;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "setp.ne.b32 q, %7, 0;\n\t"
      "setp.eq.b32 pt, %5, %5;\n\t"
      "add.u32 d2, %0, %17;\n\t"
      "mov.b64 ad, {%1, %2};\n\t"
      "mov.b64 bd, {%3, %4};\n\t"
      "mov.b32 b, %3;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, p;\n\t"
      "add.u32 a, %1, 256;\n\t"
      "add.u32 b, %3, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 512;\n\t"
      "add.u32 b, %3, %9;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 768;\n\t"
      "add.u32 b, %3, %10;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1024;\n\t"
      "add.u32 b, %3, %11;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1280;\n\t"
      "add.u32 b, %3, %12;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1536;\n\t"
      "add.u32 b, %3, %13;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 1792;\n\t"
      "add.u32 b, %3, %14;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 2048;\n\t"
      "add.u32 b, %3, %15;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b, b, %16;\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "}"
      ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
      "r"(uint32_t(issue)), "r"(off[1]), "r"(off[2]), "r"(off[3]), "r"(off[4]), "r"(off[5]), "r"(off[6]),
      "r"(off[7]), "r"(off[8]), "r"(hstep), "r"(n_mma)
      : "memory");
}

// 4 consecutive K=16 steps of a 1x1 filter: Filter blocks a_lo + u*4 KB, Image views b_lo + u*kstep.
__device__ __forceinline__ void umma_run4_bh1(
    bool issue, uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
    uint32_t idesc, uint32_t accumulate, uint32_t kstep) {
  asm volatile(
      "{\n\t.reg .pred p, q, pt;\n\t.reg .b64 ad, bd;\n\t.reg .b32 a, b, b2, d2;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "setp.ne.b32 q, %7, 0;\n\t"
      "setp.eq.b32 pt, %5, %5;\n\t"
      "mov.b32 b, %3;\n\t"
      "mov.b64 ad, {%1, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t"
      "add.u32 a, %1, 256;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 512;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 768;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "}"
      ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
      "r"(uint32_t(issue)), "r"(kstep)
      : "memory");
}

// 4 consecutive K=16 steps of a 1x1 filter: Filter blocks a_lo + u*4 KB, Image views b_lo + u*kstep (and + hstep into d + n_mma).
__device__ __forceinline__ void umma_run4_bh2(
    bool issue, uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
    uint32_t idesc, uint32_t accumulate, uint32_t kstep, uint32_t hstep, uint32_t n_mma) {
  asm volatile(
      "{\n\t.reg .pred p, q, pt;\n\t.reg .b64 ad, bd;\n\t.reg .b32 a, b, b2, d2;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "setp.ne.b32 q, %7, 0;\n\t"
      "setp.eq.b32 pt, %5, %5;\n\t"
      "mov.b32 b, %3;\n\t"
      "add.u32 d2, %0, %10;\n\t"
      "mov.b64 ad, {%1, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t"
      "add.u32 b2, b, %9;\n\t"
      "mov.b64 bd, {b2, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, p;\n\t"
      "add.u32 a, %1, 256;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b2, b, %9;\n\t"
      "mov.b64 bd, {b2, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 512;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b2, b, %9;\n\t"
      "mov.b64 bd, {b2, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "add.u32 a, %1, 768;\n\t"
      "add.u32 b, b, %8;\n\t"
      "mov.b64 ad, {a, %2};\n\t"
      "mov.b64 bd, {b, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, pt;\n\t"
      "add.u32 b2, b, %9;\n\t"
      "mov.b64 bd, {b2, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [d2], ad, bd, %5, pt;\n\t"
      "}"
      ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate),
      "r"(uint32_t(issue)), "r"(kstep), "r"(hstep), "r"(n_mma)
      : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
// True in exactly one (always the same) lane of a fully active warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 32-byte store: one full sector per lane (sm_100 has 256-bit global stores)
__device__ __forceinline__ void st_global_v8(void* ptr, uint32_t a0, uint32_t a1, uint32_t a2,
                                             uint32_t a3, uint32_t a4, uint32_t a5, uint32_t a6,
                                             uint32_t a7) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(ptr), "r"(a0),
               "r"(a1), "r"(a2), "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7)
               : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(uint32_t lo_f32_bits, uint32_t hi_f32_bits) {
  const __nv_bfloat162 v =
      __floats2bfloat162_rn(__uint_as_float(lo_f32_bits), __uint_as_float(hi_f32_bits));
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Four lanes of a quad each hold four 8-word (32-byte) sectors of their own accumulator row.
// After the call lane q of the quad holds sector q of the quad's rows 0..3 (slot j = row j): a 4x4
// transpose of sectors in two butterfly stages of warp shuffles.  With it the four lanes of a quad
// write one whole 128-byte line of ONE row per store instruction, and a warp eight whole lines,
// instead of 32 lanes writing one sector each to 32 different lines (one per out-channel plane),
// which the memory system absorbs at well under half the rate.
__device__ __forceinline__ void quad_transpose_sectors(uint32_t (&s)[4][8], int lane) {
  const bool b0 = lane & 1, b1 = lane & 2;
#pragma unroll
  for (int c = 0; c < 4; c += 2) {
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const uint32_t send = b0 ? s[c][w] : s[c + 1][w];
      const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
      if (b0) s[c][w] = recv; else s[c + 1][w] = recv;
    }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const uint32_t send = b1 ? s[i][w] : s[2 + i][w];
      const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 2);
      if (b1) s[i][w] = recv; else s[2 + i][w] = recv;
    }
  }
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst),
      "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}

// After the main loop a producer must not leave while its copies may still be landing.
__device__ __forceinline__ void drain_ring(uint32_t bar_full0, uint32_t it, uint32_t stages,
                                           int* status, uint64_t limit) {
  const uint32_t back = it < stages ? it : stages;
  for (uint32_t j = 0; j < back; ++j) {
    const uint32_t i2 = it - 1 - j;
    const uint32_t s = i2 % stages;
    const uint32_t ph = (i2 / stages) & 1u;
    const uint64_t t0 = globaltimer_ns();
    while (!mbar_try_wait(bar_full0 + 8u * s, ph)) {
      if (globaltimer_ns() - t0 > limit) {
        atomicOr(status, kStatDrainWait);
        break;
      }
    }
  }
}

}  // namespace

// ---- thread-block clusters and distributed shared memory ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Hardware barrier over all threads of all CTAs of the cluster; release/acquire orders the
// distributed-shared-memory stores issued before it against the loads issued after it.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The address of this CTA's shared-memory location `local` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t cluster_map_shared(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c,
                                              uint32_t d) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b),
               "r"(c), "r"(d)
               : "memory");
}
// Asynchronous copy from this CTA's shared memory into a peer CTA's (both addresses and the size
// multiples of 16 bytes); the bytes are credited to the PEER's mbarrier `bar_cluster`.
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster, uint32_t src_local,
                                                  uint32_t bytes, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst_cluster),
      "r"(src_local), "r"(bytes), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c,
                                             uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d)
               : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c,
                                             uint32_t& d) {
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}

}  // namespace cconv
