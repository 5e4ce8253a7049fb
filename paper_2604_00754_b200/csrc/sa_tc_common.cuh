// Thin wrappers over the sm_100a instructions the tensor-core kernels are built from:
// mbarriers with bounded waits, proxy and tcgen05 fences, tcgen05.mma / commit / ld / st,
// and the descriptor words.  Everything here is file-local to its includer.
#pragma once

#include "sa_common.cuh"

namespace sa {
namespace {

constexpr long long kWaitCycles = 2000000000ll;  // bound of every mbarrier wait: about a second

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the limit ran out or another thread already gave up.
// try_wait that lets the hardware park the thread for up to `ns` nanoseconds while the phase
// is incomplete, instead of returning at once: a waiting warp then costs next to no issue slots.
__device__ __forceinline__ bool mbar_try_parked(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* gave_up,
                                          int* status, long long limit = kWaitCycles) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_parked(bar, parity, 2000u)) return true;
    if (*gave_up) return false;
    if (clock64() - t0 > limit) {
      *gave_up = 1;
      atomicCAS(status, SA_OK, SA_ERR_TIMEOUT);
      return false;
    }
  }
}

// Should this CTA leave without doing its work?  Yes when an earlier check rejected perm/inv
// (abort_flag) or some CTA has already recorded a timeout: the rest of the grid then leaves at
// once instead of each waiting out its own limit.  Thread 0 alone reads the two words, once,
// in its set-up block, and leaves the answer in `slot` (an int in shared memory); after the
// kernel's first __syncthreads every thread reads the same answer there, whatever another
// kernel writes to the status word in the meantime.
__device__ __forceinline__ void note_skip(volatile int* slot, const int* status,
                                          const int* abort_flag) {
  *slot = (abort_flag && *(volatile const int*)abort_flag) ||
          *(volatile const int*)status == SA_ERR_TIMEOUT;
}
// After that __syncthreads: leave (the allocating warp hands its tensor memory back first).
#define SA_LEAVE_IF_SKIPPED(slot, alloc_warp, tmem, cols)                                     \
  if (*(slot)) {                                                                              \
    if (warp == (alloc_warp)) {                                                               \
      tc_fence_after();                                                                       \
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem),       \
                   "r"((uint32_t)(cols)) : "memory");                                         \
    }                                                                                         \
    return;                                                                                   \
  }

// Orders shared-memory writes made through the generic proxy (cp.async) that this thread
// has observed before its later tensor-core reads of the same memory.
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}
// Four consecutive K steps (16 elements each) of D (+)= A B^T with both operands in shared
// memory; each step moves both descriptors on by 32 bytes inside the 128-byte swizzle row.
// Written as one block so that the issuing thread spends three instructions per product.
__device__ __forceinline__ void mma_ss_x4(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc,
                                          uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "setp.ne.b32 p0, %4, 0;\n\tsetp.eq.b32 p1, %3, %3;\n\t"
      "add.u64 a1, %1, 2;\n\tadd.u64 b1, %2, 2;\n\t"
      "add.u64 a2, %1, 4;\n\tadd.u64 b2, %2, 4;\n\t"
      "add.u64 a3, %1, 6;\n\tadd.u64 b3, %2, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %3, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %3, p1;\n\t}"
      ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc0)
      : "memory");
}
// Four consecutive K steps of D (+)= A B with A (bf16 pairs, 8 columns per step) in tensor
// memory and B in shared memory, 16 rows (2048 bytes) further on each step.
__device__ __forceinline__ void mma_ts_x4(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc,
                                          uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
      "setp.ne.b32 p0, %4, 0;\n\tsetp.eq.b32 p1, %3, %3;\n\t"
      "add.u32 a1, %1, 8;\n\tadd.u64 b1, %2, 128;\n\t"
      "add.u32 a2, %1, 16;\n\tadd.u64 b2, %2, 256;\n\t"
      "add.u32 a3, %1, 24;\n\tadd.u64 b3, %2, 384;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a1], b1, %3, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a2], b2, %3, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a3], b3, %3, p1;\n\t}"
      ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0)
      : "memory");
}

#define SA_R8(v, o) "=r"(v[o]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), \
                    "=r"(v[o + 4]), "=r"(v[o + 5]), "=r"(v[o + 6]), "=r"(v[o + 7])
#define SA_W8(v, o) "r"(v[o]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), \
                    "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7])

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : SA_R8(v, 0), SA_R8(v, 8), SA_R8(v, 16), SA_R8(v, 24)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
      ::SA_W8(v, 0), SA_W8(v, 8), SA_W8(v, 16), SA_W8(v, 24), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&v)[8]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
      ::SA_W8(v, 0), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::SA_W8(v, 0), SA_W8(v, 8), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// ---------------------------------------------------------------------- descriptors

__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}

// Shared-memory matrix descriptor (128-byte swizzle): bits 0-13 start address, 16-29 leading
// byte offset, 32-45 stride byte offset (all in 16-byte units), bit 46 descriptor version 1
// (sm_100), bits 61-63 layout type 2.  The issuer assembles it from two prepared words.
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

}  // namespace
}  // namespace sa
