// mbarrier and bulk-copy helpers shared by the kernels that stage data through shared memory
// (descent kernels, Hessian and int8 GEMM pipelines).  Every wait is bounded: it gives up after a
// number of clock cycles and reports that to the caller, who records kFlagWaitTimeout in the
// device status word, lets its copies in flight finish and returns.
#pragma once

#include <stdint.h>

namespace cdq {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// Makes the initialised barriers visible to the asynchronous proxy (the copy engine).
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// Waits for the phase with the given parity, at most `cycles` clock cycles.  False if it ran out.
__device__ __forceinline__ bool mbar_wait_cycles(uint32_t bar, uint32_t parity, long long cycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    if (mbar_try_wait(bar, parity)) return true;
  } while (clock64() - t0 < cycles);
  return false;
}
// The same with the 32-bit clock (fewer registers in a hot loop); cycles < 2^31.
__device__ __forceinline__ bool mbar_wait_clock32(uint32_t bar, uint32_t parity, unsigned cycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned t0 = (unsigned)clock();
  do {
    if (mbar_try_wait(bar, parity)) return true;
  } while ((unsigned)clock() - t0 < cycles);
  return false;
}
// Bounded wait for the pipelines whose roles (producer, MMA issuer, epilogue) give up together: false if the
// wait ran out (the flag is then set) or another role has already given up.
__device__ __forceinline__ bool mbar_wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                   uint32_t spin_limit) {
  for (uint32_t it = 0; it < spin_limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// tcgen05.commit: the mbarrier is arrived on once the MMAs issued so far have completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Generic-proxy writes to shared memory (a zero fill, say) before the copy engine touches it.
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// 1-D bulk copy global -> this CTA's shared memory, completion counted in bytes on `bar`.
// bytes % 16 == 0; both addresses 16-byte aligned.  No multicast.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

}  // namespace cdq
