// Asynchronous bulk copies from global to shared memory and the mbarriers that count their bytes.
// Every wait is bounded: a wait that runs out returns false, the caller reports ACCEPT_DEV_COPY_TIMEOUT
// and leaves; no kernel of this library can spin for ever.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace accept {

__device__ __forceinline__ uint32_t smem_address(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbarrier_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbarrier_expect_bytes(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbarrier_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_copy_to_shared(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// How long a wait for an asynchronous copy may last.  A copy lands within microseconds; the limit only has
// to outlast the time a kernel may sit descheduled on a GPU that is time-sliced between processes (the
// timer keeps running meanwhile), which is a matter of milliseconds.
#ifdef ACCEPT_TEST_COPY_STALL
// Tests-only build: every stage announces 16 bytes more than its copies deliver, so all copies land but no
// phase ever completes; the waits run out (after 2 ms) and the kernel must report it and leave cleanly.
constexpr unsigned long long kCopyWaitNs = 2000000ull;
constexpr uint32_t kCopyAnnounceExtra = 16u;
#else
constexpr unsigned long long kCopyWaitNs = 200000000ull;
constexpr uint32_t kCopyAnnounceExtra = 0u;
#endif

// Waits for the phase of the given parity; gives up after kCopyWaitNs.
__device__ __forceinline__ bool mbarrier_wait(uint32_t bar, uint32_t parity) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if ((it & 63u) == 63u) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > kCopyWaitNs) return false;
    }
  }
}

}  // namespace accept
