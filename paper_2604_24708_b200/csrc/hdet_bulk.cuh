// Bulk asynchronous copies between global and shared memory (sm_90+ `cp.async.bulk`, the untiled
// form of the tensor memory accelerator) and the shared-memory barriers that track them.
//
// Every copy stays inside one CTA and one GPU: the destination of a load is the issuing CTA's own
// shared memory, no cluster is launched and no copy is sent to more than one CTA.  Rules of the
// instruction: both addresses 16-byte aligned, size a multiple of 16 bytes.
//
// Every wait in this file is bounded: a barrier that does not complete within about a second makes
// the wait return false, and the caller records that in the status word and leaves the tile.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace hdet {
namespace bulk {

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void barrier_init(uint32_t bar, uint32_t arrivals) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(arrivals) : "memory");
}

// Makes freshly initialised barriers visible to the copy engine.
__device__ __forceinline__ void barrier_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// One arrival that also announces `bytes` of copy traffic the barrier has to see before it completes.
__device__ __forceinline__ void barrier_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void barrier_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool barrier_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}

// Longest time any wait spins: 2e9 SM cycles, about a second.
constexpr long long kWaitLimitCycles = 2000000000ll;

// Waits for the phase with the given parity.  Returns false once the limit has passed.
__device__ __forceinline__ bool barrier_wait(uint32_t bar, uint32_t parity, long long limit_cycles = kWaitLimitCycles) {
  if (barrier_try_wait(bar, parity)) return true;
  const long long start = clock64();
  for (;;) {
    for (int i = 0; i < 32; ++i)
      if (barrier_try_wait(bar, parity)) return true;
    if (clock64() - start > limit_cycles) return false;
  }
}

// global -> this CTA's shared memory; completion is counted in bytes on `bar`.
__device__ __forceinline__ void load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// shared -> global, tracked by the issuing thread's bulk groups.
__device__ __forceinline__ void store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ void commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

// Blocks until the stores committed so far have finished READING shared memory (the data may still
// be on its way to global memory; visibility at kernel end is guaranteed as for any store).
__device__ __forceinline__ void wait_stores_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Orders a thread's ordinary shared-memory writes before later copies issued by the copy engine.
__device__ __forceinline__ void publish_smem_writes() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

}  // namespace bulk
}  // namespace hdet
