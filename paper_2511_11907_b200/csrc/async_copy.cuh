// Shared-memory staging primitives for sm_100a: mbarrier phases, bulk asynchronous copies
// (cp.async.bulk, the untiled TMA path) and programmatic dependent launch.
//
// Every wait is bounded: a wait that does not complete within kWaitTries attempts returns
// false, and the caller records an error word and leaves its loop, so that no kernel of this
// library can spin forever.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace kvswap {

constexpr uint32_t kWaitTries = 1u << 20;     // attempts per wait (each suspends briefly in hardware)

// Device error words (written to the first word of the workspace, read by
// kvswap_read_device_status).
enum : uint32_t {
  kDevOk = 0,
  kDevTimeoutFull = 1,    // a consumer waited for staged data that never arrived
  kDevTimeoutEmpty = 2,   // the producer waited for a stage that was never released
  kDevBadIndex = 3,       // KVSWAP_CHECK_INDICES: a group index or count out of range was skipped or clamped
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous proxy.
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// Bounded wait for the phase with the given parity.  Returns false on timeout.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitTries; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

// Bulk copy global -> this CTA's shared memory; completion is counted in bytes on `bar`.
// dst, src and bytes must be multiples of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// Programmatic dependent launch: `pdl_wait` blocks until every kernel this launch depends on has
// completed and its writes are visible (a no-op for an ordinary launch); `pdl_trigger` lets the
// next kernel in the stream begin its own prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace kvswap
