// mbarrier / bulk-copy helpers shared by the pipelined kernels.  Every wait is
// bounded: when a barrier does not flip within ~2 s the waiting thread records
// HBL_ERR_TIMEOUT in the library's status word and raises the CTA's abort flag,
// which every other waiter polls.
#pragma once

#include "hbl_common.cuh"

namespace hbl {
namespace pipe {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// try_wait with a suspend-time hint: the hardware parks the thread until the phase completes or
// the hint runs out, instead of having it re-issue the instruction back to back.
__device__ __forceinline__ bool mbar_try_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
// Returns false when aborted (this thread's timeout, or another role's).
// POLITE waiters (anything but the thread that feeds the tensor core) park between polls so that
// they do not take issue slots from the warps that are on the critical path.
// limit_ns: how long the barrier may take to flip before the wait gives up (the kernels use the default).
constexpr uint64_t kWaitLimitNs = 2000000000ull;
template <bool POLITE = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try(bar, parity)) return true;
  if (*abort_flag) return false;
  const uint64_t t0 = global_ns();
  uint32_t polls = 0;
  for (;;) {
    if (POLITE ? mbar_try_hint(bar, parity, 2000u) : mbar_try(bar, parity)) return true;
    if (POLITE) __nanosleep(40);
    if ((++polls & (POLITE ? 15u : 255u)) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit_ns) {
        report_device_error(status, HBL_ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}
// Untiled bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), completing on `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

}  // namespace pipe
}  // namespace hbl
