// hbl_selftest_wait_timeout: makes one of the library's bounded device-side waits run out, on purpose and
// harmlessly, so that the path every pipelined kernel takes when a barrier never flips -- record
// HBL_ERR_TIMEOUT, raise the thread block's abort flag, let the other roles leave their waits, drain, free the
// tensor memory, return -- can be exercised on a GPU.  The kernel waits, with a short limit, on an mbarrier
// that nobody ever arrives at; nothing traps, nothing faults, and no wait is unbounded.
#include "hbl_pipeline.cuh"

namespace hbl {
namespace {

using namespace pipe;

__global__ void __launch_bounds__(96, 1) wait_timeout_kernel(int* status, unsigned long long limit_ns, int* left_by_abort) {
  __shared__ __align__(8) uint64_t never_bar;      // one arrival expected, none ever made
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(&never_bar, 1);
    abort_flag_s = 0;
    mbar_fence_init();
  }
  if (warp == 1) {                                  // the contraction kernels hold tensor memory while they wait: so does this one
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(32) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // the role whose wait runs out: reports the timeout and raises the abort flag
    if (lane == 0) (void)mbar_wait<false>(&never_bar, 0, abort_flag, status, limit_ns);
  } else if (warp == 2) {
    // a second role, parked on the same barrier with the kernels' own limit: it must leave because of the
    // abort flag, long before its own limit
    const bool got = __all_sync(0xffffffffu, mbar_wait<true>(&never_bar, 0, abort_flag, status));
    if (lane == 0 && !got && *abort_flag) *left_by_abort = 1;
  }

  // teardown, as in the pipelined kernels
  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32) : "memory");
  }
}

}  // namespace
}  // namespace hbl

using namespace hbl;

extern "C" int hbl_selftest_wait_timeout(int limit_us, int* left_by_abort, void* stream) {
  if (limit_us <= 0 || limit_us > 1000000) return HBL_ERR_SHAPE;      // at most one second
  if (!left_by_abort) return HBL_ERR_NULL;
  int* status = device_status_word();
  if (status == nullptr) return HBL_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  HBL_CUDA_OK(cudaMemsetAsync(left_by_abort, 0, sizeof(int), s));
  wait_timeout_kernel<<<1, 96, 0, s>>>(status, (unsigned long long)limit_us * 1000ull, left_by_abort);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}
