// Entry points that exist only in the test build (-DSB_TEST_KERNELS); declared in include/specblock_test.h.
#ifdef SB_TEST_KERNELS

#include "tc_common.cuh"

namespace sb {

// The bounded wait of the tcgen05 kernels, run to its limit on purpose: warp 0 waits on an mbarrier
// that nobody ever arrives at, with the limit given by the caller; warp 1 waits on the same barrier with
// the ordinary two-second limit and must be released by the first warp's abort flag.  Nothing
// faults or hangs: both waits return false, the status word is set as the product kernels set it,
// and the kernel ends.
__global__ void __launch_bounds__(64) wait_expiry_kernel(unsigned long long limit_ns, int* status,
                                                         unsigned long long* elapsed_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  unsigned long long t0, t1;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  bool ok;
  if (threadIdx.x < 32) {
    ok = mbar_wait_poll(smem_u32(&bar), 0, &abort_flag, limit_ns);
  } else {
    ok = mbar_wait(&bar, 0, &abort_flag);
  }
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
  if (!ok) atomicMax(status, (int)SB_ERR_CUDA);
  if ((threadIdx.x & 31) == 0) elapsed_ns[threadIdx.x >> 5] = t1 - t0;
}

}  // namespace sb

extern "C" sb_status sb_test_wait_expires(int64_t limit_ns, int32_t* status, uint64_t* elapsed_ns, void* stream) {
  if (limit_ns < 1000 || limit_ns > 100000000 || !status || !elapsed_ns) return SB_ERR_INVALID_ARG;  // 1 us .. 100 ms
  sb::wait_expiry_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>((unsigned long long)limit_ns, status,
                                                                        reinterpret_cast<unsigned long long*>(elapsed_ns));
  return sb::launch_check();
}

#endif  // SB_TEST_KERNELS
