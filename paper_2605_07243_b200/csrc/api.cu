// Library-wide entry points: status text, version, launch counter.
#include "common.cuh"

namespace sb {
long long g_launch_count = 0;
#ifdef SB_CHECKED
// Accesses the checked build refused (one counter for every kernel of the library: this build is
// compiled with relocatable device code so that all source files share it).
__device__ unsigned long long g_checked_violations = 0;
#endif
}

#ifdef SB_CHECKED
// Checked build only (declared in include/specblock_test.h): number of accesses refused since the
// last call, read after synchronising the device; the counter is cleared.
extern "C" sb_status sb_checked_violations(int64_t* count) {
  if (!count) return SB_ERR_INVALID_ARG;
  unsigned long long v = 0, zero = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpyFromSymbol(&v, sb::g_checked_violations, sizeof(v)) != cudaSuccess ||
      cudaMemcpyToSymbol(sb::g_checked_violations, &zero, sizeof(zero)) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  *count = (int64_t)v;
  return SB_OK;
}

namespace sb {
__global__ void checked_selftest_kernel(int* status) {
  // one access inside its extent, one just past it: the second must be refused and counted
  if (SB_CHECKED_ACCESS(3, 4, status)) status[1] = 1;
  if (SB_CHECKED_ACCESS(4, 4, status)) status[1] = 2;
}
}  // namespace sb

// Checked build only: proves that the guard fires.  status: device int32[2], caller-zeroed; afterwards
// status[0] == SB_ERR_BOUNDS, status[1] == 1 (only the in-range access ran), and the counter reads 1.
extern "C" sb_status sb_checked_selftest(int32_t* status, void* stream) {
  if (!status) return SB_ERR_INVALID_ARG;
  sb::checked_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(status);
  return sb::launch_check();
}
#endif

extern "C" const char* sb_status_string(sb_status s) {
  switch (s) {
    case SB_OK: return "ok";
    case SB_ERR_INVALID_ARG: return "invalid argument";
    case SB_ERR_UNSUPPORTED: return "unsupported shape or limit";
    case SB_ERR_WORKSPACE: return "workspace too small";
    case SB_ERR_INVALID_TREE: return "invalid tree";
    case SB_ERR_BOUNDS: return "position or page outside the cache";
    case SB_ERR_CUDA: return "CUDA call failed";
  }
  return "unknown status";
}

extern "C" int32_t sb_version(void) { return 100; }

extern "C" int64_t sb_kernel_launch_count(void) { return sb::g_launch_count; }
