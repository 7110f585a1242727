// Library-wide entry points: status text, version, launch counter.
#include "common.cuh"

namespace sb {
long long g_launch_count = 0;
}

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
