/*
 * Entry points of the TEST build (libspecblock_test.so, compiled with -DSB_TEST_KERNELS) and of the
 * CHECKED build (libspecblock_checked.so, -DSB_CHECKED) of the SpecBlock library.  The library proper
 * (libspecblock.so) exports none of them.  The paper has no
 * counterpart for anything here: these are checks of the implementation's own safety nets.
 */
#ifndef SPECBLOCK_TEST_H
#define SPECBLOCK_TEST_H

#include "specblock.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * sb_test_wait_expires -- lets the bounded device-side wait of the tensor-core kernels run out.
 *   Launches one CTA of two warps on `stream`.  Warp 0 waits on an mbarrier that nobody arrives at and
 *   gives up after limit_ns (1 us .. 100 ms); warp 1 waits on the same barrier with the library's
 *   ordinary limit (two seconds) and is released early by the abort flag warp 0 sets.  Both then record
 *   the failure exactly as the product kernels do: *status (device int32, caller-zeroed) becomes
 *   SB_ERR_CUDA.  elapsed_ns (device uint64[2]) receives how long each warp waited.  Nothing faults,
 *   traps or hangs; the context stays usable.  Returns SB_ERR_INVALID_ARG for a limit outside the
 *   range or NULL pointers.
 */
sb_status sb_test_wait_expires(int64_t limit_ns, int32_t* status, uint64_t* elapsed_ns, void* stream);

/*
 * sb_checked_violations -- checked build only.  In that build every index a kernel computes from
 *   device data (page ids, cache slots, query/output rows, workspace offsets, node ids) is verified
 *   against the extent of what it indexes right before the access; a violation skips the access,
 *   counts, and sets SB_ERR_BOUNDS in the call's status word where the kernel does not overwrite it
 *   later.  This call synchronises the device, returns the number of refused accesses since the last
 *   call in *count (host int64) and clears the counter.  A correct library on valid inputs gives 0.
 */
sb_status sb_checked_violations(int64_t* count);

/*
 * sb_checked_selftest -- checked build only: shows that the guard fires.  One thread makes one access
 *   inside a 4-element extent and one just past it.  status: device int32[2], caller-zeroed; afterwards
 *   status[0] == SB_ERR_BOUNDS, status[1] == 1 (only the in-range access ran) and
 *   sb_checked_violations() reads 1.
 */
sb_status sb_checked_selftest(int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif

#endif
