// Shared device/host helpers of the SpecBlock CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include <atomic>

#include <nvtx3/nvToolsExt.h>

#include "../../include/specblock.h"

namespace sb {

// NVTX range around an entry point: a profiler's timeline shows which call enqueued which kernels
// (header-only NVTX; costs a few nanoseconds when no tool is attached).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// Host-side count of kernel launches made by this library (read by benchmarks).
extern long long g_launch_count;

inline sb_status launch_check() {
  ++g_launch_count;
  return cudaGetLastError() == cudaSuccess ? SB_OK : SB_ERR_CUDA;
}

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Experiment switches exist only in the test build (-DSB_TEST_KERNELS); the library proper reads no
// environment variable, on the launch path or anywhere else.
#ifdef SB_TEST_KERNELS
inline const char* test_knob(const char* name) { return getenv(name); }
#else
inline const char* test_knob(const char*) { return nullptr; }
#endif

// Kernel attributes (dynamic shared memory, cluster size) and occupancy figures belong to a device,
// not to the process: caches of them are arrays indexed by the current device.  -1: no usable device.
constexpr int kMaxDevices = 64;
inline int device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return -1;
  }
  return dev;
}
// One-time set-up of the current device (cudaFuncSetAttribute and the like).  `fn` returns true on
// success and must be idempotent: two host threads that meet here for the first time may both run it.
struct PerDeviceOnce {
  std::atomic<int> done[kMaxDevices];
  template <typename F>
  bool run(F fn) {
    const int dev = device_slot();
    if (dev < 0) return false;
    if (done[dev].load(std::memory_order_acquire)) return true;
    if (!fn()) return false;
    done[dev].store(1, std::memory_order_release);
    return true;
  }
};
// A small integer fact of the current device, computed on first use (-1 = not known yet).
struct PerDeviceInt {
  std::atomic<int> value_plus_1[kMaxDevices];  // zero-initialised: 0 = unknown
  template <typename F>
  int get(F compute, int fallback) {
    const int dev = device_slot();
    if (dev < 0) return fallback;
    int v = value_plus_1[dev].load(std::memory_order_acquire);
    if (v == 0) {
      v = compute() + 1;
      value_plus_1[dev].store(v, std::memory_order_release);
    }
    return v - 1;
  }
};

// Programmatic dependent launch.  A kernel started with launch_dependent() may begin while its
// predecessor in the stream is still running; it must execute pdl_wait() before it reads anything
// the predecessor writes (and always before it ends, so that completion stays transitive along
// the stream).  The predecessor lets it start early with pdl_release().
__device__ inline void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ inline void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline sb_status launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t cs, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

// Checked build (-DSB_CHECKED, libspecblock_checked.so): every index a kernel computes from device
// data -- page ids, cache slots, query/output rows, workspace offsets -- is verified against the extent
// of what it indexes right before the access.  A violation sets SB_ERR_BOUNDS in the call's status
// word and the access is skipped.  The library proper compiles the test away.  (This pool has no
// compute-sanitizer; this build plus canary-padded buffers in the tests stand in for it.)
#ifdef SB_CHECKED
extern __device__ unsigned long long g_checked_violations;  // api.cu; read and cleared by sb_checked_violations()
__device__ inline bool checked_access(long long idx, long long limit, int* status_word) {
  if (idx >= 0 && idx < limit) return true;
  atomicAdd(&g_checked_violations, 1ull);
  if (status_word) atomicMax(status_word, (int)SB_ERR_BOUNDS);  // a kernel's own final status may overwrite this
  return false;
}
#define SB_CHECKED_ACCESS(idx, limit, status_word) ::sb::checked_access((long long)(idx), (long long)(limit), (status_word))
#else
#define SB_CHECKED_ACCESS(idx, limit, status_word) true
#endif

// Elements of one layer of a K or V cache.
__host__ __device__ inline long long kv_cache_elems(const sb_tree_batch& tb) {
  const long long rows = tb.page_size == 0 ? (long long)tb.batch * tb.kv_capacity : (long long)tb.num_pages * tb.page_size;
  return rows * tb.n_kv_heads * tb.head_dim;
}

// Per-sequence facts every CTA of a sequence derives identically from device data.
struct SeqInfo {
  int n;       // tree nodes
  int P;       // prefix length
  int q0;      // first node with a query row
  int q_off;   // first row of this sequence in q / out
  int nq;      // query nodes
  int err;     // 0 or an sb_status for this sequence (tree shape and lengths only)
};

// Length/shape checks that need no pass over arrays.
__device__ inline SeqInfo load_seq_info(const sb_tree_batch& tb, const int* q_node_begin,
                                        const int* q_offsets, int total_q, int b) {
  SeqInfo s;
  const int o = tb.node_offsets[b];
  s.n = tb.node_offsets[b + 1] - o;
  s.P = tb.prefix_len[b];
  s.q0 = q_node_begin ? q_node_begin[b] : 0;
  s.q_off = q_offsets ? q_offsets[b] : o;
  s.nq = s.n - s.q0;
  s.err = 0;
  if (s.n < 0 || s.n > tb.max_nodes || s.n > SB_MAX_NODES || o < 0 ||
      (long long)o + s.n > tb.total_nodes || s.q0 < 0 || s.q0 > s.n) {
    s.err = SB_ERR_INVALID_TREE;
  } else if (s.P < 0 || (long long)s.P + s.n > tb.max_kv_len ||
             (tb.page_size == 0 ? (long long)s.P + s.n > tb.kv_capacity
                                : (long long)s.P + s.n > (long long)tb.max_pages * tb.page_size) ||
             s.q_off < 0 || (long long)s.q_off + s.nq > total_q) {
    s.err = SB_ERR_BOUNDS;
  }
  if (s.err) { s.n = 0; s.nq = 0; s.P = 0; }
  return s;
}

// The threads that run a planning helper together: the whole CTA, or its first `n` threads (a multiple
// of 32) meeting at named barrier 1 while the CTA's other warps do something else.
struct ThreadGroup {
  int tid, n;
  bool whole_cta;
  __device__ void sync() const {
    if (whole_cta) __syncthreads();
    else asm volatile("bar.sync 1, %0;" ::"r"(n) : "memory");
  }
};
__device__ inline ThreadGroup whole_cta() { return ThreadGroup{(int)threadIdx.x, (int)blockDim.x, true}; }
__device__ inline ThreadGroup first_threads(int n) { return ThreadGroup{(int)threadIdx.x, n, false}; }

// Builds anc[i] = {i} U anc[parent[i]] for one tree into shared memory (4 words per node) and
// returns false for an invalid tree.  `s_parent` is scratch of n ints.  Every thread of the
// group must call it; it contains barriers of the group.
__device__ inline bool build_ancestors_smem(const int* __restrict__ parent_g, int n, int* s_parent, uint32_t* s_anc,
                                            int* s_depth, const ThreadGroup grp = whole_cta()) {
  __shared__ int s_bad;
  if (grp.tid == 0) s_bad = 0;
  grp.sync();
  for (int i = grp.tid; i < n; i += grp.n) {
    const int p = parent_g[i];
    s_parent[i] = p;
    if (p < -1 || p >= i) s_bad = 1;
  }
  grp.sync();
  const bool ok = s_bad == 0;
  for (int i = grp.tid; i < n; i += grp.n) {
    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;
    int d = -1;
    if (ok) {
      // parent[a] < a for every a, so the walk ends after at most n steps
      for (int a = i; a >= 0; a = s_parent[a]) {
        const uint32_t bit = 1u << (a & 31);
        const int w = a >> 5;
        m0 |= w == 0 ? bit : 0u;
        m1 |= w == 1 ? bit : 0u;
        m2 |= w == 2 ? bit : 0u;
        m3 |= w == 3 ? bit : 0u;
        ++d;
      }
    }
    s_anc[4 * i + 0] = m0;
    s_anc[4 * i + 1] = m1;
    s_anc[4 * i + 2] = m2;
    s_anc[4 * i + 3] = m3;
    if (s_depth) s_depth[i] = d < 0 ? 0 : d;
  }
  grp.sync();
  return ok;
}

// Element offset (in bf16 elements) of cache row (sequence b, logical position j), kv head 0.
// Bad page ids are clamped to page 0 so that no access leaves the pool; the sequence's
// designated CTA reports them.
__device__ inline long long kv_row_elem_offset(const sb_tree_batch& tb, int b, int j) {
  long long row;
  if (tb.page_size == 0) {
    row = (long long)b * tb.kv_capacity + j;
  } else {
    const int lp = j / tb.page_size;
    int page = tb.page_table[(long long)b * tb.max_pages + lp];
    if (page < 0 || page >= tb.num_pages) page = 0;
    row = (long long)page * tb.page_size + (j - lp * tb.page_size);
  }
  return row * tb.n_kv_heads * (long long)tb.head_dim;
}

// True when every page the sequence's [0, len) positions need is inside the pool.
__device__ inline bool pages_in_pool(const sb_tree_batch& tb, int b, int len, const ThreadGroup grp = whole_cta()) {
  if (tb.page_size == 0) return true;
  __shared__ int s_bad_page;
  if (grp.tid == 0) s_bad_page = 0;
  grp.sync();
  const int need = ceil_div(len, tb.page_size);
  for (int p = grp.tid; p < need; p += grp.n) {
    const int page = tb.page_table[(long long)b * tb.max_pages + p];
    if (page < 0 || page >= tb.num_pages) s_bad_page = 1;
  }
  grp.sync();
  return s_bad_page == 0;
}

__device__ inline float bf16_bits_to_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// NaN takes part in max / top-k as -infinity.
__device__ inline float score_of(float x) { return x != x ? -INFINITY : x; }

}  // namespace sb
