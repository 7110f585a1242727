// sb_tree_ancestors: ancestor bitmask and depth of every tree node (App. A.2, Fig. 4).
// One CTA per sequence; a tree has at most 128 nodes, so this is latency-only work.
#include "common.cuh"

namespace sb {

__global__ void __launch_bounds__(128) tree_ancestors_kernel(int batch, const int* __restrict__ node_offsets,
                                                             const int* __restrict__ parent, int max_nodes,
                                                             uint32_t* __restrict__ anc_mask,
                                                             int* __restrict__ depth, int* __restrict__ status) {
  __shared__ int s_parent[SB_MAX_NODES];
  __shared__ uint32_t s_anc[SB_MAX_NODES * 4];
  __shared__ int s_depth[SB_MAX_NODES];
  const int b = blockIdx.x;
  const int o = node_offsets[b];
  int n = node_offsets[b + 1] - o;
  // A count outside the limits cannot be indexed safely: report it and write nothing.
  if (n < 0 || n > max_nodes || n > SB_MAX_NODES || o < 0) {
    if (threadIdx.x == 0) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  const bool ok = build_ancestors_smem(parent + o, n, s_parent, s_anc, s_depth);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    if (anc_mask) {
      uint4 m = ok ? make_uint4(s_anc[4 * i], s_anc[4 * i + 1], s_anc[4 * i + 2], s_anc[4 * i + 3])
                   : make_uint4(0, 0, 0, 0);
      reinterpret_cast<uint4*>(anc_mask)[o + i] = m;
    }
    if (depth) depth[o + i] = ok ? s_depth[i] : 0;
  }
  if (threadIdx.x == 0) status[b] = ok ? SB_OK : SB_ERR_INVALID_TREE;
}

}  // namespace sb

extern "C" sb_status sb_tree_ancestors(int32_t batch, const int32_t* node_offsets, const int32_t* parent,
                                       int32_t max_nodes, uint32_t* anc_mask, int32_t* depth,
                                       int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_tree_ancestors");
  if (batch < 1 || !node_offsets || !parent || !status) return SB_ERR_INVALID_ARG;
  if (max_nodes < 1 || max_nodes > SB_MAX_NODES) return SB_ERR_UNSUPPORTED;
  if (anc_mask && (reinterpret_cast<uintptr_t>(anc_mask) & 15)) return SB_ERR_INVALID_ARG;
  sb::tree_ancestors_kernel<<<batch, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      batch, node_offsets, parent, max_nodes, anc_mask, depth, status);
  return sb::launch_check();
}
