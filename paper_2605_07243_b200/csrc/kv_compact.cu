// sb_kv_compact: keep the committed path's K/V right behind the prefix (Sec. 3.1 / App. A.2: later
// forwards see every committed position's cached keys and values as the verified prefix).
//
// cache[P + j] <- cache[P + path[j]] for j = 0..accept_len, in place, every layer, K and V.  A path
// is strictly increasing with path[0] = 0, so path[j] >= j: a destination slot is never the source
// of a LATER copy, only possibly of an earlier one.  Each thread owns one 16-byte column of the
// row for all j and moves the rows in groups of eight (eight loads, then eight stores), ascending:
// every source is read before the copy that overwrites it, and no two threads touch the same
// bytes, so no barrier is needed.
#include "common.cuh"

namespace sb {

constexpr int COMPACT_THREADS = 128;
constexpr int COMPACT_GROUP = 8;

__global__ void __launch_bounds__(COMPACT_THREADS) kv_compact_kernel(const sb_tree_batch tb, int n_layers,
                                                                     long long layer_stride_elems,
                                                                     const int* __restrict__ path_nodes,
                                                                     const int* __restrict__ accept_len,
                                                                     int max_depth, int* __restrict__ new_len,
                                                                     int* __restrict__ status) {
  __shared__ int s_path[SB_MAX_DEPTH + 1];
  __shared__ int s_err;
  const int b = blockIdx.z;
  const int layer = blockIdx.y >> 1, is_v = blockIdx.y & 1;
  const int o = tb.node_offsets[b];
  const int n = tb.node_offsets[b + 1] - o;
  const int P = tb.prefix_len[b];
  const int a = accept_len[b];
  if (threadIdx.x == 0) {
    int err = 0;
    if (n < 1 || n > SB_MAX_NODES || a < 0 || a > max_depth) {
      err = SB_ERR_INVALID_TREE;
    } else {
      const int* path = path_nodes + (long long)b * (max_depth + 1);
      for (int j = 0; j <= a; ++j) {
        const int pj = path[j];
        s_path[j] = pj;
        if (j == 0 ? pj != 0 : (pj <= s_path[j - 1] || pj >= n)) err = SB_ERR_INVALID_TREE;
      }
      if (!err) {
        const long long last = (long long)P + s_path[a];
        if (P < 0 || (tb.page_size == 0 ? last >= tb.kv_capacity
                                         : last >= (long long)tb.max_pages * tb.page_size))
          err = SB_ERR_BOUNDS;
      }
      if (!err && tb.page_size > 0) {
        for (int j = 0; j <= a; ++j) {
          const int page = tb.page_table[(long long)b * tb.max_pages + (P + s_path[j]) / tb.page_size];
          const int page2 = tb.page_table[(long long)b * tb.max_pages + (P + j) / tb.page_size];
          if (page < 0 || page >= tb.num_pages || page2 < 0 || page2 >= tb.num_pages) err = SB_ERR_BOUNDS;
        }
      }
    }
    s_err = err;
    if (blockIdx.x == 0 && blockIdx.y == 0) {
      status[b] = err;
      new_len[b] = err ? P : P + a + 1;
    }
  }
  __syncthreads();
  if (s_err) return;
  const int units = tb.n_kv_heads * tb.head_dim / 8;  // 16-byte columns of one cache row
  const int u = blockIdx.x * COMPACT_THREADS + threadIdx.x;
  if (u >= units) return;
  uint16_t* cache = static_cast<uint16_t*>(const_cast<void*>(is_v ? tb.v_cache : tb.k_cache)) +
                    (long long)layer * layer_stride_elems;
  for (int j0 = 1; j0 <= a; j0 += COMPACT_GROUP) {  // j = 0 maps the root onto itself
    uint4 regs[COMPACT_GROUP];
#pragma unroll
    for (int t = 0; t < COMPACT_GROUP; ++t) {
      const int j = j0 + t;
      if (j <= a) {
        const long long src = kv_row_elem_offset(tb, b, P + s_path[j]) + u * 8;
        if (SB_CHECKED_ACCESS(src + 7, kv_cache_elems(tb), &status[b])) regs[t] = *reinterpret_cast<const uint4*>(cache + src);
      }
    }
#pragma unroll
    for (int t = 0; t < COMPACT_GROUP; ++t) {
      const int j = j0 + t;
      if (j <= a && s_path[j] != j) {
        const long long dst = kv_row_elem_offset(tb, b, P + j) + u * 8;
        if (SB_CHECKED_ACCESS(dst + 7, kv_cache_elems(tb), &status[b])) *reinterpret_cast<uint4*>(cache + dst) = regs[t];
      }
    }
  }
}

// sb_path_rows: one CTA per sequence; thread j looks up the row of path node j, thread 0 checks the order.
__global__ void __launch_bounds__(64) path_rows_kernel(const int* __restrict__ node_offsets,
                                                       const int* __restrict__ node_row,
                                                       const int* __restrict__ row_begin,
                                                       const int* __restrict__ path_nodes,
                                                       const int* __restrict__ accept_len, int max_depth,
                                                       int* __restrict__ path_rows, int* __restrict__ status) {
  __shared__ int s_rows[SB_MAX_DEPTH + 1];
  __shared__ int s_err;
  const int b = blockIdx.x, j = threadIdx.x;
  const int o = node_offsets[b];
  const int n = node_offsets[b + 1] - o;
  const int a = accept_len[b];
  const int r0 = row_begin ? row_begin[b] : 0;
  const bool shape_ok = n >= 1 && a >= 0 && a <= max_depth;
  if (j == 0) s_err = shape_ok ? 0 : (int)SB_ERR_INVALID_TREE;
  __syncthreads();
  if (j <= max_depth) {
    int row = -1;
    if (shape_ok && j <= a) {
      const int self = path_nodes[(long long)b * (max_depth + 1) + j];
      if (self < 0 || self >= n) atomicExch(&s_err, (int)SB_ERR_INVALID_TREE);
      if (j == 0) {
        row = 0;
      } else {
        const int nr = (self >= 0 && self < n) ? node_row[o + self] : -1;
        if (nr < r0 || nr < 0) atomicExch(&s_err, (int)SB_ERR_INVALID_TREE);
        else row = 1 + nr - r0;
      }
    }
    s_rows[j] = row;
  }
  __syncthreads();
  if (j == 0 && !s_err)
    for (int t = 1; t <= a; ++t)
      if (s_rows[t] <= s_rows[t - 1]) s_err = SB_ERR_INVALID_TREE;
  __syncthreads();
  if (j <= max_depth) path_rows[(long long)b * (max_depth + 1) + j] = s_err ? (j == 0 ? 0 : -1) : s_rows[j];
  if (j == 0) status[b] = s_err;
}

}  // namespace sb

extern "C" sb_status sb_path_rows(int32_t batch, const int32_t* node_offsets, const int32_t* node_row,
                                  const int32_t* row_begin, const int32_t* path_nodes, const int32_t* accept_len,
                                  int32_t max_depth, int32_t* path_rows, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_path_rows");
  using namespace sb;
  if (batch < 1 || !node_offsets || !node_row || !path_nodes || !accept_len || !path_rows || !status)
    return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH) return SB_ERR_UNSUPPORTED;
  path_rows_kernel<<<batch, 64, 0, static_cast<cudaStream_t>(stream)>>>(node_offsets, node_row, row_begin, path_nodes,
                                                                        accept_len, max_depth, path_rows, status);
  return launch_check();
}

extern "C" sb_status sb_kv_compact(const sb_tree_batch* tb, int32_t n_layers, int64_t layer_stride_elems,
                                   const int32_t* path_nodes, const int32_t* accept_len, int32_t max_depth,
                                   int32_t* new_len, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_kv_compact");
  using namespace sb;
  if (!tb || tb->batch < 1 || !tb->k_cache || !tb->v_cache || !tb->prefix_len || !tb->node_offsets ||
      !path_nodes || !accept_len || !new_len || !status || n_layers < 1 || tb->n_kv_heads < 1)
    return SB_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(tb->k_cache) & 15) || (reinterpret_cast<uintptr_t>(tb->v_cache) & 15) ||
      (layer_stride_elems % 8) != 0 || layer_stride_elems < 0)
    return SB_ERR_INVALID_ARG;
  if (tb->head_dim < 8 || tb->head_dim % 8 != 0) return SB_ERR_UNSUPPORTED;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH) return SB_ERR_UNSUPPORTED;
  if (tb->page_size < 0) return SB_ERR_INVALID_ARG;
  if (tb->page_size > 0 && (!tb->page_table || tb->max_pages < 1 || tb->num_pages < 1)) return SB_ERR_INVALID_ARG;
  if (tb->page_size == 0 && tb->kv_capacity < 1) return SB_ERR_INVALID_ARG;
  if (2 * (long long)n_layers > 65535 || tb->batch > 65535) return SB_ERR_UNSUPPORTED;
  const int units = tb->n_kv_heads * tb->head_dim / 8;
  dim3 grid(ceil_div(units, COMPACT_THREADS), 2 * n_layers, tb->batch);
  kv_compact_kernel<<<grid, COMPACT_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      *tb, n_layers, layer_stride_elems, path_nodes, accept_len, max_depth, new_len, status);
  return launch_check();
}
