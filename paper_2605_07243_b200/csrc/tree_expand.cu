// sb_tree_expand: per-row top-k over the drafter's scores and bucket-driven branching
// (Sec. 3.2; App. A.5 maps b(.); Alg. 1 "attach the top-b(bkt) tokens").
//
//   topk_partial_kernel : streams the [rows][vocab] fp32 scores once.  A CTA owns one (row, vocab
//                         chunk); each thread keeps its 16 best in registers (ids ascend inside a
//                         thread, so insertion only needs a strict compare against the current
//                         worst), the CTA then pops the 16 best of all threads in order.
//   expand_finish_kernel: one CTA: a warp per row merges the chunk lists (value descending, id
//                         ascending); then one thread walks the rows in order and appends the
//                         new nodes -- the append order is sequential by definition and touches at
//                         most `node_budget` (<= a few hundred) entries.
#include "common.cuh"

namespace sb {

constexpr int TOPK_THREADS = 256;
constexpr int kNoId = 0x7fffffff;

__device__ inline bool ranks_before(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

__global__ void __launch_bounds__(TOPK_THREADS) topk_partial_kernel(const float* __restrict__ scores,
                                                                    long long row_stride, int vocab, int chunk,
                                                                    int n_chunks, bool vec_ok,
                                                                    float* __restrict__ part_val,
                                                                    int* __restrict__ part_idx) {
  __shared__ float s_val[SB_KMAX][TOPK_THREADS];  // [rank][thread]: conflict-free per-thread lists
  __shared__ int s_idx[SB_KMAX][TOPK_THREADS];
  __shared__ float s_wv[TOPK_THREADS / 32];
  __shared__ int s_wi[TOPK_THREADS / 32], s_wt[TOPK_THREADS / 32];
  __shared__ int s_winner;
  const int row = blockIdx.y, c = blockIdx.x, tid = threadIdx.x;
  const float* base = scores + (long long)row * row_stride;
  const int begin = c * chunk;
  const int end = min(vocab, begin + chunk);

  float v[SB_KMAX];
  int id[SB_KMAX];
#pragma unroll
  for (int k = 0; k < SB_KMAX; ++k) { v[k] = -INFINITY; id[k] = kNoId; }

  auto offer = [&](float x, int xi) {
    x = score_of(x);
    if (!ranks_before(x, xi, v[SB_KMAX - 1], id[SB_KMAX - 1])) return;
    v[SB_KMAX - 1] = x;
    id[SB_KMAX - 1] = xi;
#pragma unroll
    for (int k = SB_KMAX - 1; k > 0; --k) {
      if (ranks_before(v[k], id[k], v[k - 1], id[k - 1])) {
        const float tv = v[k]; v[k] = v[k - 1]; v[k - 1] = tv;
        const int ti = id[k]; id[k] = id[k - 1]; id[k - 1] = ti;
      }
    }
  };

  if (vec_ok) {
    const int n_vec = max(0, (end - begin) / 4);
    const float4* vb = reinterpret_cast<const float4*>(base + begin);
    for (int t = tid; t < n_vec; t += TOPK_THREADS) {
      const float4 x = __ldg(vb + t);
      const int i0 = begin + 4 * t;
      offer(x.x, i0);
      offer(x.y, i0 + 1);
      offer(x.z, i0 + 2);
      offer(x.w, i0 + 3);
    }
    for (int i = begin + n_vec * 4 + tid; i < end; i += TOPK_THREADS) offer(base[i], i);
  } else {
    for (int i = begin + tid; i < end; i += TOPK_THREADS) offer(base[i], i);
  }
#pragma unroll
  for (int k = 0; k < SB_KMAX; ++k) { s_val[k][tid] = v[k]; s_idx[k][tid] = id[k]; }
  __syncthreads();

  // pop the CTA's best SB_KMAX in order
  int pos = 0;
  for (int round = 0; round < SB_KMAX; ++round) {
    float hv = pos < SB_KMAX ? s_val[pos][tid] : -INFINITY;
    int hi = pos < SB_KMAX ? s_idx[pos][tid] : kNoId;
    int ht = tid;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, hv, s);
      const int oi = __shfl_xor_sync(0xffffffffu, hi, s);
      const int ot = __shfl_xor_sync(0xffffffffu, ht, s);
      if (ranks_before(ov, oi, hv, hi)) { hv = ov; hi = oi; ht = ot; }
    }
    if ((tid & 31) == 0) { s_wv[tid >> 5] = hv; s_wi[tid >> 5] = hi; s_wt[tid >> 5] = ht; }
    __syncthreads();
    if (tid == 0) {
      float bv = s_wv[0];
      int bi = s_wi[0], bt = s_wt[0];
      for (int w = 1; w < TOPK_THREADS / 32; ++w)
        if (ranks_before(s_wv[w], s_wi[w], bv, bi)) { bv = s_wv[w]; bi = s_wi[w]; bt = s_wt[w]; }
      const long long o = ((long long)row * n_chunks + c) * SB_KMAX + round;
      part_val[o] = bv;
      part_idx[o] = bi;
      s_winner = bi == kNoId ? -1 : bt;
    }
    __syncthreads();
    if (tid == s_winner) ++pos;
  }
}

constexpr int FINISH_THREADS = 1024;

__global__ void __launch_bounds__(FINISH_THREADS) expand_finish_kernel(
    int n_rows, int n_chunks, const float* __restrict__ part_val, const int* __restrict__ part_idx, int block_k,
    const uint8_t* __restrict__ bucket, int4 bmap, const int* __restrict__ start_parent, int node_budget,
    int vocab, int* __restrict__ n_nodes, int* __restrict__ tok, int* __restrict__ parent, int* __restrict__ depth,
    int* __restrict__ node_row, int* __restrict__ node_rank, int* __restrict__ topk_tok,
    float* __restrict__ topk_val, int* __restrict__ status) {
  __shared__ int s_bad;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  // (1) merge the chunk lists of every row: lane c walks chunk c's sorted list
  for (int r = warp; r < n_rows; r += FINISH_THREADS / 32) {
    int pos = 0;
    const long long lb = ((long long)r * n_chunks + lane) * SB_KMAX;
    for (int round = 0; round < SB_KMAX; ++round) {
      const bool have = lane < n_chunks && pos < SB_KMAX;
      float hv = have ? part_val[lb + pos] : -INFINITY;
      int hi = have ? part_idx[lb + pos] : kNoId;
      int hl = lane;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, hv, s);
        const int oi = __shfl_xor_sync(0xffffffffu, hi, s);
        const int ol = __shfl_xor_sync(0xffffffffu, hl, s);
        if (ranks_before(ov, oi, hv, hi)) { hv = ov; hi = oi; hl = ol; }
      }
      if (lane == 0) {
        topk_tok[r * SB_KMAX + round] = hi == kNoId ? -1 : hi;
        topk_val[r * SB_KMAX + round] = hv;
      }
      if (hi != kNoId && lane == hl) ++pos;
    }
  }
  // (2) argument checks that need device data
  const int n0 = *n_nodes;
  if (threadIdx.x == 0 && (n0 < 0 || n0 > node_budget)) s_bad = 1;
  for (int r = threadIdx.x; r < n_rows; r += FINISH_THREADS)
    if (bucket[r] > 3) s_bad = 1;
  for (int i = threadIdx.x; i < n_rows / block_k; i += FINISH_THREADS)
    if (start_parent[i] < -1 || start_parent[i] >= n0) s_bad = 1;
  __syncthreads();
  if (s_bad) {
    if (threadIdx.x == 0) *status = SB_ERR_INVALID_ARG;
    return;
  }
  // (3) append in row order
  if (threadIdx.x == 0) {
    const int widths[4] = {bmap.x, bmap.y, bmap.z, bmap.w};
    int n = n0, chain = -1;
    bool chain_alive = false;
    for (int r = 0; r < n_rows; ++r) {
      const int kpos = r % block_k;
      int b = widths[bucket[r]];
      if (b > vocab) b = vocab;
      const int attach = kpos == 0 ? start_parent[r / block_k] : chain;
      const bool alive = kpos == 0 ? true : chain_alive;
      chain_alive = false;
      if (!alive) continue;
      for (int j = 0; j < b && n < node_budget; ++j) {
        tok[n] = topk_tok[r * SB_KMAX + j];
        parent[n] = attach;
        depth[n] = attach == -1 ? 0 : depth[attach] + 1;
        node_row[n] = r;
        node_rank[n] = j;
        if (j == 0) { chain = n; chain_alive = true; }
        ++n;
      }
    }
    *n_nodes = n;
    *status = SB_OK;
  }
}

static int topk_chunks(int n_rows, int vocab) {
  int nc = ceil_div(2 * 148, n_rows > 0 ? n_rows : 1);
  const int max_nc = ceil_div(vocab, 2048);
  if (nc > max_nc) nc = max_nc;
  if (nc > 32) nc = 32;
  if (nc < 1) nc = 1;
  return nc;
}

}  // namespace sb

extern "C" size_t sb_tree_expand_workspace_bytes(int32_t n_rows, int32_t vocab) {
  if (n_rows < 1 || vocab < 1) return 0;
  const size_t nc = (size_t)sb::topk_chunks(n_rows, vocab);
  return 2 * (((size_t)n_rows * nc * SB_KMAX * 4 + 255) & ~(size_t)255);
}

extern "C" sb_status sb_tree_expand(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                    int32_t block_k, const uint8_t* bucket, const int32_t* bmap,
                                    const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                                    int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                                    int32_t* node_rank, int32_t* topk_tok, float* topk_val, void* workspace,
                                    size_t workspace_bytes, int32_t* status, void* stream) {
  using namespace sb;
  if (!scores || !bucket || !bmap || !start_parent || !n_nodes || !tok || !parent || !depth || !node_row ||
      !node_rank || !topk_tok || !topk_val || !status || n_rows < 1 || vocab < 1 || row_stride < vocab ||
      block_k < 1 || n_rows % block_k != 0 || node_budget < 1)
    return SB_ERR_INVALID_ARG;
  for (int m = 0; m < 4; ++m)
    if (bmap[m] < 0 || bmap[m] > SB_KMAX) return SB_ERR_INVALID_ARG;
  if (n_rows > 65535) return SB_ERR_UNSUPPORTED;
  const size_t need = sb_tree_expand_workspace_bytes(n_rows, vocab);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int nc = topk_chunks(n_rows, vocab);
  int chunk = ceil_div(vocab, nc);
  chunk = ceil_div(chunk, 4) * 4;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(scores) & 15) == 0 && row_stride % 4 == 0;
  float* part_val = static_cast<float*>(workspace);
  int* part_idx = reinterpret_cast<int*>(static_cast<char*>(workspace) + need / 2);
  dim3 grid(nc, n_rows);
  topk_partial_kernel<<<grid, TOPK_THREADS, 0, cs>>>(scores, row_stride, vocab, chunk, nc, vec_ok, part_val,
                                                     part_idx);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  expand_finish_kernel<<<1, FINISH_THREADS, 0, cs>>>(n_rows, nc, part_val, part_idx, block_k, bucket,
                                                     make_int4(bmap[0], bmap[1], bmap[2], bmap[3]),
                                                     start_parent, node_budget, vocab, n_nodes, tok, parent,
                                                     depth, node_row, node_rank, topk_tok, topk_val, status);
  return launch_check();
}
