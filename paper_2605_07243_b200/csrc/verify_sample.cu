// sb_verify_sample: stochastic verification of a draft tree at temperature T > 0 by multi-candidate
// rejection sampling (Sec. 4.1 evaluates "temperature 0 and 1.0"; Sec. 4.2 "rejection sampling
// against a high-entropy target").  The paper names the procedure only; the order of the steps is
// the one stated in include/specblock.h.
//
//   verify_sample_kernel : a cluster of 8 CTAs per sequence walks its tree from the root, all CTAs
//                       taking the same decisions from the same data.  The target distribution p of
//                       the current node and the draft distribution q that proposed its children live
//                       unnormalised in a workspace (2 x vocab floats per sequence, L2-resident) next
//                       to their sums, so p(x) / q(x) is two loads.  The vocabulary is cut into 256
//                       contiguous segments, one per warp of the cluster; sums and maxima are reduced
//                       per CTA and exchanged through distributed shared memory (every CTA adds the
//                       eight partials in rank order).  A rejection is one pass that measures
//                       max(p - q, 0) and one that writes it; the bonus token is drawn by an ordered
//                       prefix search (segment totals, then a shuffle scan row by row inside the
//                       segment that holds the target mass).  All random numbers are inputs.
#include <cooperative_groups.h>

#include "common.cuh"

namespace sb {
namespace cg = cooperative_groups;

constexpr int VS_THREADS = 1024;
constexpr int VS_CLUSTER = 8;
constexpr int VS_WARPS = VS_THREADS / 32;
constexpr int VS_SEGS = VS_CLUSTER * VS_WARPS;  // vocabulary segments, one per warp of the cluster
constexpr float kVsLog2e = 1.4426950408889634f;

// Cluster-wide reductions.  Each CTA reduces its threads, thread 0 stores the CTA's partial into
// slot [rank] of EVERY CTA's exchange array (distributed shared memory), and after a cluster
// barrier every thread combines the eight partials in rank order: all threads of the cluster get
// the same value.  The exchange array is double-buffered (`flip`): a buffer is rewritten two
// reductions later, when every CTA has passed the barrier that followed its last read.
struct ClusterRed {
  float* s_warp;  // [VS_WARPS]
  float* s_cl;    // [2][VS_CLUSTER]
  int flip;
};
template <bool IS_MAX>
__device__ inline float vs_cluster_reduce(float v, ClusterRed& cr, cg::cluster_group& cluster) {
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    const float o = __shfl_xor_sync(0xffffffffu, v, sft);
    v = IS_MAX ? fmaxf(v, o) : v + o;
  }
  __syncthreads();  // s_warp may still be read from the previous reduction
  if ((threadIdx.x & 31) == 0) cr.s_warp[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    float r = cr.s_warp[0];
    for (int w = 1; w < VS_WARPS; ++w) r = IS_MAX ? fmaxf(r, cr.s_warp[w]) : r + cr.s_warp[w];
    float* slot = cr.s_cl + cr.flip * VS_CLUSTER + cluster.block_rank();
    for (int k = 0; k < VS_CLUSTER; ++k) *cluster.map_shared_rank(slot, k) = r;
  }
  cluster.sync();
  const float* part = cr.s_cl + cr.flip * VS_CLUSTER;
  float r = part[0];
  for (int k = 1; k < VS_CLUSTER; ++k) r = IS_MAX ? fmaxf(r, part[k]) : r + part[k];
  cr.flip ^= 1;
  return r;
}

template <typename T>
__device__ inline float vs_value(const T* row, int v);
template <>
__device__ inline float vs_value<float>(const float* row, int v) { return score_of(row[v]); }
template <>
__device__ inline float vs_value<uint16_t>(const uint16_t* row, int v) { return score_of(bf16_bits_to_float(row[v])); }

// dst[v] = exp((row[v] - max) / T) over this warp's segment [v_begin, v_end) (1 everywhere when the
// row has no finite value); returns the sum over the whole vocabulary.
template <typename T>
__device__ float vs_load_softmax(const T* row, int v_begin, int v_end, float inv_t, float* dst, ClusterRed& cr,
                                 cg::cluster_group& cluster) {
  const int lane = threadIdx.x & 31;
  float m = -INFINITY;
  for (int v = v_begin + lane; v < v_end; v += 32) m = fmaxf(m, vs_value<T>(row, v));
  m = vs_cluster_reduce<true>(m, cr, cluster);
  float z = 0.f;
  const float k = inv_t * kVsLog2e;
  for (int v = v_begin + lane; v < v_end; v += 32) {
    const float e = m == -INFINITY ? 1.f : exp2f((vs_value<T>(row, v) - m) * k);
    dst[v] = e;
    z += e;
  }
  return vs_cluster_reduce<false>(z, cr, cluster);
}

__global__ void __launch_bounds__(VS_THREADS) verify_sample_kernel(
    const void* __restrict__ logits, int dtype, long long row_stride, int vocab, const float* __restrict__ scores,
    long long score_stride, int n_rows, int total_nodes, const int* __restrict__ node_offsets,
    const int* __restrict__ parent, const int* __restrict__ tok, const int* __restrict__ child_row, float inv_t,
    const float* __restrict__ u_accept, const float* __restrict__ u_bonus, int max_depth, int* __restrict__ accept_len,
    int* __restrict__ path_nodes, int* __restrict__ out_tokens, int* __restrict__ bonus, float* work,
    int* __restrict__ status) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ int s_parent[SB_MAX_NODES], s_tok[SB_MAX_NODES], s_kids[SB_MAX_NODES];
  __shared__ float s_warp[VS_WARPS];
  __shared__ float s_cl[2 * VS_CLUSTER];
  __shared__ float s_seg[VS_SEGS];  // segment totals of the whole cluster (every CTA holds a copy)
  __shared__ int s_nk, s_take, s_bad, s_seg_of;
  __shared__ float s_need, s_qx;
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int crank = (int)cluster.block_rank();
  const bool writer = crank == 0 && tid == 0;  // the one thread that writes the per-sequence outputs
  ClusterRed cr = {s_warp, s_cl, 0};
  const int o = node_offsets[b];
  const int n = node_offsets[b + 1] - o;
  int* path = path_nodes + (long long)b * (max_depth + 1);
  int* otok = out_tokens + (long long)b * (max_depth + 1);
  if (crank == 0)
    for (int t = tid; t <= max_depth; t += VS_THREADS) { path[t] = -1; otok[t] = -1; }
  if (tid == 0) s_bad = 0;
  if (writer) { accept_len[b] = 0; bonus[b] = -1; }
  __syncthreads();
  // every CTA of the cluster takes the same exits: the data below is the same for all of them
  if (n < 1 || n > SB_MAX_NODES || o < 0 || (long long)o + n > total_nodes) {
    if (writer) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  if (tid < n) {
    const int p = parent[o + tid];
    s_parent[tid] = p;
    s_tok[tid] = tok[o + tid];
    if (tid == 0 ? p != -1 : (p < 0 || p >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (writer) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  float* pw = work + (long long)b * 2 * vocab;  // target distribution, unnormalised: p = pw / zp
  float* qw = pw + vocab;                       // draft distribution, unnormalised: q = qw / zq
  // this warp's contiguous segment of the vocabulary
  const int seg_len = ceil_div(ceil_div(vocab, VS_SEGS), 32) * 32;
  const int seg_id = crank * VS_WARPS + warp;
  const int v_begin = min(vocab, seg_id * seg_len), v_end = min(vocab, (seg_id + 1) * seg_len);
  auto load_target = [&](int node) {
    return dtype == SB_BF16
               ? vs_load_softmax(static_cast<const uint16_t*>(logits) + (long long)(o + node) * row_stride, v_begin,
                                 v_end, inv_t, pw, cr, cluster)
               : vs_load_softmax(static_cast<const float*>(logits) + (long long)(o + node) * row_stride, v_begin,
                                 v_end, inv_t, pw, cr, cluster);
  };

  int a = 0, depth = 0;
  float zp = load_target(0);
  int err = 0;
  for (;;) {
    __syncthreads();
    if (tid == 0) {  // children of a, in increasing index
      int nk = 0;
      for (int c = a + 1; c < n; ++c)
        if (s_parent[c] == a) s_kids[nk++] = c;
      s_nk = nk;
    }
    __syncthreads();
    const int nk = s_nk;
    if (nk == 0 || depth == max_depth) break;
    const int row = child_row[o + a];
    if (row < 0 || row >= n_rows) { err = SB_ERR_BOUNDS; break; }
    float zq = vs_load_softmax(scores + (long long)row * score_stride, v_begin, v_end, inv_t, qw, cr, cluster);
    int accepted = -1;
    for (int k = 0; k < nk; ++k) {
      const int c = s_kids[k];
      const int x = s_tok[c];
      const bool in_vocab = x >= 0 && x < vocab;
      cluster.sync();  // pw / qw as the previous round left them, whichever CTA wrote them
      if (tid == 0) {
        // these two words may have been written by another CTA of the cluster: read them from L2
        const float pxu = in_vocab ? __ldcg(pw + x) : 0.f, qxu = in_vocab ? __ldcg(qw + x) : 0.f;
        const float px = pxu / zp;
        const float qx = zq > 0.f ? qxu / zq : 0.f;
        s_take = qx > 0.f ? (u_accept[o + c] < px / qx) : (px > 0.f);
        s_qx = qxu;
      }
      __syncthreads();
      if (s_take) { accepted = c; break; }
      // rejected: the target becomes max(p - q, 0) (kept as it is if nothing remains), and the
      // rejected token leaves the draft distribution (cleared by the thread that owns it)
      const float ip = 1.f / zp, iq = zq > 0.f ? 1.f / zq : 0.f;
      float z = 0.f;
      for (int v = v_begin + lane; v < v_end; v += 32) z += fmaxf(pw[v] * ip - qw[v] * iq, 0.f);
      z = vs_cluster_reduce<false>(z, cr, cluster);
      for (int v = v_begin + lane; v < v_end; v += 32) {
        if (z > 0.f) pw[v] = fmaxf(pw[v] * ip - qw[v] * iq, 0.f);
        if (v == x) qw[v] = 0.f;
      }
      if (z > 0.f) zp = z;
      zq = fmaxf(zq - s_qx, 0.f);
    }
    if (accepted < 0) break;
    a = accepted;
    ++depth;
    if (writer) { path[depth] = a; otok[depth - 1] = s_tok[a]; }
    cluster.sync();  // nobody still reads the old pw
    zp = load_target(a);
  }
  if (err) {  // uniform over the cluster
    __syncthreads();
    if (crank == 0)
      for (int t = tid; t <= max_depth; t += VS_THREADS) { path[t] = -1; otok[t] = -1; }
    if (writer) status[b] = err;
    return;
  }
  cluster.sync();
  // bonus: the smallest v whose inclusive prefix sum of pw exceeds u * total
  float part = 0.f;
  for (int v = v_begin + lane; v < v_end; v += 32) part += pw[v];
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) part += __shfl_xor_sync(0xffffffffu, part, sft);
  if (lane < VS_CLUSTER) *cluster.map_shared_rank(&s_seg[seg_id], lane) = part;  // lane k -> CTA k's copy
  cluster.sync();
  if (tid == 0) {
    float total = 0.f;
    for (int g = 0; g < VS_SEGS; ++g) total += s_seg[g];
    const float target = u_bonus[b] * total;
    float cum = 0.f;
    int found = -1;
    for (int g = 0; g < VS_SEGS && found < 0; ++g) {
      if (cum + s_seg[g] > target) found = g;
      else cum += s_seg[g];
    }
    if (found < 0)  // rounding left no prefix above the target: the last segment with any mass
      for (int g = VS_SEGS - 1; g >= 0 && found < 0; --g)
        if (s_seg[g] > 0.f) found = g;
    s_seg_of = found;
    s_need = target - cum;  // mass still to cross inside the segment
  }
  __syncthreads();
  if (s_seg_of == seg_id) {  // exactly one warp of the cluster
    const float need = s_need;
    float run = 0.f;
    int pick = -1, last_pos = -1;
    for (int v0 = v_begin; v0 < v_end && pick < 0; v0 += 32) {
      const int v = v0 + lane;
      const float x = v < v_end ? pw[v] : 0.f;
      float inc = x;
#pragma unroll
      for (int sft = 1; sft < 32; sft <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, inc, sft);
        if (lane >= sft) inc += up;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, v < v_end && run + inc > need);
      const unsigned pos = __ballot_sync(0xffffffffu, x > 0.f);
      if (hit) pick = v0 + __ffs(hit) - 1;
      if (pos) last_pos = v0 + 31 - __clz(pos);
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (pick < 0) pick = last_pos;  // the segment's total said yes, its ordered prefix sums did not
    if (lane == 0) { bonus[b] = pick; otok[depth] = pick; }
  }
  if (writer) {
    accept_len[b] = depth;
    path[0] = 0;
    status[b] = SB_OK;
  }
}

}  // namespace sb

extern "C" size_t sb_verify_sample_workspace_bytes(int32_t batch, int32_t vocab) {
  if (batch < 1 || vocab < 1) return 0;
  return (size_t)batch * 2 * (size_t)vocab * sizeof(float);
}

extern "C" sb_status sb_verify_sample(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                                      const float* scores, int64_t score_stride, int32_t n_rows, int32_t batch,
                                      int32_t total_nodes, const int32_t* node_offsets, const int32_t* parent,
                                      const int32_t* tok, const int32_t* child_row, float temperature,
                                      const float* u_accept, const float* u_bonus, int32_t max_depth,
                                      int32_t* accept_len, int32_t* path_nodes, int32_t* out_tokens, int32_t* bonus,
                                      void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  using namespace sb;
  if (!logits || !scores || !node_offsets || !parent || !tok || !child_row || !u_accept || !u_bonus || !accept_len ||
      !path_nodes || !out_tokens || !bonus || !status || batch < 1 || total_nodes < 1 || vocab < 1 || n_rows < 1 ||
      row_stride < vocab || score_stride < vocab || !(temperature > 0.f))
    return SB_ERR_INVALID_ARG;
  if (dtype != SB_BF16 && dtype != SB_F32) return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH || batch > 65535) return SB_ERR_UNSUPPORTED;
  const size_t need = sb_verify_sample_workspace_bytes(batch, vocab);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 15)) return SB_ERR_WORKSPACE;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(VS_CLUSTER, batch);
  cfg.blockDim = dim3(VS_THREADS);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = VS_CLUSTER;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, verify_sample_kernel, logits, (int)dtype, (long long)row_stride, (int)vocab, scores,
                         (long long)score_stride, (int)n_rows, (int)total_nodes, node_offsets, parent, tok, child_row,
                         1.0f / temperature, u_accept, u_bonus, (int)max_depth, accept_len, path_nodes, out_tokens,
                         bonus, static_cast<float*>(workspace), status) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}
