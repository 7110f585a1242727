// sb_verifier_signal: the verifier-derived update signal s = sum over rejected positions of (1 - r)
// (Sec. 3.4, the verifier-derived signal; Alg. 2 line 2), one verify iteration at a time.
//
//   verifier_signal_kernel : a cluster of SIG_CLUSTER CTAs per sequence.  Every CTA reads the
//                       sequence's accept result, finds the drafter row that predicted the token
//                       after the last accepted node, and scans its share of that row once with a
//                       running (maximum, sum of exponentials) per thread.  The CTA pairs meet in
//                       the shared memory of the cluster's first CTA (distributed shared memory),
//                       which combines them in rank order and writes r and the updated sum.
#include <cooperative_groups.h>

#include "common.cuh"

namespace sb {
namespace cg = cooperative_groups;

constexpr int SIG_THREADS = 512;
constexpr int SIG_CLUSTER = 8;
constexpr int SIG_VEC = 8;  // 16-byte loads in flight per thread
constexpr float kLog2e = 1.4426950408889634f;

// (m, z) = (maximum, sum of 2^((x - m) * log2 e)) of a set; the empty set is (-inf, 0).
struct MaxSum {
  float m, z;
};
__device__ inline MaxSum combine(MaxSum a, MaxSum b) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return {m, 0.f};
  return {m, a.z * exp2f((a.m - m) * kLog2e) + b.z * exp2f((b.m - m) * kLog2e)};
}
// a batch of values whose maximum is bm joins the running pair
__device__ inline void join_batch(MaxSum& run, float bm, const float* x, int n) {
  if (bm == -INFINITY) return;
  const float m = fmaxf(run.m, bm);
  float z = run.z * exp2f((run.m - m) * kLog2e);  // run.m = -inf: 0 * 0
  for (int i = 0; i < n; ++i) z += exp2f((x[i] - m) * kLog2e);
  run.m = m;
  run.z = z;
}

__global__ void __launch_bounds__(SIG_THREADS) verifier_signal_kernel(
    const float* __restrict__ scores, long long row_stride, int n_rows, int vocab, int total_nodes,
    const int* __restrict__ node_offsets, const int* __restrict__ child_row, const int* __restrict__ path_nodes,
    const int* __restrict__ accept_len, const int* __restrict__ bonus, int max_depth, float* __restrict__ r_prob,
    float* __restrict__ signal, int* __restrict__ status) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ MaxSum s_warp[SIG_THREADS / 32];
  __shared__ MaxSum s_part[SIG_CLUSTER];  // used in the cluster's first CTA
  const int b = blockIdx.y, crank = (int)cluster.block_rank(), tid = threadIdx.x;

  // the same few loads in every thread of the cluster: the decisions below are uniform
  const int o = node_offsets[b], n = node_offsets[b + 1] - o;
  const int a = accept_len[b];
  int err = 0, row = -1;
  if (a < 0 || a > max_depth || o < 0 || n < 1 || (long long)o + n > total_nodes) {
    err = SB_ERR_BOUNDS;
  } else {
    const int best = path_nodes[(long long)b * (max_depth + 1) + a];
    if (best < 0 || best >= n) err = SB_ERR_BOUNDS;
    else {
      row = child_row[o + best];
      if (row >= n_rows) err = SB_ERR_BOUNDS;
    }
  }
  if (err || row < 0) {  // nothing to scan: an error, or nothing was drafted after the last accepted node
    if (crank == 0 && tid == 0) {
      r_prob[b] = -1.f;
      status[b] = err;
    }
    return;
  }
  const int tok = bonus[b];
  const float* x = scores + (long long)row * row_stride;

  // this CTA's share of the row: whole 4-element groups
  const int groups = ceil_div(vocab, 4);
  const int per = ceil_div(groups, SIG_CLUSTER);
  const int begin = min(vocab, crank * per * 4), end = min(vocab, (crank + 1) * per * 4);
  MaxSum run = {-INFINITY, 0.f};
  const bool vec_ok = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
  if (vec_ok) {
    const int n_vec = (end - begin) / 4;
    const float4* vb = reinterpret_cast<const float4*>(x + begin);
    for (int t0 = tid; t0 < n_vec; t0 += SIG_VEC * SIG_THREADS) {
      float v[4 * SIG_VEC];
      float bm = -INFINITY;
#pragma unroll
      for (int q = 0; q < SIG_VEC; ++q) {
        float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (t0 + q * SIG_THREADS < n_vec) t = __ldg(vb + t0 + q * SIG_THREADS);
        v[4 * q] = score_of(t.x); v[4 * q + 1] = score_of(t.y); v[4 * q + 2] = score_of(t.z); v[4 * q + 3] = score_of(t.w);
      }
#pragma unroll
      for (int i = 0; i < 4 * SIG_VEC; ++i) bm = fmaxf(bm, v[i]);
      join_batch(run, bm, v, 4 * SIG_VEC);  // padding is -inf: it adds exactly 0
    }
    for (int i = begin + n_vec * 4 + tid; i < end; i += SIG_THREADS) {
      const float xv = score_of(x[i]);
      join_batch(run, xv, &xv, 1);
    }
  } else {
    for (int i = begin + tid; i < end; i += SIG_THREADS) {
      const float xv = score_of(x[i]);
      join_batch(run, xv, &xv, 1);
    }
  }
  // CTA pair, in a fixed order
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    MaxSum oth = {__shfl_xor_sync(0xffffffffu, run.m, sft), __shfl_xor_sync(0xffffffffu, run.z, sft)};
    run = combine(run, oth);
  }
  if ((tid & 31) == 0) s_warp[tid >> 5] = run;
  __syncthreads();
  if (tid == 0) {
    MaxSum c = s_warp[0];
    for (int w = 1; w < SIG_THREADS / 32; ++w) c = combine(c, s_warp[w]);
    *cluster.map_shared_rank(&s_part[crank], 0) = c;  // a store into the first CTA's shared memory
  }
  cluster.sync();
  if (crank == 0 && tid == 0) {
    MaxSum c = s_part[0];
    for (int k = 1; k < SIG_CLUSTER; ++k) c = combine(c, s_part[k]);
    float r;
    if (tok < 0 || tok >= vocab) r = 0.f;                  // not a token of the drafter's vocabulary
    else if (c.m == -INFINITY) r = 1.f / (float)vocab;     // no finite score: read as a flat distribution
    else r = exp2f((score_of(x[tok]) - c.m) * kLog2e) / c.z;
    r_prob[b] = r;
    signal[b] += 1.f - r;
    status[b] = SB_OK;
  }
}

}  // namespace sb

extern "C" sb_status sb_verifier_signal(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                        int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                                        const int32_t* child_row, const int32_t* path_nodes,
                                        const int32_t* accept_len, const int32_t* bonus, int32_t max_depth,
                                        float* r_prob, float* signal, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_verifier_signal");
  using namespace sb;
  if (!scores || !node_offsets || !child_row || !path_nodes || !accept_len || !bonus || !r_prob || !signal ||
      !status || n_rows < 1 || vocab < 1 || batch < 1 || total_nodes < 1 || row_stride < vocab)
    return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH || batch > 65535) return SB_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(scores) & 3) return SB_ERR_INVALID_ARG;
  // rows start on 16-byte boundaries only if the stride keeps them there; otherwise the kernel's
  // per-row alignment test sends that row down the scalar path
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(SIG_CLUSTER, batch);
  cfg.blockDim = dim3(SIG_THREADS);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = SIG_CLUSTER;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, verifier_signal_kernel, scores, (long long)row_stride, (int)n_rows, (int)vocab,
                         (int)total_nodes, node_offsets, child_row, path_nodes, accept_len, bonus, (int)max_depth,
                         r_prob, signal, status) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}
