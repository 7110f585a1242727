// Pieces shared by the tree-attention kernels: call parameters, per-sequence planning, the
// visibility window of the tree mask, and the in-cluster merge of KV chunks.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace sb {

namespace cg = cooperative_groups;
typedef __nv_bfloat16 bf16;

struct AttnParams {
  sb_tree_batch tb;
  const int* q_node_begin;
  const int* q_offsets;
  int total_q;
  const bf16* q;
  bf16* out;
  float* lse;
  float scale_log2;  // softmax scale * log2(e): scores are kept in the base-2 domain
  int num_splits;   // KV chunks per (sequence, KV head, row tile) = cluster size * outer
  int outer;        // clusters per (sequence, KV head, row tile); > 1 needs the merge kernel
  float* part_o;    // [outer][total_q*Hq][D] normalised partial outputs
  float* part_lse;  // [outer][total_q*Hq]    base-2 log-sum-exp of each partial
  int* status;
  int G;            // query heads per KV head
};

constexpr float kLn2 = 0.6931471805599453f;

// What a CTA may do for its sequence after the shape checks.
struct SeqPlan {
  SeqInfo info;
  bool can_write;  // the sequence's output rows are inside q/out
  bool compute;    // tree and lengths are valid: run the attention
};

// Must be called by every thread of the CTA (contains barriers).  `designated` CTAs (one per
// sequence) also scan the page table and publish the sequence's status word.
__device__ inline SeqPlan plan_sequence(const AttnParams& p, int b, bool designated, int* s_parent,
                                        uint32_t* s_anc) {
  SeqPlan sp;
  sp.info = load_seq_info(p.tb, p.q_node_begin, p.q_offsets, p.total_q, b);
  int err = sp.info.err;
  // Which rows may be zero-filled on error: recompute the raw row range.
  const int o = p.tb.node_offsets[b];
  const int n_raw = p.tb.node_offsets[b + 1] - o;
  const int q0 = p.q_node_begin ? p.q_node_begin[b] : 0;
  const int q_off = p.q_offsets ? p.q_offsets[b] : o;
  const bool rows_ok = n_raw >= 0 && n_raw <= SB_MAX_NODES && n_raw <= p.tb.max_nodes && q0 >= 0 &&
                       q0 <= n_raw && q_off >= 0 && (long long)q_off + (n_raw - q0) <= p.total_q &&
                       o >= 0 && (long long)o + n_raw <= p.tb.total_nodes;
  sp.can_write = rows_ok;
  if (rows_ok && err) {  // lengths are bad but the rows exist: keep them for zero-filling
    sp.info.nq = n_raw - q0;
    sp.info.q0 = q0;
    sp.info.q_off = q_off;
  }
  const bool tree_ok = build_ancestors_smem(p.tb.parent + (rows_ok ? o : 0), err ? 0 : sp.info.n,
                                            s_parent, s_anc, nullptr);
  if (!err && !tree_ok) err = SB_ERR_INVALID_TREE;
  if (designated) {
    const bool pages_ok = err ? true : pages_in_pool(p.tb, b, sp.info.P + sp.info.n);
    if (!err && !pages_ok) err = SB_ERR_BOUNDS;  // reported; reads were clamped into the pool
    if (threadIdx.x == 0) p.status[b] = err;
    if (!pages_ok) err = 0;  // other CTAs cannot see this; stay consistent with them
  }
  sp.compute = err == 0;
  return sp;
}

__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// 64 visibility bits of one row for the keys [rel0, rel0 + 64) counted from the first tree slot:
// keys before the tree (rel < 0) are prefix and visible, 0 <= rel < 128 follow the ancestor mask,
// later keys do not exist.  rel0 is uniform over the CTA, so the branches do not diverge.
__device__ inline uint64_t visibility_window(const uint32_t (&a)[4], int rel0) {
  const uint64_t lo = (uint64_t)a[0] | ((uint64_t)a[1] << 32);
  const uint64_t hi = (uint64_t)a[2] | ((uint64_t)a[3] << 32);
  if (rel0 <= -64) return ~0ull;
  if (rel0 < 0) return (lo << (-rel0)) | ((1ull << (-rel0)) - 1ull);
  if (rel0 == 0) return lo;
  if (rel0 < 64) return (lo >> rel0) | (hi << (64 - rel0));
  if (rel0 == 64) return hi;
  if (rel0 < 128) return hi >> (rel0 - 64);
  return 0ull;
}


// Merge of the cluster's KV chunks and final store (called by every thread of every CTA of the
// cluster after a cluster-wide barrier).  Each CTA has parked, in its own shared memory, its
// unnormalised O tile `s_red` [BM_][D+PAD], row maxima `s_m` and row sums `s_l` (base-2 domain).
// CTA `crank` reduces rows [crank*rows_per, (crank+1)*rows_per) over all S CTAs through
// distributed shared memory and writes them: final bf16 rows + natural-log LSE when the grid has
// one cluster per row tile, else one fp32 partial per cluster for the merge kernel.
template <int D, int BM_, int PAD = 8>
__device__ inline void cluster_merge_and_store(const AttnParams& p, cg::cluster_group& cluster, int S, int crank,
                                               float* s_red, float* s_m, float* s_l, float* s_w, float* s_lse,
                                               int outer_idx, int row0, int rows_total, int g, int q_off,
                                               long long rows_all, int tid, int nthreads) {
  constexpr int RS = D + PAD;
  const int Hq = p.tb.n_q_heads, G = p.G;
  constexpr int BM = BM_;
  const int NTHREADS = nthreads;
  const int rows_per = ceil_div(BM, S);
  const int r_begin = crank * rows_per;
  const int r_end = min(BM, r_begin + rows_per);
  for (int t = tid; t < r_end - r_begin; t += NTHREADS) {
    const int r = r_begin + t;
    float M = -INFINITY;
    for (int c = 0; c < S; ++c) M = fmaxf(M, cluster.map_shared_rank(s_m, c)[r]);
    float Lsum = 0.f;
    for (int c = 0; c < S; ++c) {
      const float mc = cluster.map_shared_rank(s_m, c)[r];
      const float wc = mc == -INFINITY ? 0.f : fast_exp2(mc - M);
      s_w[t * S + c] = wc;
      Lsum += wc * cluster.map_shared_rank(s_l, c)[r];
    }
    const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
    for (int c = 0; c < S; ++c) s_w[t * S + c] *= inv;
    s_lse[t] = Lsum > 0.f ? M + log2f(Lsum) : -INFINITY;
  }
  __syncthreads();
  for (int idx = tid; idx < (r_end - r_begin) * (D / 4); idx += NTHREADS) {
    const int t = idx / (D / 4), c4 = idx % (D / 4);
    const int r = r_begin + t;
    const int R = row0 + r;
    if (R >= rows_total) continue;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = 0; c < S; ++c) {
      const float w = s_w[t * S + c];
      if (w == 0.f) continue;  // that chunk saw no key for this row (its tile may be unwritten)
      const float4 v = *reinterpret_cast<const float4*>(cluster.map_shared_rank(s_red, c) + r * RS + c4 * 4);
      acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
    }
    const int node_l = R / G, hh = R - node_l * G;
    const long long grow = (long long)(q_off + node_l) * Hq + g * G + hh;
    const float lse2 = s_lse[t];
    if (p.outer == 1) {
      uint2 packed;
      packed.x = pack_bf16(acc.x, acc.y);
      packed.y = pack_bf16(acc.z, acc.w);
      *reinterpret_cast<uint2*>(p.out + grow * D + c4 * 4) = packed;
      if (p.lse && c4 == 0) p.lse[grow] = lse2 == -INFINITY ? 0.f : lse2 * kLn2;
    } else {
      *reinterpret_cast<float4*>(p.part_o + (outer_idx * rows_all + grow) * D + c4 * 4) = acc;
      if (c4 == 0) p.part_lse[outer_idx * rows_all + grow] = lse2;
    }
  }
}

}  // namespace sb
