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
  float* part_o;    // [outer][total_q*Hq][D] normalised partial outputs (fp32, or bf16 when part_bf16)
  float* part_lse;  // [outer][total_q*Hq]    base-2 log-sum-exp of each partial
  int* status;
  int G;            // query heads per KV head
  int row_tiles;    // 128-row query tiles per (sequence, KV head) in the grid
  int sort_seqs;    // 1: grid index z is the rank of a sequence by length, longest first
  int part_bf16;    // 1: part_o holds bf16 (the writer's rows are already rounded to bf16 when it stores them)
};

constexpr float kLn2 = 0.6931471805599453f;

// Longest-first launch order for ragged batches that run in several waves of CTAs: the CTAs of a
// long sequence start first, so the last wave holds the short ones (config of 16 sequences with
// 17..54 key blocks: 163 us in input order against 138 us in a schedule simulation).  Every CTA
// ranks the batch itself: sequence with rank z by (length descending, index ascending).  Any
// contents of the length arrays give a permutation.  s_len / s_perm: >= batch ints each, batch <=
// blockDim.x; the caller must not reuse them before the closing barrier.
__device__ inline int sequence_of_rank(const sb_tree_batch& tb, int z, int* s_len, int* s_perm) {
  const int B = tb.batch, tid = threadIdx.x;
  if (tid < B) s_len[tid] = tb.prefix_len[tid] + (tb.node_offsets[tid + 1] - tb.node_offsets[tid]);
  __syncthreads();
  if (tid < B) {
    const int me = s_len[tid];
    int r = 0;
    for (int j = 0; j < B; ++j) r += (s_len[j] > me || (s_len[j] == me && j < tid)) ? 1 : 0;
    s_perm[r] = tid;
  }
  __syncthreads();
  const int b = s_perm[z];
  __syncthreads();
  return b;
}

// What a CTA may do for its sequence after the shape checks.
struct SeqPlan {
  SeqInfo info;
  bool can_write;  // the sequence's output rows are inside q/out
  bool compute;    // tree and lengths are valid: run the attention
};

// First half of the planning: lengths and row ranges from the per-sequence scalars (no barrier,
// every thread computes the same values).
struct SeqPre {
  SeqInfo info;
  bool can_write;
  int node_base;  // offset of the sequence's parent[] slice (0 when it cannot be trusted)
};

__device__ inline SeqPre plan_lengths(const AttnParams& p, int b) {
  SeqPre pre;
  pre.info = load_seq_info(p.tb, p.q_node_begin, p.q_offsets, p.total_q, b);
  // Which rows may be zero-filled on error: recompute the raw row range.
  const int o = p.tb.node_offsets[b];
  const int n_raw = p.tb.node_offsets[b + 1] - o;
  const int q0 = p.q_node_begin ? p.q_node_begin[b] : 0;
  const int q_off = p.q_offsets ? p.q_offsets[b] : o;
  const bool rows_ok = n_raw >= 0 && n_raw <= SB_MAX_NODES && n_raw <= p.tb.max_nodes && q0 >= 0 &&
                       q0 <= n_raw && q_off >= 0 && (long long)q_off + (n_raw - q0) <= p.total_q &&
                       o >= 0 && (long long)o + n_raw <= p.tb.total_nodes;
  pre.can_write = rows_ok;
  pre.node_base = rows_ok ? o : 0;
  if (rows_ok && pre.info.err) {  // lengths are bad but the rows exist: keep them for zero-filling
    pre.info.nq = n_raw - q0;
    pre.info.q0 = q0;
    pre.info.q_off = q_off;
  }
  return pre;
}

// Second half: ancestor sets into shared memory, tree validity, status word.  Must be called by
// every thread of the group (contains its barriers).  `designated` CTAs (one per sequence) also scan
// the page table and publish the sequence's status word.
__device__ inline SeqPlan plan_tree(const AttnParams& p, int b, bool designated, const SeqPre& pre, int* s_parent,
                                    uint32_t* s_anc, const ThreadGroup grp = whole_cta()) {
  SeqPlan sp;
  sp.info = pre.info;
  sp.can_write = pre.can_write;
  int err = sp.info.err;
  const bool tree_ok =
      build_ancestors_smem(p.tb.parent + pre.node_base, err ? 0 : sp.info.n, s_parent, s_anc, nullptr, grp);
  if (!err && !tree_ok) err = SB_ERR_INVALID_TREE;
  if (designated) {
    const bool pages_ok = err ? true : pages_in_pool(p.tb, b, sp.info.P + sp.info.n, grp);
    if (!err && !pages_ok) err = SB_ERR_BOUNDS;  // reported; reads were clamped into the pool
    if (grp.tid == 0) p.status[b] = err;
    if (!pages_ok) err = 0;  // other CTAs cannot see this; stay consistent with them
  }
  sp.compute = err == 0;
  return sp;
}

__device__ inline SeqPlan plan_sequence(const AttnParams& p, int b, bool designated, int* s_parent,
                                        uint32_t* s_anc) {
  const SeqPre pre = plan_lengths(p, b);
  return plan_tree(p, b, designated, pre, s_parent, s_anc);
}

__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// Blackwell 3-input max and packed two-lane fp32 arithmetic (one instruction for two values).
__device__ inline float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ inline unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ inline void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ inline unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ inline unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
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


// ---- in-cluster merge of KV chunks (push model) ---------------------------------------------------
// The S chunk-CTAs of a cluster each hold an unnormalised O tile [BM][D] with row maxima m and row
// sums l (base-2 domain).  Row r of the tile is owned by CTA r / rows_per (rows_per = ceil(BM/S)).
// Every CTA stores each of its rows straight into the OWNER's shared memory (distributed shared
// memory stores need no round trip), slot [source rank][row - owner's first row]; after one
// cluster barrier each owner reduces its rows from local shared memory and writes them out.
// Buffer layout in every CTA, starting at `buf`:
//   red [S*rows_per][D+8] | m [S*rows_per] | l [S*rows_per] | w [rows_per*S] | lse [rows_per]
template <int D>
struct MergeBuf {
  static constexpr int RS = D + 8;
  float* red;
  float* m;
  float* l;
  float* w;
  float* lse;
  int rows_per;
  __device__ MergeBuf(float* buf, int BM, int S) {
    rows_per = ceil_div(BM, S);
    const int slots = S * rows_per;
    red = buf;
    m = red + slots * RS;
    l = m + slots;
    w = l + slots;
    lse = w + slots;
  }
  // floats needed for a tile of BM rows and any cluster size up to 8
  static constexpr int floats(int BM) { return (BM + 8) * RS + 4 * (BM + 8); }
};

// Destination (in the owner's shared memory) of row r of the CTA with cluster rank `crank`.
template <int D>
__device__ inline float* merge_row_dst(cg::cluster_group& cluster, const MergeBuf<D>& mb, int crank, int r, int* slot) {
  const int owner = r / mb.rows_per;
  *slot = crank * mb.rows_per + (r - owner * mb.rows_per);
  return cluster.map_shared_rank(mb.red, owner) + *slot * MergeBuf<D>::RS;
}
template <int D>
__device__ inline void merge_push_ml(cg::cluster_group& cluster, const MergeBuf<D>& mb, int crank, int r, float m, float l) {
  const int owner = r / mb.rows_per;
  const int slot = crank * mb.rows_per + (r - owner * mb.rows_per);
  cluster.map_shared_rank(mb.m, owner)[slot] = m;
  cluster.map_shared_rank(mb.l, owner)[slot] = l;
}

// After the cluster barrier: reduce this CTA's rows over the S sources and store them -- final bf16
// rows + natural-log LSE when the grid has one cluster per row tile, else one fp32 partial per
// cluster for the merge kernel.
template <int D, int BM>
__device__ inline void merge_reduce_and_store(const AttnParams& p, const MergeBuf<D>& mb, int S, int crank, int outer_idx,
                                              int row0, int rows_total, int g, int q_off, long long rows_all, int tid,
                                              int nthreads) {
  constexpr int RS = MergeBuf<D>::RS;
  constexpr int MAXS = 8;
  const int Hq = p.tb.n_q_heads, G = p.G;
  const int rows_per = mb.rows_per;
  const int r_begin = crank * rows_per;
  const int n_rows = max(0, min(BM, r_begin + rows_per) - r_begin);
  for (int t = tid; t < n_rows; t += nthreads) {
    float mc[MAXS], lc[MAXS];
#pragma unroll
    for (int c = 0; c < MAXS; ++c) {
      mc[c] = c < S ? mb.m[c * rows_per + t] : -INFINITY;
      lc[c] = c < S ? mb.l[c * rows_per + t] : 0.f;
    }
    float M = -INFINITY;
#pragma unroll
    for (int c = 0; c < MAXS; ++c) M = fmaxf(M, mc[c]);
    float Lsum = 0.f;
    float wc[MAXS];
#pragma unroll
    for (int c = 0; c < MAXS; ++c) {
      wc[c] = mc[c] == -INFINITY ? 0.f : fast_exp2(mc[c] - M);
      Lsum += wc[c] * lc[c];
    }
    const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
#pragma unroll
    for (int c = 0; c < MAXS; ++c)
      if (c < S) mb.w[t * S + c] = wc[c] * inv;
    mb.lse[t] = Lsum > 0.f ? M + log2f(Lsum) : -INFINITY;
  }
  __syncthreads();
  for (int idx = tid; idx < n_rows * (D / 4); idx += nthreads) {
    const int t = idx / (D / 4), c4 = idx % (D / 4);
    const int R = row0 + r_begin + t;
    if (R >= rows_total) continue;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int c = 0; c < MAXS; ++c) {
      const float w = c < S ? mb.w[t * S + c] : 0.f;
      // a chunk that saw no key for this row has weight 0 and left its slot unwritten
      if (w != 0.f) {
        const float4 v = *reinterpret_cast<const float4*>(mb.red + (c * rows_per + t) * RS + c4 * 4);
        acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
      }
    }
    const int node_l = R / G, hh = R - node_l * G;
    const long long grow = (long long)(q_off + node_l) * Hq + g * G + hh;
    const float lse2 = mb.lse[t];
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
