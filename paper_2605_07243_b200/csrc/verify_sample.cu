// sb_verify_sample: stochastic verification of a draft tree at temperature T > 0 by multi-candidate
// rejection sampling (Sec. 4.1 evaluates temperatures 0 and 1; Sec. 4.2 mentions rejection sampling
// against the target).  The paper names the procedure only; the order of the steps is
// the one stated in include/specblock.h.
//
//   vs_stats_kernel      : the softmax statistics of EVERY target row and every draft row, in parallel
//                       over the whole GPU: a CTA per (row, vocabulary chunk) writes the chunk's maximum
//                       m and s = sum 2^((x - m) k), k = log2(e) / T.  With them p(x) and q(x) of any
//                       token are two loads and two exponentials.
//   verify_sample_kernel : a cluster of 8 CTAs per sequence walks its tree from the root; every thread
//                       takes the same decisions from the same data.  While the target distribution of
//                       the current node is the plain softmax of its row, testing a child costs a few
//                       loads and no synchronisation at all.  Only a rejection touches the vocabulary:
//                       one pass measures max(p - q, 0) (p, q formed on the fly from the rows and their
//                       statistics, the rejected siblings' tokens taken out of q), a cluster reduction
//                       gives its sum, and the residual is written to the workspace (vocab floats per
//                       sequence), which then stands for p until a child is accepted.  The bonus token is
//                       drawn by an ordered prefix search (segment totals, then a shuffle scan row by row
//                       inside the segment that holds the target mass).  All random numbers are inputs.
#include <cooperative_groups.h>

#include "common.cuh"

namespace sb {
namespace cg = cooperative_groups;

constexpr int VS_THREADS = 1024;
constexpr int VS_CLUSTER = 8;
constexpr int VS_WARPS = VS_THREADS / 32;
constexpr int VS_SEGS = VS_CLUSTER * VS_WARPS;  // vocabulary segments, one per warp of the cluster
constexpr float kVsLog2e = 1.4426950408889634f;
constexpr int VS_STATS_THREADS = 256;
constexpr int VS_MAX_CHUNKS = 32;

template <typename T>
__device__ inline float vs_value(const T* row, int v);
template <>
__device__ inline float vs_value<float>(const float* row, int v) { return score_of(row[v]); }
template <>
__device__ inline float vs_value<uint16_t>(const uint16_t* row, int v) { return score_of(bf16_bits_to_float(row[v])); }

// ---- statistics of all rows ---------------------------------------------------------------------------

__device__ inline float vs_block_reduce(float v, bool is_max, float* s_red) {
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    const float o = __shfl_xor_sync(0xffffffffu, v, sft);
    v = is_max ? fmaxf(v, o) : v + o;
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_red[0];
  for (int w = 1; w < VS_STATS_THREADS / 32; ++w) r = is_max ? fmaxf(r, s_red[w]) : r + s_red[w];
  return r;
}

// part[(row * n_chunks + c) * 2 + {0, 1}] = (m, s) of chunk c of the row: m its maximum (NaN counts as
// -inf), s = sum of 2^((x - m) k) over its elements (0 when m = -inf).  A thread takes its elements in
// sweeps of eight 16-byte loads, all in flight before the first is used, and keeps a running (m, s);
// chunks are sized so that one sweep covers them (one trip to memory per CTA).
template <typename T>
__device__ inline void vs_chunk_stats(const T* __restrict__ base, long long row_stride, int row, int vocab, int chunk,
                                      int n_chunks, bool vec_ok, float k, float* __restrict__ part, float* s_red) {
  constexpr int VEC = 16 / sizeof(T);
  constexpr int UNROLL = 8;
  const int c = blockIdx.x, tid = threadIdx.x;
  const T* r = base + (long long)row * row_stride;
  const int begin = c * chunk, end = min(vocab, begin + chunk);
  const int n_vec = vec_ok ? max(0, (end - begin) / VEC) : 0;  // chunk is a multiple of VEC
  const uint4* vb = reinterpret_cast<const uint4*>(r + begin);
  float m = -INFINITY, s = 0.f;
  auto fold = [&](float sweep_max, auto&& sum_at) {  // sum_at(ref) = sum of 2^((x - ref) k) over the sweep
    if (sweep_max == -INFINITY) return;
    if (sweep_max > m) {
      s = m > -INFINITY ? s * exp2f((m - sweep_max) * k) : 0.f;
      m = sweep_max;
    }
    s += sum_at(m);
  };
  for (int t0 = tid; t0 < n_vec; t0 += UNROLL * VS_STATS_THREADS) {
    uint4 raw[UNROLL];
#pragma unroll
    for (int q = 0; q < UNROLL; ++q)
      if (t0 + q * VS_STATS_THREADS < n_vec) raw[q] = __ldg(vb + t0 + q * VS_STATS_THREADS);
    float mx = -INFINITY;
#pragma unroll
    for (int q = 0; q < UNROLL; ++q)
      if (t0 + q * VS_STATS_THREADS < n_vec) {
        const T* e = reinterpret_cast<const T*>(&raw[q]);
#pragma unroll
        for (int u = 0; u < VEC; ++u) mx = fmaxf(mx, vs_value<T>(e, u));
      }
    fold(mx, [&](float ref) {
      float acc = 0.f;
#pragma unroll
      for (int q = 0; q < UNROLL; ++q)
        if (t0 + q * VS_STATS_THREADS < n_vec) {
          const T* e = reinterpret_cast<const T*>(&raw[q]);
#pragma unroll
          for (int u = 0; u < VEC; ++u) acc += exp2f((vs_value<T>(e, u) - ref) * k);
        }
      return acc;
    });
  }
  for (int v = begin + n_vec * VEC + tid; v < end; v += VS_STATS_THREADS) {
    const float x = vs_value<T>(r, v);
    fold(x, [&](float ref) { return exp2f((x - ref) * k); });
  }
  const float M = vs_block_reduce(m, true, s_red);
  const float S = vs_block_reduce(m > -INFINITY ? s * exp2f((m - M) * k) : 0.f, false, s_red);
  if (tid == 0) {
    part[((long long)row * n_chunks + c) * 2] = M;
    part[((long long)row * n_chunks + c) * 2 + 1] = S;
  }
}
// One grid for both matrices: rows [0, total_nodes) are the target's logits, the rest the drafter's scores.
template <typename T>
__global__ void __launch_bounds__(VS_STATS_THREADS) vs_stats_kernel(const T* __restrict__ logits, long long row_stride,
                                                                    bool p_vec, int total_nodes,
                                                                    const float* __restrict__ scores,
                                                                    long long score_stride, bool q_vec, int vocab,
                                                                    int chunk_p, int n_chunks_p, int chunk_q,
                                                                    int n_chunks_q, float k,
                                                                    float* __restrict__ stats_p,
                                                                    float* __restrict__ stats_q) {
  __shared__ float s_red[VS_STATS_THREADS / 32];
  pdl_release();  // the walk may set itself up
  const int row = blockIdx.y;
  // the grid is as wide as the matrix with more chunks per row; a row of the other one leaves its spare CTAs idle
  if (row < total_nodes) {
    if ((int)blockIdx.x < n_chunks_p)
      vs_chunk_stats<T>(logits, row_stride, row, vocab, chunk_p, n_chunks_p, p_vec, k, stats_p, s_red);
  } else if ((int)blockIdx.x < n_chunks_q) {
    vs_chunk_stats<float>(scores, score_stride, row - total_nodes, vocab, chunk_q, n_chunks_q, q_vec, k, stats_q, s_red);
  }
}

// (M, Z) of a row from its chunk statistics (at most 32 chunks): lane c fetches chunk c, the warp combines
// them with the same shuffle tree everywhere, so every thread of the cluster gets the same bits.  A row
// without a finite value is flat: M = -inf and Z = vocab (every token counts 1).  Whole warps must call.
__device__ inline void vs_row_stats(const float* part, int n_chunks, int vocab, float k, float& M, float& Z) {
  const int lane = threadIdx.x & 31;
  float m = -INFINITY, s = 0.f;
  if (lane < n_chunks) {
    const float2 ms = __ldcg(reinterpret_cast<const float2*>(part) + lane);
    m = ms.x;
    s = ms.y;
  }
  M = m;
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sft));
  if (M == -INFINITY) { Z = (float)vocab; return; }
  Z = m > -INFINITY ? s * exp2f((m - M) * k) : 0.f;
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, sft);
}
// unnormalised probability of element value x in a row with maximum M (1 everywhere in a flat row)
__device__ inline float vs_unnorm(float x, float M, float k) { return M == -INFINITY ? 1.f : exp2f((x - M) * k); }

// ---- a lane's run of 16 consecutive elements -------------------------------------------------------------
// When a warp's segment is 512 long (vocabularies up to 131072) lane l owns [v0, v0 + 16), v0 = v_begin +
// 16 l: it fetches the run with 16-byte loads that are all in flight at once and keeps it in registers, so
// a pass over the vocabulary costs one trip to memory instead of sixteen dependent ones.
constexpr int VS_RUN = 16;
template <typename T>
__device__ inline void vs_load_run(const T* row, int v0, int vocab, bool vec_ok, float (&x)[VS_RUN]);
template <>
__device__ inline void vs_load_run<float>(const float* row, int v0, int vocab, bool vec_ok, float (&x)[VS_RUN]) {
  if (vec_ok && v0 + VS_RUN <= vocab) {
    const float4* src = reinterpret_cast<const float4*>(row + v0);
    float4 r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) r[i] = src[i];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[4 * i] = score_of(r[i].x); x[4 * i + 1] = score_of(r[i].y);
      x[4 * i + 2] = score_of(r[i].z); x[4 * i + 3] = score_of(r[i].w);
    }
  } else {
#pragma unroll
    for (int i = 0; i < VS_RUN; ++i) x[i] = v0 + i < vocab ? score_of(row[v0 + i]) : -INFINITY;
  }
}
template <>
__device__ inline void vs_load_run<uint16_t>(const uint16_t* row, int v0, int vocab, bool vec_ok, float (&x)[VS_RUN]) {
  if (vec_ok && v0 + VS_RUN <= vocab) {
    const uint4* src = reinterpret_cast<const uint4*>(row + v0);
    const uint4 r0 = src[0], r1 = src[1];
    const uint32_t w[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      x[2 * i] = score_of(__uint_as_float(w[i] << 16));
      x[2 * i + 1] = score_of(__uint_as_float(w[i] & 0xffff0000u));
    }
  } else {
#pragma unroll
    for (int i = 0; i < VS_RUN; ++i) x[i] = v0 + i < vocab ? score_of(bf16_bits_to_float(row[v0 + i])) : -INFINITY;
  }
}
__device__ inline void vs_store_run(float* dst, int v0, int vocab, bool vec_ok, const float (&y)[VS_RUN]) {
  if (vec_ok && v0 + VS_RUN <= vocab) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      reinterpret_cast<float4*>(dst + v0)[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < VS_RUN; ++i)
      if (v0 + i < vocab) dst[v0 + i] = y[i];
  }
}
// a run of raw row values -> unnormalised probabilities (0 past the vocabulary)
__device__ inline void vs_run_unnorm(float (&x)[VS_RUN], int v0, int vocab, float M, float k) {
#pragma unroll
  for (int i = 0; i < VS_RUN; ++i) x[i] = v0 + i < vocab ? vs_unnorm(x[i], M, k) : 0.f;
}

// ---- cluster-wide sum -----------------------------------------------------------------------------------
// Each CTA reduces its threads, its first warp adds the warps' partials and stores the CTA's sum into
// slot [rank] of EVERY CTA's exchange array (distributed shared memory); after a cluster barrier every
// thread adds the eight partials in rank order: all threads of the cluster get the same value.  The
// exchange array is double-buffered (`flip`): a buffer is rewritten two reductions later, when every
// CTA has passed the barrier that followed its last read.
struct ClusterRed {
  float* s_warp;  // [VS_WARPS]
  float* s_cl;    // [2][VS_CLUSTER]
  int flip;
};
__device__ inline float vs_cluster_sum(float v, ClusterRed& cr, cg::cluster_group& cluster) {
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
  __syncthreads();  // s_warp may still be read from the previous reduction
  if ((threadIdx.x & 31) == 0) cr.s_warp[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {  // lane w holds warp w's partial; lane c delivers the CTA's sum to CTA c
    float r = cr.s_warp[threadIdx.x];
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) r += __shfl_xor_sync(0xffffffffu, r, sft);
    if (threadIdx.x < VS_CLUSTER)
      *cluster.map_shared_rank(cr.s_cl + cr.flip * VS_CLUSTER + cluster.block_rank(), threadIdx.x) = r;
  }
  cluster.sync();
  const float* part = cr.s_cl + cr.flip * VS_CLUSTER;
  float r = part[0];
  for (int c = 1; c < VS_CLUSTER; ++c) r += part[c];
  cr.flip ^= 1;
  return r;
}

// ---- the walk -------------------------------------------------------------------------------------------

template <typename T>
__global__ void __launch_bounds__(VS_THREADS) verify_sample_kernel(
    const T* __restrict__ logits, long long row_stride, int vocab, const float* __restrict__ scores,
    long long score_stride, int n_rows, int total_nodes, const int* __restrict__ node_offsets,
    const int* __restrict__ parent, const int* __restrict__ tok, const int* __restrict__ child_row, float inv_t,
    const float* __restrict__ u_accept, const float* __restrict__ u_bonus, int max_depth, int n_chunks_p,
    int n_chunks_q, const float* __restrict__ stats_p, const float* __restrict__ stats_q, int* __restrict__ accept_len,
    int* __restrict__ path_nodes, int* __restrict__ out_tokens, int* __restrict__ bonus, float* work,
    int* __restrict__ status) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ int s_parent[SB_MAX_NODES], s_tok[SB_MAX_NODES], s_row[SB_MAX_NODES], s_removed[SB_MAX_NODES];
  __shared__ float s_warp[VS_WARPS];
  __shared__ float s_cl[2 * VS_CLUSTER];
  __shared__ float s_seg[VS_SEGS];  // segment totals of the whole cluster (every CTA holds a copy)
  __shared__ int s_bad, s_seg_of;
  __shared__ float s_need;
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int crank = (int)cluster.block_rank();
  const bool writer = crank == 0 && tid == 0;  // the one thread that writes the per-sequence outputs
  ClusterRed cr = {s_warp, s_cl, 0};
  const float k = inv_t * kVsLog2e;
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
    pdl_wait();
    if (writer) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  if (tid < n) {
    const int p = parent[o + tid];
    s_parent[tid] = p;
    s_tok[tid] = tok[o + tid];
    s_row[tid] = child_row[o + tid];
    if (tid == 0 ? p != -1 : (p < 0 || p >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    pdl_wait();
    if (writer) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  float* pw = work + (long long)b * vocab;  // the residual target distribution after a rejection, unnormalised
  pdl_wait();  // the statistics of the rows are complete from here on (the tree above is an input of the call)
  // this warp's contiguous segment of the vocabulary
  const int seg_len = ceil_div(ceil_div(vocab, VS_SEGS), 32) * 32;
  const int seg_id = crank * VS_WARPS + warp;
  const int v_begin = min(vocab, seg_id * seg_len), v_end = min(vocab, (seg_id + 1) * seg_len);

  // register-resident runs when a warp's segment is exactly 512 long; 16-byte accesses where alignment allows
  const bool runs = seg_len == 32 * VS_RUN;
  const int v0 = v_begin + VS_RUN * lane;
  const bool p_vec = (reinterpret_cast<uintptr_t>(logits) & 15) == 0 && (row_stride * (long long)sizeof(T)) % 16 == 0;
  const bool q_vec = (reinterpret_cast<uintptr_t>(scores) & 15) == 0 && score_stride % 4 == 0;
  const bool w_vec = vocab % 4 == 0;  // pw of sequence b starts b * vocab floats into the 256-byte aligned workspace

  // State of the walk, identical in every thread of the cluster.
  int a = 0, depth = 0, err = 0;
  const T* prow = logits + (long long)o * row_stride;  // target row of the current node
  bool p_plain = true;      // p = softmax of prow (else: pw / zp)
  float Mp, zp;             // maximum of prow; normaliser of p in either form
  vs_row_stats(stats_p + (long long)o * n_chunks_p * 2, n_chunks_p, vocab, k, Mp, zp);
  auto p_unnorm = [&](int v) { return p_plain ? vs_unnorm(vs_value<T>(prow, v), Mp, k) : pw[v]; };
  auto p_run = [&](float (&y)[VS_RUN]) {  // this lane's run of unnormalised p
    if (p_plain) {
      vs_load_run<T>(prow, v0, vocab, p_vec, y);
      vs_run_unnorm(y, v0, vocab, Mp, k);
    } else {
      vs_load_run<float>(pw, v0, vocab, w_vec, y);
#pragma unroll
      for (int i = 0; i < VS_RUN; ++i) y[i] = v0 + i < vocab ? y[i] : 0.f;
    }
  };

  for (;;) {
    // the first child of a (children are the nodes c > a with parent a, in increasing index)
    int c = a + 1;
    while (c < n && s_parent[c] != a) ++c;
    if (c >= n || depth == max_depth) break;
    const int row = s_row[a];
    if (row < 0 || row >= n_rows) { err = SB_ERR_BOUNDS; break; }
    const float* qrow = scores + (long long)row * score_stride;
    float Mq, zq;  // q = (unnormalised draft value, 0 for the removed tokens) / zq
    vs_row_stats(stats_q + (long long)row * n_chunks_q * 2, n_chunks_q, vocab, k, Mq, zq);
    int n_removed = 0;
    int accepted = -1;
    for (; c < n; ++c) {
      if (s_parent[c] != a) continue;
      const int x = s_tok[c];
      const bool in_vocab = x >= 0 && x < vocab;
      // after a rejection the residual may have been written by another CTA of the cluster: read it from L2
      const float pxu = !in_vocab ? 0.f : (p_plain ? vs_unnorm(vs_value<T>(prow, x), Mp, k) : __ldcg(pw + x));
      bool gone = false;
      for (int r = 0; r < n_removed; ++r) gone = gone || s_removed[r] == x;
      const float qxu = (!in_vocab || gone) ? 0.f : vs_unnorm(vs_value<float>(qrow, x), Mq, k);
      const float px = pxu / zp;
      const float qx = zq > 0.f ? qxu / zq : 0.f;
      const bool take = qx > 0.f ? (u_accept[o + c] < px / qx) : (px > 0.f);
      if (take) { accepted = c; break; }
      // rejected: the target becomes max(p - q, 0) (kept as it is if nothing remains), and the rejected
      // token leaves the draft distribution
      const float ip = 1.f / zp, iq = zq > 0.f ? 1.f / zq : 0.f;
      float z = 0.f;
      if (runs) {  // the residual of this lane's run stays in registers between measuring and writing
        float rp[VS_RUN], rq[VS_RUN];
        p_run(rp);
        vs_load_run<float>(qrow, v0, vocab, q_vec, rq);
        vs_run_unnorm(rq, v0, vocab, Mq, k);
        for (int r = 0; r < n_removed; ++r) {
          const int t = s_removed[r] - v0;
#pragma unroll
          for (int i = 0; i < VS_RUN; ++i)
            if (i == t) rq[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < VS_RUN; ++i) {
          rp[i] = fmaxf(rp[i] * ip - rq[i] * iq, 0.f);
          z += rp[i];
        }
        z = vs_cluster_sum(z, cr, cluster);
        if (z > 0.f) vs_store_run(pw, v0, vocab, w_vec, rp);
      } else {
        for (int v = v_begin + lane; v < v_end; v += 32) {
          bool out = false;
          for (int r = 0; r < n_removed; ++r) out = out || s_removed[r] == v;
          const float qv = out ? 0.f : vs_unnorm(vs_value<float>(qrow, v), Mq, k);
          z += fmaxf(p_unnorm(v) * ip - qv * iq, 0.f);
        }
        z = vs_cluster_sum(z, cr, cluster);
        if (z > 0.f) {
          for (int v = v_begin + lane; v < v_end; v += 32) {
            bool out = false;
            for (int r = 0; r < n_removed; ++r) out = out || s_removed[r] == v;
            const float qv = out ? 0.f : vs_unnorm(vs_value<float>(qrow, v), Mq, k);
            pw[v] = fmaxf(p_unnorm(v) * ip - qv * iq, 0.f);
          }
        }
      }
      if (z > 0.f) {
        p_plain = false;
        zp = z;
      }
      zq = fmaxf(zq - qxu, 0.f);
      __syncthreads();  // every thread has read the list of removed tokens
      if (tid == 0) s_removed[n_removed] = x;
      ++n_removed;
      cluster.sync();  // the residual and the list are complete before anyone tests the next child
    }
    if (accepted < 0) break;
    a = accepted;
    ++depth;
    if (writer) { path[depth] = a; otok[depth - 1] = s_tok[a]; }
    prow = logits + (long long)(o + a) * row_stride;
    p_plain = true;
    vs_row_stats(stats_p + (long long)(o + a) * n_chunks_p * 2, n_chunks_p, vocab, k, Mp, zp);
  }
  if (err) {  // uniform over the cluster
    __syncthreads();
    if (crank == 0)
      for (int t = tid; t <= max_depth; t += VS_THREADS) { path[t] = -1; otok[t] = -1; }
    if (writer) status[b] = err;
    return;
  }
  // bonus: the smallest v whose inclusive prefix sum of p exceeds u * total
  float part = 0.f;
  float run_p[VS_RUN];  // this lane's run of p (runs only), kept for the search inside the segment
  if (runs) {
    p_run(run_p);
#pragma unroll
    for (int i = 0; i < VS_RUN; ++i) part += run_p[i];
  } else {
    for (int v = v_begin + lane; v < v_end; v += 32) part += p_unnorm(v);
  }
  const float lane_total = part;
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) part += __shfl_xor_sync(0xffffffffu, part, sft);
  if (lane < VS_CLUSTER) *cluster.map_shared_rank(&s_seg[seg_id], lane) = part;  // lane c -> CTA c's copy
  cluster.sync();
  if (warp == 0) {  // which segment holds the target mass: lane l looks after segments 8 l .. 8 l + 7
    constexpr int PER = VS_SEGS / 32;
    float seg[PER], lsum = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      seg[i] = s_seg[lane * PER + i];
      lsum += seg[i];
    }
    float incl = lsum;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, incl, sft);
      if (lane >= sft) incl += up;
    }
    const float total = __shfl_sync(0xffffffffu, incl, 31);
    const float target = u_bonus[b] * total;
    float cum = incl - lsum, cum_at = 0.f;
    int found = -1, last_mass = -1;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      if (found < 0) {
        if (cum + seg[i] > target) { found = lane * PER + i; cum_at = cum; }
        else cum += seg[i];
      }
      if (seg[i] > 0.f) last_mass = lane * PER + i;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, found >= 0);
    const unsigned mass = __ballot_sync(0xffffffffu, last_mass >= 0);
    int g = -1;
    float before = total;  // rounding left no prefix above the target: the last segment with any mass
    if (hit) {
      g = __shfl_sync(0xffffffffu, found, __ffs(hit) - 1);
      before = __shfl_sync(0xffffffffu, cum_at, __ffs(hit) - 1);
    } else if (mass) {
      g = __shfl_sync(0xffffffffu, last_mass, 31 - __clz(mass));
    }
    if (lane == 0) {
      s_seg_of = g;
      s_need = target - before;  // mass still to cross inside the segment
    }
  }
  __syncthreads();
  if (s_seg_of == seg_id && runs) {  // exactly one warp of the cluster; lanes hold consecutive runs
    const float need = s_need;
    // exclusive prefix of the lane totals, then the crossing inside the first lane whose run reaches `need`
    float incl = lane_total;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, incl, sft);
      if (lane >= sft) incl += up;
    }
    float acc = incl - lane_total;
    int mine = -1, my_last = -1;
#pragma unroll
    for (int i = 0; i < VS_RUN; ++i) {
      acc += run_p[i];
      if (mine < 0 && run_p[i] > 0.f && acc > need) mine = v0 + i;  // v0 + i < vocab: elements past it are 0
      if (run_p[i] > 0.f) my_last = v0 + i;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, mine >= 0);
    const unsigned pos = __ballot_sync(0xffffffffu, my_last >= 0);
    int pick = -1;
    if (hit) pick = __shfl_sync(0xffffffffu, mine, __ffs(hit) - 1);
    else if (pos) pick = __shfl_sync(0xffffffffu, my_last, 31 - __clz(pos));  // the total said yes, the prefix sums did not
    if (lane == 0) { bonus[b] = pick; otok[depth] = pick; }
  } else if (s_seg_of == seg_id) {
    const float need = s_need;
    float run = 0.f;
    int pick = -1, last_pos = -1;
    for (int v0 = v_begin; v0 < v_end && pick < 0; v0 += 32) {
      const int v = v0 + lane;
      const float x = v < v_end ? p_unnorm(v) : 0.f;
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

// Chunks per row of the statistics kernel for rows of `elem_bytes`-wide elements: one sweep per CTA (256 threads x
// 8 loads of 16 bytes), and at least a few hundred CTAs in the grid when the matrix is small.
static int vs_chunks(int rows_total, int vocab, int elem_bytes) {
  const int sweep = VS_STATS_THREADS * 8 * (16 / elem_bytes);
  int nc = ceil_div(vocab, sweep);
  const int fill = ceil_div(2 * 148, rows_total > 0 ? rows_total : 1), max_nc = ceil_div(vocab, 2048);
  if (nc < fill) nc = fill < max_nc ? fill : max_nc;
  if (nc > VS_MAX_CHUNKS) nc = VS_MAX_CHUNKS;
  if (nc < 1) nc = 1;
  return nc;
}
static size_t vs_align(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace sb

extern "C" size_t sb_verify_sample_workspace_bytes(int32_t batch, int32_t vocab, int32_t total_nodes, int32_t n_rows) {
  if (batch < 1 || vocab < 1 || total_nodes < 1 || n_rows < 1) return 0;
  using namespace sb;
  // the statistics of the target rows are sized for 2-byte logits (the larger count covers fp32 ones too)
  return vs_align((size_t)batch * vocab * sizeof(float)) +
         vs_align((size_t)total_nodes * VS_MAX_CHUNKS * 2 * sizeof(float)) +
         vs_align((size_t)n_rows * VS_MAX_CHUNKS * 2 * sizeof(float));
}

extern "C" sb_status sb_verify_sample(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                                      const float* scores, int64_t score_stride, int32_t n_rows, int32_t batch,
                                      int32_t total_nodes, const int32_t* node_offsets, const int32_t* parent,
                                      const int32_t* tok, const int32_t* child_row, float temperature,
                                      const float* u_accept, const float* u_bonus, int32_t max_depth,
                                      int32_t* accept_len, int32_t* path_nodes, int32_t* out_tokens, int32_t* bonus,
                                      void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_verify_sample");
  using namespace sb;
  if (!logits || !scores || !node_offsets || !parent || !tok || !child_row || !u_accept || !u_bonus || !accept_len ||
      !path_nodes || !out_tokens || !bonus || !status || batch < 1 || total_nodes < 1 || vocab < 1 || n_rows < 1 ||
      row_stride < vocab || score_stride < vocab || !(temperature > 0.f))
    return SB_ERR_INVALID_ARG;
  if (dtype != SB_BF16 && dtype != SB_F32) return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH || batch > 65535 || (long long)total_nodes + n_rows > 65535)
    return SB_ERR_UNSUPPORTED;
  const size_t need = sb_verify_sample_workspace_bytes(batch, vocab, total_nodes, n_rows);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const float inv_t = 1.0f / temperature, k = inv_t * kVsLog2e;
  char* ws = static_cast<char*>(workspace);
  float* work = reinterpret_cast<float*>(ws);
  const int esz = dtype == SB_BF16 ? 2 : 4;
  const int ncp = vs_chunks(total_nodes + n_rows, vocab, esz), ncq = vs_chunks(total_nodes + n_rows, vocab, 4);
  float* stats_p = reinterpret_cast<float*>(ws + vs_align((size_t)batch * vocab * sizeof(float)));
  float* stats_q = reinterpret_cast<float*>(reinterpret_cast<char*>(stats_p) +
                                            vs_align((size_t)total_nodes * VS_MAX_CHUNKS * 2 * sizeof(float)));
  // statistics of every target row and every draft row, one grid
  const int chunk_p = ceil_div(ceil_div(vocab, ncp), 8) * 8, chunk_q = ceil_div(ceil_div(vocab, ncq), 8) * 8;
  const bool p_vec = (reinterpret_cast<uintptr_t>(logits) & 15) == 0 && (row_stride * esz) % 16 == 0;
  const bool q_vec = (reinterpret_cast<uintptr_t>(scores) & 15) == 0 && score_stride % 4 == 0;
  const dim3 sgrid(ncp > ncq ? ncp : ncq, total_nodes + n_rows);
  if (dtype == SB_BF16)
    vs_stats_kernel<uint16_t><<<sgrid, VS_STATS_THREADS, 0, cs>>>(static_cast<const uint16_t*>(logits), (long long)row_stride,
                                                                p_vec, (int)total_nodes, scores, (long long)score_stride,
                                                                q_vec, (int)vocab, chunk_p, ncp, chunk_q, ncq, k, stats_p,
                                                                stats_q);
  else
    vs_stats_kernel<float><<<sgrid, VS_STATS_THREADS, 0, cs>>>(static_cast<const float*>(logits), (long long)row_stride, p_vec,
                                                             (int)total_nodes, scores, (long long)score_stride, q_vec,
                                                             (int)vocab, chunk_p, ncp, chunk_q, ncq, k, stats_p, stats_q);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(VS_CLUSTER, batch);
  cfg.blockDim = dim3(VS_THREADS);
  cfg.stream = cs;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = VS_CLUSTER;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the walk orders itself (pdl_wait)
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e;
  if (dtype == SB_BF16)
    e = cudaLaunchKernelEx(&cfg, verify_sample_kernel<uint16_t>, static_cast<const uint16_t*>(logits), (long long)row_stride,
                           (int)vocab, scores, (long long)score_stride, (int)n_rows, (int)total_nodes, node_offsets, parent,
                           tok, child_row, inv_t, u_accept, u_bonus, (int)max_depth, ncp, ncq,
                           static_cast<const float*>(stats_p), static_cast<const float*>(stats_q), accept_len, path_nodes,
                           out_tokens, bonus, work, status);
  else
    e = cudaLaunchKernelEx(&cfg, verify_sample_kernel<float>, static_cast<const float*>(logits), (long long)row_stride,
                           (int)vocab, scores, (long long)score_stride, (int)n_rows, (int)total_nodes, node_offsets, parent,
                           tok, child_row, inv_t, u_accept, u_bonus, (int)max_depth, ncp, ncq,
                           static_cast<const float*>(stats_p), static_cast<const float*>(stats_q), accept_len, path_nodes,
                           out_tokens, bonus, work, status);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}
