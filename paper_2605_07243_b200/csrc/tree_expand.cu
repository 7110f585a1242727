// sb_tree_expand: per-row top-k over the drafter's scores and bucket-driven branching
// (Sec. 3.2; App. A.5 maps b(.); the attach step of Alg. 1).
//
//   topk_partial_kernel : streams the [rows][vocab] fp32 scores once from HBM (a second pass hits
//                         L1/L2).  A CTA owns one (row, vocab chunk).  Pass 1: every thread takes the
//                         maximum of its strided elements; the 16th largest of the 256 thread maxima is
//                         a threshold tau that at least 16 elements of the chunk reach.  Pass 2: only
//                         elements >= tau (a handful per CTA unless values tie) enter the per-thread
//                         sorted lists; ids ascend inside a thread, so the order (value descending, id
//                         ascending) is kept by strict compares.  The CTA then pops its 16 best in order.
//   topk_partial_reg_kernel: the same result with the chunk held in registers (one HBM pass, no re-read),
//                         used whenever rows are 16-byte aligned and a chunk has at most 16384 elements.
//   expand_rows_kernel  : the finishing kernel for up to 1024 rows, a CTA per row and no CTA waiting for another:
//                         the branching structure (widths, prefix sums, parents) depends on the inputs alone
//                         and is derived by every CTA before the dependency wait; after it the CTA ranks its
//                         row's candidates by counting larger 64-bit keys and writes the row's own nodes.
//   expand_finish_kernel: the same for any number of rows in ONE CTA.  A warp per row merges the chunk lists
//                         held in registers; then the append is done in parallel: a row is alive iff every
//                         earlier position of its block has width >= 1, its first node id is an exclusive
//                         prefix sum of the alive rows' widths, and the node budget clips the tail (a clipped
//                         rank-0 node can only silence rows that the full budget silences anyway).
#include "tc_common.cuh"

namespace sb {

constexpr int TOPK_THREADS = 256;
constexpr int kNoId = 0x7fffffff;


__device__ inline bool ranks_before(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// Softmax statistics of a chunk for the rank head's distribution summary (App. B): with m the
// chunk maximum, s = sum exp(x - m) and t = sum exp(x - m) * x.  `tmax`, `s`, `t` are this thread's
// share (s, t relative to the CTA maximum returned through *cta_max by the first call).
__device__ inline float cta_reduce_max(float v, float* s_red) {
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, sft));
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_red[0];
  for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, s_red[w]);
  __syncthreads();
  return r;
}
__device__ inline float cta_reduce_sum(float v, float* s_red) {
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += s_red[w];
  __syncthreads();
  return r;
}
__device__ inline void stats_term(float x, float m, float& s, float& t) {
  const float e = exp2f((x - m) * 1.4426950408889634f);  // x = -inf gives 0
  s += e;
  t += e > 0.f ? e * x : 0.f;
}

template <bool STATS>
__global__ void __launch_bounds__(TOPK_THREADS) topk_partial_kernel(const float* __restrict__ scores,
                                                                    long long row_stride, int vocab, int chunk,
                                                                    int n_chunks, bool vec_ok,
                                                                    float* __restrict__ part_val,
                                                                    int* __restrict__ part_idx,
                                                                    float* __restrict__ part_stats, const int* __restrict__ n_nodes_in,
    int* __restrict__ n0_snapshot) {
  __shared__ float s_val[SB_KMAX][TOPK_THREADS];  // [rank][thread]: conflict-free per-thread lists
  __shared__ int s_idx[SB_KMAX][TOPK_THREADS];
  __shared__ float s_wv[TOPK_THREADS / 32];
  __shared__ int s_wi[TOPK_THREADS / 32], s_wt[TOPK_THREADS / 32];
  __shared__ int s_winner;
  const int row = blockIdx.y, c = blockIdx.x, tid = threadIdx.x;
  const float* base = scores + (long long)row * row_stride;
  const int begin = c * chunk;
  const int end = min(vocab, begin + chunk);
  pdl_release();  // the finishing kernel may start its prologue
  if (n0_snapshot && row == 0 && c == 0 && tid == 0) *n0_snapshot = *n_nodes_in;  // the finishing kernel overwrites the counter

  // pass 1: thread maxima -> threshold tau = 16th largest of them
  const int n_vec = vec_ok ? max(0, (end - begin) / 4) : 0;
  const float4* vb = reinterpret_cast<const float4*>(base + begin);
  float tmax = -INFINITY;
  for (int t = tid; t < n_vec; t += TOPK_THREADS) {
    const float4 x = __ldg(vb + t);
    tmax = fmaxf(tmax, fmaxf(fmaxf(score_of(x.x), score_of(x.y)), fmaxf(score_of(x.z), score_of(x.w))));
  }
  for (int i = begin + n_vec * 4 + tid; i < end; i += TOPK_THREADS) tmax = fmaxf(tmax, score_of(base[i]));
  float* s_max = &s_val[0][0];  // the lists are written only after pass 2
  __shared__ float s_tau;
  s_max[tid] = tmax;
  if (tid == 0) s_tau = -INFINITY;
  __syncthreads();
  {
    int gt = 0, ge = 0;
    for (int t = 0; t < TOPK_THREADS; ++t) {
      const float o = s_max[t];
      gt += o > tmax;
      ge += o >= tmax;
    }
    if (gt < SB_KMAX && ge >= SB_KMAX) s_tau = tmax;  // every writer holds the same value
  }
  __syncthreads();
  const float tau = s_tau;
  __syncthreads();  // s_max (aliasing the lists) is dead from here on
  if (STATS) {  // chunk maximum, then one more pass (L1/L2 hits) for the two sums
    __shared__ float s_red[TOPK_THREADS / 32];
    const float cmax = cta_reduce_max(tmax, s_red);
    float ss = 0.f, tt = 0.f;
    if (cmax > -INFINITY) {
      for (int t = tid; t < n_vec; t += TOPK_THREADS) {
        const float4 x = __ldg(vb + t);
        stats_term(score_of(x.x), cmax, ss, tt);
        stats_term(score_of(x.y), cmax, ss, tt);
        stats_term(score_of(x.z), cmax, ss, tt);
        stats_term(score_of(x.w), cmax, ss, tt);
      }
      for (int i = begin + n_vec * 4 + tid; i < end; i += TOPK_THREADS) stats_term(score_of(base[i]), cmax, ss, tt);
    }
    ss = cta_reduce_sum(ss, s_red);
    tt = cta_reduce_sum(tt, s_red);
    if (tid == 0) {
      float* o = part_stats + ((long long)row * n_chunks + c) * 3;
      o[0] = cmax; o[1] = ss; o[2] = tt;
    }
  }

  float v[SB_KMAX];
  int id[SB_KMAX];
#pragma unroll
  for (int k = 0; k < SB_KMAX; ++k) { v[k] = -INFINITY; id[k] = kNoId; }

  auto offer = [&](float x, int xi) {
    x = score_of(x);
    if (x < tau) return;  // at least 16 elements of the chunk reach tau
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

// Register-resident variant for 16-byte-aligned rows and chunks of at most TOPK_REG_ELEMS
// elements: the chunk is read from HBM exactly once -- one thread issues bulk asynchronous copies
// (cp.async.bulk, 16 KB pieces, completion on an mbarrier) of the whole chunk into shared memory,
// which keeps far more bytes in flight per SM than per-thread loads can (7 us -> 3.5 us for the
// 16.4 MB of 32 x 128256 scores), then every thread takes its 64 values into registers.
// tau = the smallest of 16 group maxima (16 threads per group; 16 distinct elements reach it), so
// the chunk's 16 best are among the elements >= tau -- a few dozen unless values tie.  They are
// collected in one dense list (per-thread counts, a warp scan and one atomic per warp instead of
// one per element) and ranked all-pairs under (value descending, id ascending).  If more than
// TOPK_CAND of them exist (massive ties) the per-thread sorted-list method takes over, fed from the
// same registers.
constexpr int TOPK_VEC_PER_THREAD = 16;
constexpr int TOPK_REG_ELEMS = TOPK_THREADS * TOPK_VEC_PER_THREAD * 4;  // 16384
constexpr int TOPK_CAND = 512;
constexpr int TOPK_STAGE_BYTES = TOPK_REG_ELEMS * 4;     // dynamic shared memory: the staged chunk

// The body shared by topk_partial_reg_kernel and expand_cluster_kernel: the 16 best of one (row, chunk)
// in order, written to out_val / out_idx (16 entries each; global memory, or a cluster peer's shared
// memory through a generic pointer), and with STATS the chunk's (m, s, t) to stats_out.  `while_loading`
// runs after the chunk's bulk copies have been issued and before they are awaited.  Every thread of
// the CTA must call it (barriers inside); all threads return together.
template <bool STATS, typename F>
__device__ __forceinline__ void topk_reg_chunk(const float* __restrict__ base, int begin, int end,
                                               float* out_val, int* out_idx, float* stats_out, F while_loading) {
  __shared__ float s_val[SB_KMAX][TOPK_THREADS];  // fallback lists; the candidate arrays alias them
  __shared__ int s_idx[SB_KMAX][TOPK_THREADS];
  __shared__ float s_group[16];
  __shared__ float s_wv[TOPK_THREADS / 32];
  __shared__ int s_wi[TOPK_THREADS / 32], s_wt[TOPK_THREADS / 32];
  __shared__ int s_winner, s_count;
  __shared__ uint64_t s_bar;
  __shared__ int s_abort;
  extern __shared__ float4 s_stage[];  // the chunk as it lies in memory
  float* s_cv = &s_val[0][0];
  int* s_ci = &s_idx[0][0];
  const int tid = threadIdx.x, lane = tid & 31;
  const int n_elems = max(0, end - begin);
  const int n_vec = n_elems / 4;  // whole float4s; up to 3 tail elements are handled apart
  const float4* vb = reinterpret_cast<const float4*>(base + begin);
  if (tid == 0) {
    s_abort = 0;
    s_count = 0;
    mbar_init(&s_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0 && n_vec > 0) {
    mbar_expect_tx(&s_bar, (uint32_t)n_vec * 16u);
    for (int off = 0; off < n_vec; off += 1024)  // 16 KB pieces
      bulk_load_1d(smem_u32(s_stage + off), vb + off, (uint32_t)min(1024, n_vec - off) * 16u, &s_bar);
  }
  while_loading();
  const bool staged = n_vec == 0 || mbar_wait(&s_bar, 0, &s_abort);  // bounded; else read global memory directly

  float4 x[TOPK_VEC_PER_THREAD];
  float tmax = -INFINITY;
#pragma unroll
  for (int i = 0; i < TOPK_VEC_PER_THREAD; ++i) {
    const int v = tid + i * TOPK_THREADS;
    float4 t = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (v < n_vec) {
      t = staged ? s_stage[v] : __ldg(vb + v);
      t.x = score_of(t.x); t.y = score_of(t.y); t.z = score_of(t.z); t.w = score_of(t.w);
    }
    x[i] = t;
    tmax = fmaxf(tmax, fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w)));
  }
  if (STATS) {  // softmax statistics of the chunk from the values already in registers
    __shared__ float s_red[TOPK_THREADS / 32];
    float tail_max = -INFINITY;
    if (tid == 0)
      for (int id2 = begin + 4 * n_vec; id2 < end; ++id2) tail_max = fmaxf(tail_max, score_of(base[id2]));
    const float cmax = cta_reduce_max(fmaxf(tmax, tail_max), s_red);
    float ss = 0.f, tt = 0.f;
    if (cmax > -INFINITY) {
#pragma unroll
      for (int i = 0; i < TOPK_VEC_PER_THREAD; ++i) {
        if (tid + i * TOPK_THREADS < n_vec) {
          stats_term(x[i].x, cmax, ss, tt);
          stats_term(x[i].y, cmax, ss, tt);
          stats_term(x[i].z, cmax, ss, tt);
          stats_term(x[i].w, cmax, ss, tt);
        }
      }
      if (tid == 0)
        for (int id2 = begin + 4 * n_vec; id2 < end; ++id2) stats_term(score_of(base[id2]), cmax, ss, tt);
    }
    ss = cta_reduce_sum(ss, s_red);
    tt = cta_reduce_sum(tt, s_red);
    if (tid == 0) {
      stats_out[0] = cmax; stats_out[1] = ss; stats_out[2] = tt;
    }
  }
  float gmax = tmax;
#pragma unroll
  for (int sft = 8; sft > 0; sft >>= 1) gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, sft));
  if ((tid & 15) == 0) s_group[tid >> 4] = gmax;
  __syncthreads();
  float tau = s_group[0];
#pragma unroll
  for (int i = 1; i < 16; ++i) tau = fminf(tau, s_group[i]);

  // The elements >= tau go to one dense list.  Every thread counts its own (64 compares), a warp
  // scan turns the counts into offsets, one atomic per warp reserves the warp's range, and only
  // the few threads that hold any write them: no per-element atomics or votes.
  int mine = 0;
#pragma unroll
  for (int i = 0; i < TOPK_VEC_PER_THREAD; ++i) {
    if (tid + i * TOPK_THREADS < n_vec)  // padding beyond the chunk is not an element
      mine += (x[i].x >= tau) + (x[i].y >= tau) + (x[i].z >= tau) + (x[i].w >= tau);
  }
  const int n_tail = end - (begin + 4 * n_vec);  // up to 3 elements past the last float4: always candidates
  if (tid == 0) mine += n_tail;
  int incl = mine;
#pragma unroll
  for (int sft = 1; sft < 32; sft <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, sft);
    if (lane >= sft) incl += up;
  }
  int wbase = 0;
  if (lane == 31 && incl > 0) wbase = atomicAdd(&s_count, incl);
  wbase = __shfl_sync(0xffffffffu, wbase, 31);
  if (mine > 0) {
    int pos = wbase + incl - mine;
    auto put = [&](float v, int id) {
      if (pos < TOPK_CAND) { s_cv[pos] = v; s_ci[pos] = id; }
      ++pos;
    };
#pragma unroll
    for (int i = 0; i < TOPK_VEC_PER_THREAD; ++i) {
      const int vi = tid + i * TOPK_THREADS;
      if (vi < n_vec) {
        const int id0 = begin + 4 * vi;
        if (x[i].x >= tau) put(x[i].x, id0);
        if (x[i].y >= tau) put(x[i].y, id0 + 1);
        if (x[i].z >= tau) put(x[i].z, id0 + 2);
        if (x[i].w >= tau) put(x[i].w, id0 + 3);
      }
    }
    if (tid == 0)
      for (int id = begin + 4 * n_vec; id < end; ++id) put(score_of(base[id]), id);
  }
  __syncthreads();
  const int count = s_count;
  if (count <= TOPK_CAND) {
    // rank of candidate a = number of candidates that come before it; four threads share one
    // candidate (a quarter of the comparisons each, combined by shuffles)
    for (int a0 = 0; a0 < count; a0 += TOPK_THREADS / 4) {
      const int a = a0 + (tid >> 2);
      const bool live = a < count;
      const float v = live ? s_cv[a] : 0.f;
      const int id = live ? s_ci[a] : 0;
      int r = 0;
      if (live)
        for (int b2 = tid & 3; b2 < count; b2 += 4) r += ranks_before(s_cv[b2], s_ci[b2], v, id) ? 1 : 0;
      r += __shfl_xor_sync(0xffffffffu, r, 1);
      r += __shfl_xor_sync(0xffffffffu, r, 2);
      if (live && (tid & 3) == 0 && r < SB_KMAX) { out_val[r] = v; out_idx[r] = id; }
    }
    if (tid < SB_KMAX && tid >= count) { out_val[tid] = -INFINITY; out_idx[tid] = kNoId; }
    return;
  }
  // ---- massive ties: per-thread sorted lists (ids ascend inside a thread), then ordered pops ----
  __syncthreads();  // the candidate arrays alias the lists
  float v[SB_KMAX];
  int id[SB_KMAX];
#pragma unroll
  for (int k = 0; k < SB_KMAX; ++k) { v[k] = -INFINITY; id[k] = kNoId; }
  auto offer = [&](float xv, int xi) {
    if (xv < tau) return;
    if (!ranks_before(xv, xi, v[SB_KMAX - 1], id[SB_KMAX - 1])) return;
    v[SB_KMAX - 1] = xv;
    id[SB_KMAX - 1] = xi;
#pragma unroll
    for (int k = SB_KMAX - 1; k > 0; --k) {
      if (ranks_before(v[k], id[k], v[k - 1], id[k - 1])) {
        const float tv = v[k]; v[k] = v[k - 1]; v[k - 1] = tv;
        const int ti = id[k]; id[k] = id[k - 1]; id[k - 1] = ti;
      }
    }
  };
#pragma unroll
  for (int i = 0; i < TOPK_VEC_PER_THREAD; ++i) {
    const int vi = tid + i * TOPK_THREADS;
    if (vi < n_vec) {
      const int id0 = begin + 4 * vi;
      offer(x[i].x, id0); offer(x[i].y, id0 + 1); offer(x[i].z, id0 + 2); offer(x[i].w, id0 + 3);
    }
  }
  if (tid == 0)
    for (int i2 = begin + 4 * n_vec; i2 < end; ++i2) offer(score_of(base[i2]), i2);
#pragma unroll
  for (int k = 0; k < SB_KMAX; ++k) { s_val[k][tid] = v[k]; s_idx[k][tid] = id[k]; }
  __syncthreads();
  int pos = 0;
  for (int round = 0; round < SB_KMAX; ++round) {
    float hv = pos < SB_KMAX ? s_val[pos][tid] : -INFINITY;
    int hi = pos < SB_KMAX ? s_idx[pos][tid] : kNoId;
    int ht = tid;
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, hv, sft);
      const int oi = __shfl_xor_sync(0xffffffffu, hi, sft);
      const int ot = __shfl_xor_sync(0xffffffffu, ht, sft);
      if (ranks_before(ov, oi, hv, hi)) { hv = ov; hi = oi; ht = ot; }
    }
    if ((tid & 31) == 0) { s_wv[tid >> 5] = hv; s_wi[tid >> 5] = hi; s_wt[tid >> 5] = ht; }
    __syncthreads();
    if (tid == 0) {
      float bv = s_wv[0];
      int bi = s_wi[0], bt = s_wt[0];
      for (int w = 1; w < TOPK_THREADS / 32; ++w)
        if (ranks_before(s_wv[w], s_wi[w], bv, bi)) { bv = s_wv[w]; bi = s_wi[w]; bt = s_wt[w]; }
      out_val[round] = bv;
      out_idx[round] = bi;
      s_winner = bi == kNoId ? -1 : bt;
    }
    __syncthreads();
    if (tid == s_winner) ++pos;
  }
}

template <bool STATS>
__global__ void __launch_bounds__(TOPK_THREADS) topk_partial_reg_kernel(const float* __restrict__ scores,
                                                                        long long row_stride, int vocab, int chunk,
                                                                        int n_chunks, float* __restrict__ part_val,
                                                                        int* __restrict__ part_idx,
                                                                        float* __restrict__ part_stats, const int* __restrict__ n_nodes_in,
                                                                        int* __restrict__ n0_snapshot) {
  const int row = blockIdx.y, c = blockIdx.x;
  const float* base = scores + (long long)row * row_stride;
  const int begin = c * chunk;
  const int end = min(vocab, begin + chunk);
  pdl_release();  // the finishing kernel may start its prologue
  if (n0_snapshot && row == 0 && c == 0 && threadIdx.x == 0) *n0_snapshot = *n_nodes_in;  // the finishing kernel overwrites the counter
  const long long out0 = ((long long)row * n_chunks + c) * SB_KMAX;
  topk_reg_chunk<STATS>(base, begin, end, part_val + out0, part_idx + out0,
                        STATS ? part_stats + ((long long)row * n_chunks + c) * 3 : nullptr, []() {});
}

constexpr int FINISH_THREADS = 1024;

__global__ void __launch_bounds__(FINISH_THREADS) expand_finish_kernel(
    int n_rows, int n_chunks, const float* __restrict__ part_val, const int* __restrict__ part_idx, int block_k,
    const uint8_t* __restrict__ bucket, int4 bmap, const int* __restrict__ start_parent, int node_budget,
    int vocab, int* __restrict__ n_nodes, int* __restrict__ tok, int* __restrict__ parent, int* __restrict__ depth,
    int* __restrict__ node_row, int* __restrict__ node_rank, int* __restrict__ topk_tok,
    float* __restrict__ topk_val, int* __restrict__ child_row, int row_base, int* __restrict__ status) {
  __shared__ int s_bad;
  __shared__ int s_warp_sum[FINISH_THREADS / 32];
  __shared__ int s_first[FINISH_THREADS + 1];  // first node id of each row of the current slab
  __shared__ int s_carry;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) s_bad = 0;
  // Scalars of the first slab of rows are fetched now so that their latency hides under the merge.
  const int rows_slab0 = (FINISH_THREADS / block_k) * block_k;
  const bool pre_row = tid < rows_slab0 && tid < n_rows;
  const int pre_start = pre_row ? start_parent[tid / block_k] : -1;
  int pre_bucket[4] = {0, 0, 0, 0};  // buckets of this row and of up to three earlier positions of its block
  if (pre_row) {
    const int kp = tid % block_k;
    pre_bucket[0] = bucket[tid];
    if (kp >= 1) pre_bucket[1] = bucket[tid - 1];
    if (kp >= 2) pre_bucket[2] = bucket[tid - 2];
    if (kp >= 3) pre_bucket[3] = bucket[tid - 3];
  }
  const int pre_n0 = *n_nodes;
  const int pre_depth = (pre_row && pre_start >= 0 && pre_start < pre_n0) ? depth[pre_start] : 0;
  pdl_wait();  // the chunk lists of the scan kernel are complete from here on
  __syncthreads();
  // (1) merge the chunk lists of every row: lane c holds chunk c's sorted list in registers and
  //     pops it by shifting
  for (int r = warp; r < n_rows; r += FINISH_THREADS / 32) {
    float lv[SB_KMAX];
    int li[SB_KMAX];
    if (lane < n_chunks) {
      const float4* pv = reinterpret_cast<const float4*>(part_val + ((long long)r * n_chunks + lane) * SB_KMAX);
      const int4* pi = reinterpret_cast<const int4*>(part_idx + ((long long)r * n_chunks + lane) * SB_KMAX);
#pragma unroll
      for (int q = 0; q < SB_KMAX / 4; ++q) {
        const float4 a = pv[q];
        const int4 c = pi[q];
        lv[4 * q] = a.x; lv[4 * q + 1] = a.y; lv[4 * q + 2] = a.z; lv[4 * q + 3] = a.w;
        li[4 * q] = c.x; li[4 * q + 1] = c.y; li[4 * q + 2] = c.z; li[4 * q + 3] = c.w;
      }
    } else {
#pragma unroll
      for (int k = 0; k < SB_KMAX; ++k) { lv[k] = -INFINITY; li[k] = kNoId; }
    }
    float keep_v = -INFINITY;
    int keep_i = -1;
#pragma unroll
    for (int round = 0; round < SB_KMAX; ++round) {
      float hv = lv[0];
      int hi = li[0], hl = lane;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, hv, s);
        const int oi = __shfl_xor_sync(0xffffffffu, hi, s);
        const int ol = __shfl_xor_sync(0xffffffffu, hl, s);
        if (ranks_before(ov, oi, hv, hi)) { hv = ov; hi = oi; hl = ol; }
      }
      if (lane == round) { keep_v = hv; keep_i = hi == kNoId ? -1 : hi; }
      if (hi != kNoId && lane == hl) {
#pragma unroll
        for (int k = 0; k + 1 < SB_KMAX; ++k) { lv[k] = lv[k + 1]; li[k] = li[k + 1]; }
        lv[SB_KMAX - 1] = -INFINITY;
        li[SB_KMAX - 1] = kNoId;
      }
    }
    if (lane < SB_KMAX) {
      topk_tok[r * SB_KMAX + lane] = keep_i;
      topk_val[r * SB_KMAX + lane] = keep_v;
    }
  }
  // (2) argument checks that need device data
  const int n0 = pre_n0;
  if (tid == 0 && (n0 < 0 || n0 > node_budget)) s_bad = 1;
  for (int r = tid; r < n_rows; r += FINISH_THREADS)
    if (bucket[r] > 3) s_bad = 1;
  for (int i = tid; i < n_rows / block_k; i += FINISH_THREADS)
    if (start_parent[i] < -1 || start_parent[i] >= n0) s_bad = 1;
  if (tid == 0) s_carry = n0;
  __syncthreads();  // also publishes the merged lists to the whole CTA
  if (s_bad) {
    if (tid == 0) *status = SB_ERR_INVALID_ARG;
    return;
  }
  // (3) append, a slab of FINISH_THREADS rows at a time (slabs are cut at block boundaries)
  const int rows_per_slab = (FINISH_THREADS / block_k) * block_k > 0 ? (FINISH_THREADS / block_k) * block_k : 0;
  if (rows_per_slab == 0) {  // a block longer than a slab is not supported
    if (tid == 0) *status = SB_ERR_UNSUPPORTED;
    return;
  }
  for (int slab = 0; slab < n_rows; slab += rows_per_slab) {
    const int r = slab + tid;
    int width = 0, kpos = 0, start = -1;
    if (tid < rows_per_slab && r < n_rows) {
      kpos = r % block_k;
      start = slab == 0 ? pre_start : start_parent[r / block_k];
      auto width_of_bucket = [&](int bk) {
        const int w = bk == 0 ? bmap.x : bk == 1 ? bmap.y : bk == 2 ? bmap.z : bmap.w;
        return w < vocab ? w : vocab;
      };
      bool alive = true;
      for (int k = 1; k <= kpos; ++k) {
        const int bk = (slab == 0 && k <= 3) ? (k == 1 ? pre_bucket[1] : k == 2 ? pre_bucket[2] : pre_bucket[3]) : bucket[r - k];
        alive = alive && width_of_bucket(bk) >= 1;
      }
      width = alive ? width_of_bucket(slab == 0 ? pre_bucket[0] : bucket[r]) : 0;
    }
    // exclusive scan of the widths over the slab
    int incl = width;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, s);
      if (lane >= s) incl += o;
    }
    if (lane == 31) s_warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = s_warp_sum[lane];
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, w, s);
        if (lane >= s) w += o;
      }
      s_warp_sum[lane] = w;  // inclusive over warps
    }
    __syncthreads();
    const int carry = s_carry;
    const int first = carry + (warp > 0 ? s_warp_sum[warp - 1] : 0) + incl - width;
    s_first[tid] = first;
    __syncthreads();
    if (width > 0) {
      const int par = kpos == 0 ? start : s_first[tid - 1];  // rank-0 node of the previous position
      const int base_depth = start == -1 ? 0 : (slab == 0 ? pre_depth : depth[start]) + 1;
      for (int j = 0; j < width && first + j < node_budget; ++j) {
        const int n = first + j;
        if (!SB_CHECKED_ACCESS(n, node_budget, status)) break;
        tok[n] = topk_tok[r * SB_KMAX + j];
        parent[n] = par;
        depth[n] = base_depth + kpos;
        node_row[n] = row_base + r;
        node_rank[n] = j;
      }
      if (child_row && par >= 0 && first < node_budget && SB_CHECKED_ACCESS(par, node_budget, status))
        child_row[par] = row_base + r;  // this row proposed par's children
    }
    __syncthreads();
    if (tid == 0) s_carry = carry + s_warp_sum[FINISH_THREADS / 32 - 1];
    __syncthreads();
  }
  if (tid == 0) {
    *n_nodes = s_carry < node_budget ? s_carry : node_budget;
    *status = SB_OK;
  }
}

// The finishing kernel for up to ROWS_MAX rows: grid = rows, one CTA per row, no CTA waits for another.
//  - Before the dependency wait (so under the scan kernel): every CTA derives, from the call's inputs
//    alone, the width of every row (a row is alive iff every earlier position of its block has width
//    >= 1) and their exclusive prefix sum; it keeps what its own row needs (first node id relative to the
//    old node count, width, the previous row's first id = the parent of positions k > 0).
//  - After the wait: the old node count (a snapshot the scan kernel took of the in/out counter, which
//    CTA 0 overwrites at the end), the argument checks that need it, then the merge of the row's chunk
//    lists -- one sortable 64-bit key per candidate (the value mapped to an unsigned integer that grows
//    with it, -0 as +0 so that equal values tie, then the complement of the id; fillers below every real
//    entry and distinct by position), every candidate's rank = the number of larger keys, counted by
//    several threads per candidate -- and the row's own nodes: rank j < width becomes node first + j.
constexpr int ROWS_THREADS = 256;
constexpr int ROWS_MAX = 4 * ROWS_THREADS;
constexpr int MERGE_MAX = 32 * SB_KMAX;  // at most 32 chunk lists per row

__global__ void __launch_bounds__(ROWS_THREADS) expand_rows_kernel(
    int n_rows, int n_chunks, const float* __restrict__ part_val, const int* __restrict__ part_idx, int block_k,
    const uint8_t* __restrict__ bucket, int4 bmap, const int* __restrict__ start_parent, int node_budget,
    int vocab, const int* __restrict__ n0_snapshot, int* __restrict__ n_nodes, int* __restrict__ tok,
    int* __restrict__ parent, int* __restrict__ depth, int* __restrict__ node_row, int* __restrict__ node_rank,
    int* __restrict__ topk_tok, float* __restrict__ topk_val, int* __restrict__ child_row, int row_base,
    int* __restrict__ status) {
  __shared__ __align__(16) unsigned long long s_key[MERGE_MAX];
  __shared__ float s_val[MERGE_MAX];
  __shared__ int s_rank[MERGE_MAX];
  __shared__ int s_warp_sum[ROWS_THREADS / 32];
  __shared__ int s_my[3];  // this CTA's row: first id (relative), width, the previous row's first id (relative)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rr = blockIdx.x;
  const int n_cand = n_chunks * SB_KMAX;
  auto width_of_bucket = [&](int bk) {
    const int w = bk == 0 ? bmap.x : bk == 1 ? bmap.y : bk == 2 ? bmap.z : bmap.w;
    return w < vocab ? w : vocab;
  };
  // ---- inputs only: widths of all rows, their prefix sums, this row's share -------------------------
  const int rpt = ceil_div(n_rows, ROWS_THREADS);  // consecutive rows per thread (<= 4)
  int w_loc[4] = {0, 0, 0, 0};
  int wsum = 0;
  bool bad = false;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = tid * rpt + i;
    if (i < rpt && r < n_rows) {
      const int kpos = r % block_k;
      const int bk = bucket[r];
      bad = bad || bk > 3;
      bool alive = true;
      for (int k = 1; k <= kpos; ++k) alive = alive && width_of_bucket(bucket[r - k]) >= 1;
      w_loc[i] = alive ? width_of_bucket(bk) : 0;
      wsum += w_loc[i];
    }
  }
  int sp_loc[4] = {-1, -1, -1, -1};  // this thread's share of the starts, checked once the node count is known
  const int n_starts = n_rows / block_k;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (tid + i * ROWS_THREADS < n_starts) sp_loc[i] = start_parent[tid + i * ROWS_THREADS];
  const int start = start_parent[rr / block_k];
  const int start_depth = (start >= 0 && start < node_budget) ? depth[start] : 0;  // an existing node: never rewritten
  int incl = wsum;
#pragma unroll
  for (int sft = 1; sft < 32; sft <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, sft);
    if (lane >= sft) incl += o;
  }
  if (lane == 31) s_warp_sum[warp] = incl;
  for (int c = tid; c < n_cand; c += ROWS_THREADS) s_rank[c] = 0;
  __syncthreads();
  int run = incl - wsum;
  for (int w = 0; w < warp; ++w) run += s_warp_sum[w];
  int total = 0;
  for (int w = 0; w < ROWS_THREADS / 32; ++w) total += s_warp_sum[w];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = tid * rpt + i;
    if (i < rpt) {
      if (r == rr) { s_my[0] = run; s_my[1] = w_loc[i]; }
      if (r == rr - 1) s_my[2] = run;
      run += w_loc[i];
    }
  }
  pdl_wait();  // the chunk lists and the snapshot of the node count are complete from here on
  const int n0 = *n0_snapshot;
  bad = bad || n0 < 0 || n0 > node_budget;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (tid + i * ROWS_THREADS < n_starts) bad = bad || sp_loc[i] < -1 || sp_loc[i] >= n0;
  // ---- merge this row's chunk lists ----------------------------------------------------------------------
  const float* pv = part_val + (long long)rr * n_cand;
  const int* pi = part_idx + (long long)rr * n_cand;
  for (int c = tid; c < n_cand; c += ROWS_THREADS) {
    float v = pv[c];
    const int id = pi[c];
    s_val[c] = v;
    if (!(v == v)) v = -INFINITY;
    uint32_t u = __float_as_uint(v == 0.f ? 0.f : v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    const uint32_t low = id == kNoId ? 0x7fffffffu - (uint32_t)c : 0xffffffffu - (uint32_t)id;
    s_key[c] = ((unsigned long long)u << 32) | low;
  }
  const int any_bad = __syncthreads_or(bad ? 1 : 0);  // also publishes the keys, s_my and the zeroed counts
  {
    // candidate c, part p of the list: `parts` threads share one candidate
    const int parts = n_cand <= ROWS_THREADS ? ROWS_THREADS / n_cand : 1;
    const int n_pairs = n_cand / 2;
    const int per = ceil_div(n_pairs, parts);
    const ulonglong2* kp = reinterpret_cast<const ulonglong2*>(s_key);
    for (int w = tid; w < n_cand * parts; w += ROWS_THREADS) {
      const int c = w % n_cand, part = w / n_cand;
      const unsigned long long key = s_key[c];
      const int hi = min(n_pairs, (part + 1) * per);
      int cnt = 0;
#pragma unroll 2
      for (int o = part * per; o < hi; ++o) {
        const ulonglong2 k2 = kp[o];
        cnt += (k2.x > key ? 1 : 0) + (k2.y > key ? 1 : 0);
      }
      if (cnt) atomicAdd(&s_rank[c], cnt);
    }
  }
  __syncthreads();
  const int first = n0 + s_my[0], width = s_my[1];
  const int kpos = rr % block_k;
  const int par = kpos == 0 ? start : n0 + s_my[2];  // the rank-0 node of the previous position
  const int node_depth = (start == -1 ? 0 : start_depth + 1) + kpos;
  for (int c = tid; c < n_cand; c += ROWS_THREADS) {
    const int rank = s_rank[c];
    if (rank >= SB_KMAX) continue;
    const uint32_t low = (uint32_t)s_key[c];
    const int id = low < 0x80000000u ? -1 : (int)(0xffffffffu - low);
    topk_tok[rr * SB_KMAX + rank] = id;
    topk_val[rr * SB_KMAX + rank] = s_val[c];
    if (!any_bad && rank < width && first + rank < node_budget && SB_CHECKED_ACCESS(first + rank, node_budget, status)) {
      const int n = first + rank;
      tok[n] = id;
      parent[n] = par;
      depth[n] = node_depth;
      node_row[n] = row_base + rr;
      node_rank[n] = rank;
    }
  }
  // this row proposed the children of `par`: recorded for the calls that need the draft distribution of a node
  if (tid == 0 && child_row && !any_bad && width > 0 && first < node_budget && par >= 0 &&
      SB_CHECKED_ACCESS(par, node_budget, status))
    child_row[par] = row_base + rr;
  if (rr == 0 && tid == 0) {
    if (any_bad) {
      *status = SB_ERR_INVALID_ARG;
    } else {
      const int n_new = n0 + total;
      *n_nodes = n_new < node_budget ? n_new : node_budget;
      *status = SB_OK;
    }
  }
}

// ---- scan and finish in ONE kernel: the chunk CTAs of a row are a thread-block cluster -------------------
// For rows whose chunks fit the register-resident scan and one cluster (at most 16 chunks): every CTA takes
// the 16 best of its chunk exactly as topk_partial_reg_kernel does, but writes them into the shared memory of
// the cluster's first CTA (distributed shared memory) instead of a workspace; after one cluster barrier that
// CTA ranks the row's candidates and writes the row's top-16 and its own nodes, as expand_rows_kernel does.
// No chunk lists travel through global memory and no second grid has to start before a row is finished.
// The branching structure (which rows are alive, where their nodes go) depends on the inputs alone and is
// derived by the first CTA while its chunk is in flight.  The node counter is only READ here (by every
// finishing CTA, whenever it starts): the new count and the status word are written by expand_commit_kernel,
// a one-warp programmatic dependent that starts after this whole grid has completed, so no CTA of this grid
// can ever see the counter already advanced.
constexpr int XC_MAX_CHUNKS = 16;

__global__ void __launch_bounds__(TOPK_THREADS) expand_cluster_kernel(
    const float* __restrict__ scores, long long row_stride, int vocab, int chunk, int n_rows, int block_k,
    const uint8_t* __restrict__ bucket, int4 bmap, const int* __restrict__ start_parent, int node_budget,
    const int* __restrict__ n_nodes, int* __restrict__ tok, int* __restrict__ parent, int* __restrict__ depth,
    int* __restrict__ node_row, int* __restrict__ node_rank, int* __restrict__ topk_tok, float* __restrict__ topk_val,
    int* __restrict__ child_row, int row_base, int* __restrict__ commit, int* __restrict__ status) {
  static_assert(ROWS_THREADS == TOPK_THREADS, "the row structure is derived with the scan's block size");
  __shared__ float s_cand_val[XC_MAX_CHUNKS * SB_KMAX];  // the row's chunk lists: written by the cluster's CTAs
  __shared__ int s_cand_idx[XC_MAX_CHUNKS * SB_KMAX];
  __shared__ __align__(16) unsigned long long s_key[XC_MAX_CHUNKS * SB_KMAX];
  __shared__ int s_rank[XC_MAX_CHUNKS * SB_KMAX];
  __shared__ int s_warp_sum[ROWS_THREADS / 32];
  __shared__ int s_my[3];  // this row: first id (relative), width, the previous row's first id (relative)
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, rr = blockIdx.y;  // the cluster spans x: c is also the rank in the cluster
  const int n_chunks = gridDim.x;
  const int n_cand = n_chunks * SB_KMAX;
  const float* base = scores + (long long)rr * row_stride;
  const int begin = c * chunk;
  const int end = min(vocab, begin + chunk);
  pdl_release();  // expand_commit_kernel may take its place; it waits for this grid before it reads or writes

  auto width_of_bucket = [&](int bk) {
    const int w = bk == 0 ? bmap.x : bk == 1 ? bmap.y : bk == 2 ? bmap.z : bmap.w;
    return w < vocab ? w : vocab;
  };
  bool bad = false;
  int total = 0, n0 = 0, start = -1, start_depth = 0;
  auto structure = [&]() {
    if (c != 0) return;
    // inputs only: widths of all rows, their prefix sums, this row's share (as in expand_rows_kernel)
    const int rpt = ceil_div(n_rows, ROWS_THREADS);  // consecutive rows per thread (<= 4)
    int w_loc[4] = {0, 0, 0, 0};
    int wsum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = tid * rpt + i;
      if (i < rpt && r < n_rows) {
        const int kpos = r % block_k;
        const int bk = bucket[r];
        bad = bad || bk > 3;
        bool alive = true;
        for (int k = 1; k <= kpos; ++k) alive = alive && width_of_bucket(bucket[r - k]) >= 1;
        w_loc[i] = alive ? width_of_bucket(bk) : 0;
        wsum += w_loc[i];
      }
    }
    n0 = *n_nodes;  // the count before this call: nothing in this grid writes it
    bad = bad || n0 < 0 || n0 > node_budget;
    const int n_starts = n_rows / block_k;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (tid + i * ROWS_THREADS < n_starts) {
        const int sp = start_parent[tid + i * ROWS_THREADS];
        bad = bad || sp < -1 || sp >= n0;
      }
    start = start_parent[rr / block_k];
    start_depth = (start >= 0 && start < node_budget) ? depth[start] : 0;  // an existing node: never rewritten
    int incl = wsum;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, sft);
      if (lane >= sft) incl += o;
    }
    if (lane == 31) s_warp_sum[warp] = incl;
    for (int k = tid; k < n_cand; k += ROWS_THREADS) s_rank[k] = 0;
    __syncthreads();
    int run = incl - wsum;
    for (int w = 0; w < warp; ++w) run += s_warp_sum[w];
    for (int w = 0; w < ROWS_THREADS / 32; ++w) total += s_warp_sum[w];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = tid * rpt + i;
      if (i < rpt) {
        if (r == rr) { s_my[0] = run; s_my[1] = w_loc[i]; }
        if (r == rr - 1) s_my[2] = run;
        run += w_loc[i];
      }
    }
  };
  // the 16 best of this chunk, straight into the first CTA's candidate arrays
  float* out_val = cluster.map_shared_rank(s_cand_val, 0) + c * SB_KMAX;
  int* out_idx = cluster.map_shared_rank(s_cand_idx, 0) + c * SB_KMAX;
  topk_reg_chunk<false>(base, begin, end, out_val, out_idx, nullptr, structure);
  cluster.sync();  // every chunk's list has landed in the first CTA
  if (c != 0) return;

  // ---- merge this row's chunk lists (as expand_rows_kernel) -------------------------------------------------
  for (int k = tid; k < n_cand; k += ROWS_THREADS) {
    float v = s_cand_val[k];
    const int id = s_cand_idx[k];
    if (!(v == v)) v = -INFINITY;
    uint32_t u = __float_as_uint(v == 0.f ? 0.f : v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    const uint32_t low = id == kNoId ? 0x7fffffffu - (uint32_t)k : 0xffffffffu - (uint32_t)id;
    s_key[k] = ((unsigned long long)u << 32) | low;
  }
  const int any_bad = __syncthreads_or(bad ? 1 : 0);  // also publishes the keys
  {
    const int parts = n_cand <= ROWS_THREADS ? ROWS_THREADS / n_cand : 1;
    const int n_pairs = n_cand / 2;
    const int per = ceil_div(n_pairs, parts);
    const ulonglong2* kp = reinterpret_cast<const ulonglong2*>(s_key);
    for (int w = tid; w < n_cand * parts; w += ROWS_THREADS) {
      const int k = w % n_cand, part = w / n_cand;
      const unsigned long long key = s_key[k];
      const int hi = min(n_pairs, (part + 1) * per);
      int cnt = 0;
#pragma unroll 2
      for (int o = part * per; o < hi; ++o) {
        const ulonglong2 k2 = kp[o];
        cnt += (k2.x > key ? 1 : 0) + (k2.y > key ? 1 : 0);
      }
      if (cnt) atomicAdd(&s_rank[k], cnt);
    }
  }
  __syncthreads();
  const int first = n0 + s_my[0], width = s_my[1];
  const int kpos = rr % block_k;
  const int par = kpos == 0 ? start : n0 + s_my[2];  // the rank-0 node of the previous position
  const int node_depth = (start == -1 ? 0 : start_depth + 1) + kpos;
  for (int k = tid; k < n_cand; k += ROWS_THREADS) {
    const int rank = s_rank[k];
    if (rank >= SB_KMAX) continue;
    const uint32_t low = (uint32_t)s_key[k];
    const int id = low < 0x80000000u ? -1 : (int)(0xffffffffu - low);
    topk_tok[rr * SB_KMAX + rank] = id;
    topk_val[rr * SB_KMAX + rank] = s_cand_val[k];
    if (!any_bad && rank < width && first + rank < node_budget && SB_CHECKED_ACCESS(first + rank, node_budget, status)) {
      const int n = first + rank;
      tok[n] = id;
      parent[n] = par;
      depth[n] = node_depth;
      node_row[n] = row_base + rr;
      node_rank[n] = rank;
    }
  }
  if (tid == 0 && child_row && !any_bad && width > 0 && first < node_budget && par >= 0 &&
      SB_CHECKED_ACCESS(par, node_budget, status))
    child_row[par] = row_base + rr;
  if (rr == 0 && tid == 0) {  // what expand_commit_kernel publishes once the whole grid is done
    const int n_new = n0 + total;
    commit[0] = any_bad ? -1 : (n_new < node_budget ? n_new : node_budget);
  }
}

// One warp, a programmatic dependent of expand_cluster_kernel: the new node count and the status word.
__global__ void expand_commit_kernel(const int* __restrict__ commit, int* __restrict__ n_nodes, int* __restrict__ status) {
  pdl_release();
  pdl_wait();  // every CTA of the expansion grid has completed (and has read the old count)
  if (threadIdx.x == 0) {
    const int n_new = commit[0];
    if (n_new < 0) {
      *status = SB_ERR_INVALID_ARG;
    } else {
      *n_nodes = n_new;
      *status = SB_OK;
    }
  }
}

// psi(p) of every row from the chunk partials: a warp per row merges the chunk lists (value
// descending, id ascending) and the chunk statistics (m, s, t):  M = max m_c,
// S = sum s_c e^(m_c - M), T = sum t_c e^(m_c - M); ln Z = M + ln S; entropy = ln Z - T / S.
__global__ void __launch_bounds__(256) rank_features_finish_kernel(int n_rows, int n_chunks, int vocab,
                                                                   const float* __restrict__ part_val,
                                                                   const int* __restrict__ part_idx,
                                                                   const float* __restrict__ part_stats,
                                                                   float* __restrict__ features) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * 8 + warp;
  pdl_wait();  // the chunk lists and statistics of the scan kernel are complete from here on
  if (r >= n_rows) return;
  float lv[SB_KMAX];
  int li[SB_KMAX];
  float m = -INFINITY, sc = 0.f, tc = 0.f;
  if (lane < n_chunks) {
    const float4* pv = reinterpret_cast<const float4*>(part_val + ((long long)r * n_chunks + lane) * SB_KMAX);
    const int4* pi = reinterpret_cast<const int4*>(part_idx + ((long long)r * n_chunks + lane) * SB_KMAX);
#pragma unroll
    for (int q = 0; q < SB_KMAX / 4; ++q) {
      const float4 a = pv[q];
      const int4 c = pi[q];
      lv[4 * q] = a.x; lv[4 * q + 1] = a.y; lv[4 * q + 2] = a.z; lv[4 * q + 3] = a.w;
      li[4 * q] = c.x; li[4 * q + 1] = c.y; li[4 * q + 2] = c.z; li[4 * q + 3] = c.w;
    }
    const float* st = part_stats + ((long long)r * n_chunks + lane) * 3;
    m = st[0]; sc = st[1]; tc = st[2];
  } else {
#pragma unroll
    for (int k = 0; k < SB_KMAX; ++k) { lv[k] = -INFINITY; li[k] = kNoId; }
  }
  float M = m;
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sft));
  const float wgt = m > -INFINITY ? exp2f((m - M) * 1.4426950408889634f) : 0.f;
  float S = sc * wgt, T = tc * wgt;
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    S += __shfl_xor_sync(0xffffffffu, S, sft);
    T += __shfl_xor_sync(0xffffffffu, T, sft);
  }
  // the ten best values of the row, in order (lane k keeps rank k)
  float keep = -INFINITY;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    float hv = lv[0];
    int hi = li[0], hl = lane;
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, hv, sft);
      const int oi = __shfl_xor_sync(0xffffffffu, hi, sft);
      const int ol = __shfl_xor_sync(0xffffffffu, hl, sft);
      if (ranks_before(ov, oi, hv, hi)) { hv = ov; hi = oi; hl = ol; }
    }
    if (lane == round) keep = hi == kNoId ? NAN : hv;  // NaN marks "no such rank"
    if (hi != kNoId && lane == hl) {
#pragma unroll
      for (int k = 0; k + 1 < SB_KMAX; ++k) { lv[k] = lv[k + 1]; li[k] = li[k + 1]; }
      lv[SB_KMAX - 1] = -INFINITY;
      li[SB_KMAX - 1] = kNoId;
    }
  }
  const bool flat = !(M > -INFINITY);  // no finite score: reported as the uniform distribution
  const float log_z = flat ? logf((float)vocab) : M + logf(S);
  const float v0 = __shfl_sync(0xffffffffu, keep, 0);
  const float v1 = __shfl_sync(0xffffffffu, keep, 1);
  const float v2 = __shfl_sync(0xffffffffu, keep, 2);
  const float v4 = __shfl_sync(0xffffffffu, keep, 4);
  float* f = features + (long long)r * 15;
  if (lane < 10) {
    const bool exists = keep == keep;
    f[lane] = !exists ? -INFINITY : (flat ? -log_z : keep - log_z);
  }
  if (lane == 10) f[10] = v1 == v1 ? (flat ? 0.f : v0 - v1) : INFINITY;
  if (lane == 11) f[11] = v2 == v2 ? (flat ? 0.f : v0 - v2) : INFINITY;
  if (lane == 12) f[12] = v4 == v4 ? (flat ? 0.f : v0 - v4) : INFINITY;
  if (lane == 13) f[13] = flat ? 1.f / (float)vocab : expf(v0 - log_z);
  if (lane == 14) f[14] = flat ? log_z : log_z - T / S;
}

static int topk_chunks(int n_rows, int vocab) {
  // two CTAs of the partial kernels are resident per SM: keep rows * chunks within one wave
  int nc = (2 * 148) / (n_rows > 0 ? n_rows : 1);
  const int max_nc = ceil_div(vocab, 2048);
  if (nc > max_nc) nc = max_nc;
  const int reg_nc = ceil_div(vocab, TOPK_REG_ELEMS);  // chunks that fit the register-resident kernel
  if (nc < reg_nc) nc = reg_nc;
  if (nc > 32) nc = 32;
  if (nc < 1) nc = 1;
  return nc;
}

// Bytes of one kind of chunk lists (values, or ids) of all rows, rounded to 256.
static size_t topk_list_bytes(int n_rows, int vocab) {
  return ((size_t)n_rows * topk_chunks(n_rows, vocab) * SB_KMAX * 4 + 255) & ~(size_t)255;
}

// Dynamic shared memory of topk_partial_reg_kernel: the staged chunk.  Both instantiations are told
// once that they may exceed the default 48 KB together with their static arrays.
static size_t topk_stage_bytes(int chunk) {
  static PerDeviceOnce once;
  once.run([]() {
    const bool ok =
        cudaFuncSetAttribute(expand_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TOPK_STAGE_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(expand_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(topk_partial_reg_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, TOPK_STAGE_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(topk_partial_reg_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TOPK_STAGE_BYTES) == cudaSuccess;
    if (!ok) cudaGetLastError();
    return ok;  // a failure shows as a launch error of the scan
  });
  return (size_t)chunk * sizeof(float);
}

// Launch configuration of expand_cluster_kernel for `nc` chunks per row.
static cudaLaunchConfig_t expand_cluster_config(dim3 grid, int nc, size_t smem, cudaStream_t cs, cudaLaunchAttribute* attr) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(TOPK_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = cs;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = nc;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cfg;
}

// Clusters of `nc` CTAs of expand_cluster_kernel that can be resident at once on the current device.
static int expand_cluster_fit(int nc) {
  static PerDeviceInt cache[XC_MAX_CHUNKS + 1];
  if (nc < 1 || nc > XC_MAX_CHUNKS) return 0;
  return cache[nc].get([&]() {
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = expand_cluster_config(dim3(nc, 64), nc, topk_stage_bytes(TOPK_REG_ELEMS), nullptr, attr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, expand_cluster_kernel, &cfg) != cudaSuccess) {
      cudaGetLastError();
      n = 0;
    }
    return n;
  }, 0);
}

// Chunks per row for expand_cluster_kernel: as many as topk_chunks() wants while all rows' clusters are
// resident together (288 CTAs in clusters of 9 do not fit a B200, 256 in clusters of 8 do), never fewer
// than the register-resident scan needs.
static int expand_cluster_chunks(int n_rows, int vocab) {
  const int reg_nc = ceil_div(vocab, TOPK_REG_ELEMS);
  int nc = topk_chunks(n_rows, vocab);
  if (nc > XC_MAX_CHUNKS) nc = XC_MAX_CHUNKS;
  while (nc > reg_nc && expand_cluster_fit(nc) < n_rows) --nc;
  return nc;
}

}  // namespace sb

extern "C" size_t sb_tree_expand_workspace_bytes(int32_t n_rows, int32_t vocab) {
  if (n_rows < 1 || vocab < 1) return 0;
  return 2 * sb::topk_list_bytes(n_rows, vocab) + 256;  // value lists, id lists, the snapshot of the node count
}

// sb_tree_expand, and with `features` the distribution summaries of sb_rank_features from the same scan.
static sb_status expand_impl(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                             int32_t block_k, const uint8_t* bucket, const int32_t* bmap,
                             const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                             int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                             int32_t* node_rank, int32_t* topk_tok, float* topk_val, float* features,
                             int32_t* child_row, int32_t row_base, void* workspace, size_t workspace_bytes,
                             int32_t* status, void* stream) {
  using namespace sb;
  if (!scores || !bucket || !bmap || !start_parent || !n_nodes || !tok || !parent || !depth || !node_row ||
      !node_rank || !topk_tok || !topk_val || !status || n_rows < 1 || vocab < 1 || row_stride < vocab ||
      block_k < 1 || n_rows % block_k != 0 || node_budget < 1)
    return SB_ERR_INVALID_ARG;
  for (int m = 0; m < 4; ++m)
    if (bmap[m] < 0 || bmap[m] > SB_KMAX) return SB_ERR_INVALID_ARG;
  if (n_rows > 65535 || block_k > FINISH_THREADS) return SB_ERR_UNSUPPORTED;
  const size_t need = features ? sb_rank_features_workspace_bytes(n_rows, vocab) : sb_tree_expand_workspace_bytes(n_rows, vocab);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int nc = topk_chunks(n_rows, vocab);
  int chunk = ceil_div(vocab, nc);
  chunk = ceil_div(chunk, 4) * 4;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(scores) & 15) == 0 && row_stride % 4 == 0;
  const size_t list_bytes = topk_list_bytes(n_rows, vocab);
  float* part_val = static_cast<float*>(workspace);
  int* part_idx = reinterpret_cast<int*>(static_cast<char*>(workspace) + list_bytes);
  int* n0_snapshot = reinterpret_cast<int*>(static_cast<char*>(workspace) + 2 * list_bytes);
  float* part_stats = features ? reinterpret_cast<float*>(static_cast<char*>(workspace) + 2 * list_bytes + 256) : nullptr;
  const bool by_rows = n_rows <= ROWS_MAX;  // else the single-CTA finishing kernel, which reads the counter itself
  int* snap = by_rows ? n0_snapshot : nullptr;
  dim3 grid(nc, n_rows);
  const bool reg = vec_ok && chunk <= TOPK_REG_ELEMS;
  if (vec_ok && !features && by_rows && ceil_div(vocab, TOPK_REG_ELEMS) <= XC_MAX_CHUNKS) {
    // scan and finish in one grid: the chunks of a row are a cluster (expand_cluster_kernel), then a one-warp commit
    const int ncc = expand_cluster_chunks(n_rows, vocab);
    const int cchunk = ceil_div(ceil_div(vocab, ncc), 4) * 4;
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = expand_cluster_config(dim3(ncc, n_rows), ncc, topk_stage_bytes(cchunk), cs, attr);
    if (cudaLaunchKernelEx(&cfg, expand_cluster_kernel, scores, (long long)row_stride, (int)vocab, cchunk, (int)n_rows,
                           (int)block_k, bucket, make_int4(bmap[0], bmap[1], bmap[2], bmap[3]), start_parent,
                           (int)node_budget, (const int*)n_nodes, tok, parent, depth, node_row, node_rank, topk_tok,
                           topk_val, child_row, (int)row_base, n0_snapshot, status) != cudaSuccess) {
      cudaGetLastError();
      return SB_ERR_CUDA;
    }
    sb_status st1 = launch_check();
    if (st1 != SB_OK) return st1;
    return launch_dependent(expand_commit_kernel, dim3(1), dim3(32), cs, (const int*)n0_snapshot, n_nodes, status);
  }
  if (reg && features)
    topk_partial_reg_kernel<true><<<grid, TOPK_THREADS, topk_stage_bytes(chunk), cs>>>(scores, row_stride, vocab, chunk, nc,
                                                                                    part_val, part_idx, part_stats, n_nodes, snap);
  else if (reg)
    topk_partial_reg_kernel<false><<<grid, TOPK_THREADS, topk_stage_bytes(chunk), cs>>>(scores, row_stride, vocab, chunk, nc,
                                                                                     part_val, part_idx, nullptr, n_nodes, snap);
  else if (features)
    topk_partial_kernel<true><<<grid, TOPK_THREADS, 0, cs>>>(scores, row_stride, vocab, chunk, nc, vec_ok, part_val, part_idx,
                                                             part_stats, n_nodes, snap);
  else
    topk_partial_kernel<false><<<grid, TOPK_THREADS, 0, cs>>>(scores, row_stride, vocab, chunk, nc, vec_ok, part_val, part_idx,
                                                              nullptr, n_nodes, snap);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  if (by_rows)
    st = launch_dependent(expand_rows_kernel, dim3(n_rows), dim3(ROWS_THREADS), cs, n_rows, nc, part_val, part_idx,
                          block_k, bucket, make_int4(bmap[0], bmap[1], bmap[2], bmap[3]), start_parent, node_budget,
                          vocab, n0_snapshot, n_nodes, tok, parent, depth, node_row, node_rank, topk_tok, topk_val,
                          child_row, (int)row_base, status);
  else
    st = launch_dependent(expand_finish_kernel, dim3(1), dim3(FINISH_THREADS), cs, n_rows, nc, part_val, part_idx,
                          block_k, bucket, make_int4(bmap[0], bmap[1], bmap[2], bmap[3]), start_parent, node_budget,
                          vocab, n_nodes, tok, parent, depth, node_row, node_rank, topk_tok, topk_val, child_row,
                          (int)row_base, status);
  if (st != SB_OK || !features) return st;
  // the summaries read the same chunk lists and the chunk statistics; as a dependent of the finishing kernel
  // (which waited for the scan) their wait covers the scan too
  return launch_dependent(rank_features_finish_kernel, dim3(ceil_div(n_rows, 8)), dim3(256), cs, n_rows, nc, vocab,
                          part_val, part_idx, part_stats, features);
}

extern "C" sb_status sb_tree_expand(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                    int32_t block_k, const uint8_t* bucket, const int32_t* bmap,
                                    const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                                    int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                                    int32_t* node_rank, int32_t* topk_tok, float* topk_val, void* workspace,
                                    size_t workspace_bytes, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_tree_expand");
  return expand_impl(scores, row_stride, n_rows, vocab, block_k, bucket, bmap, start_parent, node_budget, n_nodes, tok,
                     parent, depth, node_row, node_rank, topk_tok, topk_val, nullptr, nullptr, 0, workspace,
                     workspace_bytes, status, stream);
}

extern "C" sb_status sb_tree_expand_features(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                             int32_t block_k, const uint8_t* bucket, const int32_t* bmap,
                                             const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                                             int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                                             int32_t* node_rank, int32_t* topk_tok, float* topk_val, float* features,
                                             int32_t* child_row, int32_t row_base, void* workspace,
                                             size_t workspace_bytes, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_tree_expand_features");
  if (!features || row_base < 0) return SB_ERR_INVALID_ARG;
  return expand_impl(scores, row_stride, n_rows, vocab, block_k, bucket, bmap, start_parent, node_budget, n_nodes, tok,
                     parent, depth, node_row, node_rank, topk_tok, topk_val, features, child_row, row_base, workspace,
                     workspace_bytes, status, stream);
}

extern "C" size_t sb_rank_features_workspace_bytes(int32_t n_rows, int32_t vocab) {
  if (n_rows < 1 || vocab < 1) return 0;
  const size_t nc = (size_t)sb::topk_chunks(n_rows, vocab);
  return sb_tree_expand_workspace_bytes(n_rows, vocab) + (((size_t)n_rows * nc * 3 * 4 + 255) & ~(size_t)255);
}

extern "C" sb_status sb_rank_features(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                      float* features, void* workspace, size_t workspace_bytes, void* stream) {
  sb::TraceRange trace_range("sb_rank_features");
  using namespace sb;
  if (!scores || !features || n_rows < 1 || vocab < 1 || row_stride < vocab) return SB_ERR_INVALID_ARG;
  if (n_rows > 65535) return SB_ERR_UNSUPPORTED;
  const size_t need = sb_rank_features_workspace_bytes(n_rows, vocab);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int nc = topk_chunks(n_rows, vocab);
  int chunk = ceil_div(vocab, nc);
  chunk = ceil_div(chunk, 4) * 4;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(scores) & 15) == 0 && row_stride % 4 == 0;
  const size_t list_bytes = topk_list_bytes(n_rows, vocab);
  float* part_val = static_cast<float*>(workspace);
  int* part_idx = reinterpret_cast<int*>(static_cast<char*>(workspace) + list_bytes);
  float* part_stats = reinterpret_cast<float*>(static_cast<char*>(workspace) + 2 * list_bytes + 256);
  dim3 grid(nc, n_rows);
  if (vec_ok && chunk <= TOPK_REG_ELEMS)
    topk_partial_reg_kernel<true><<<grid, TOPK_THREADS, topk_stage_bytes(chunk), cs>>>(scores, row_stride, vocab, chunk, nc, part_val,
                                                                 part_idx, part_stats, nullptr, nullptr);
  else
    topk_partial_kernel<true><<<grid, TOPK_THREADS, 0, cs>>>(scores, row_stride, vocab, chunk, nc, vec_ok, part_val,
                                                             part_idx, part_stats, nullptr, nullptr);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  return launch_dependent(rank_features_finish_kernel, dim3(ceil_div(n_rows, 8)), dim3(256), cs, n_rows, nc, vocab,
                          part_val, part_idx, part_stats, features);
}
