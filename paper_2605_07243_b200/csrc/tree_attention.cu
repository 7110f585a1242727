// sb_tree_attention: tree-masked split-KV attention of one layer (Sec. 3.1; App. A.2; Alg. 1 "verify").
//
// Every node of a draft tree attends to the whole verified prefix plus its own ancestors
// (itself included).  Query rows of one KV head are packed as (node, head-in-group) so a CTA's
// 128-row tile shares every K/V tile it streams (GQA head packing).  The ancestor sets live in
// shared memory as one 128-bit mask per node and are applied only to the KV tiles that overlap
// the tree's cache slots; prefix tiles run unmasked.  The KV range of a (sequence, KV head, row
// tile) is cut into `num_splits` chunks handled by different CTAs.  Up to 8 chunk-CTAs form a
// thread-block cluster and merge their (out, max, sum) triples through distributed shared
// memory, so for up to 8 chunks nothing but the final result is written; beyond 8 chunks each
// cluster writes one partial and a second kernel merges the clusters' (out, log-sum-exp) pairs.
//
// Kernels in this file
//   attn_merge_kernel  : log-sum-exp merge of the clusters' partials (only beyond one cluster of chunks).
//   The attention itself runs on the tcgen05/TMEM kernels of tree_attention_tc.cu / tree_attention_tc2.cu;
//   the library has this one backend and reads no environment variable.
// Only in the test build (-DSB_TEST_KERNELS, libspecblock_test.so), as independent cross-checks of the
// tcgen05 kernels and as switches that force a kernel variant onto a shape the planner would not give it:
//   attn_simple_kernel : one warp per query row, fp32 FMA (SB_ATTN_IMPL=simple).
//   attn_mma_kernel    : flash-decode with bf16 mma.sync (m16n8k16), fp32 accumulate, 3-stage cp.async
//                        K/V pipeline in XOR-swizzled shared memory (SB_ATTN_IMPL=mma).
//   SB_ATTN_TWO_TILES, SB_ATTN_MAX_CLUSTER, SB_NO_PDL, SB_DEBUG.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "attention_common.cuh"

namespace sb {

// tcgen05 kernel (tree_attention_tc.cu)
sb_status launch_attn_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs);
int attn_tc_max_active_clusters(int D, int cluster);
sb_status launch_attn_tc2(const AttnParams& p, dim3 grid, cudaStream_t cs);

constexpr int BM = 128;       // query rows per CTA tile

#ifdef SB_TEST_KERNELS
// ----------------------------------------------------------------------------------------------
// Simple kernel: one warp per (node, head) row.
// ----------------------------------------------------------------------------------------------

template <int D>
__global__ void __launch_bounds__(256) attn_simple_kernel(const AttnParams p) {
  constexpr int E = D / 32;  // elements per lane
  __shared__ int s_parent[SB_MAX_NODES];
  __shared__ uint32_t s_anc[SB_MAX_NODES * 4];
  const int b = blockIdx.y;
  const SeqPlan sp = plan_sequence(p, b, blockIdx.x == 0, s_parent, s_anc);
  const SeqInfo& si = sp.info;
  const int Hq = p.tb.n_q_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rr = blockIdx.x * 8 + warp;
  if (!sp.can_write || rr >= si.nq * Hq) return;
  const int node = si.q0 + rr / Hq, h = rr % Hq, g = h / p.G;
  const long long grow = (long long)si.q_off * Hq + rr;
  bf16* orow = p.out + grow * D + lane * E;
  if (!sp.compute) {
#pragma unroll
    for (int e = 0; e < E; ++e) orow[e] = __float2bfloat16(0.f);
    if (p.lse && lane == 0) p.lse[grow] = 0.f;
    return;
  }
  float qv[E], acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    qv[e] = __bfloat162float(p.q[grow * D + lane * E + e]);
    acc[e] = 0.f;
  }
  const bf16* kc = static_cast<const bf16*>(p.tb.k_cache);
  const bf16* vc = static_cast<const bf16*>(p.tb.v_cache);
  float m = -INFINITY, l = 0.f;
  const int L = si.P + si.n;
  for (int j = 0; j < L; ++j) {
    const int rel = j - si.P;
    if (rel >= 0 && !((s_anc[4 * node + (rel >> 5)] >> (rel & 31)) & 1u)) continue;
    const long long off = kv_row_elem_offset(p.tb, b, j) + (long long)g * D + lane * E;
    float dot = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) dot += qv[e] * __bfloat162float(kc[off + e]);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
    const float s2 = dot * p.scale_log2;
    const float m_new = fmaxf(m, s2);
    const float corr = exp2f(m - m_new);
    const float pj = exp2f(s2 - m_new);
    l = l * corr + pj;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + pj * __bfloat162float(vc[off + e]);
    m = m_new;
  }
#pragma unroll
  for (int e = 0; e < E; ++e) orow[e] = __float2bfloat16(acc[e] / l);
  if (p.lse && lane == 0) p.lse[grow] = (m + log2f(l)) * kLn2;
}

// ----------------------------------------------------------------------------------------------
// Tensor-core (mma.sync) flash-decode kernel.
// ----------------------------------------------------------------------------------------------

constexpr int BN = 64;        // keys per pipeline stage (BM = 8 warps x 16 rows)
constexpr int NTHREADS = 256;
constexpr int STAGES = 3;

__device__ inline void cp_async_16(void* smem_dst, const void* gmem_src, int src_bytes) {
  const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(gmem_src), "r"(src_bytes));
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ inline void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ inline void ldmatrix_x4(uint32_t (&r)[4], const void* smem_src) {
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(smem_src));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}
__device__ inline void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_src) {
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(smem_src));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}
__device__ inline void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <int D>
constexpr size_t attn_mma_smem_bytes() {
  return 2560 + (size_t)BM * D * 2 + 2 * (size_t)STAGES * BN * D * 2;
}

template <int D>
__global__ void __launch_bounds__(NTHREADS, 1) attn_mma_kernel(const AttnParams p) {
  constexpr int CH = D / 8;       // 16-byte chunks per row
  constexpr int KSTEPS = D / 16;  // MMA k-steps of Q.K^T
  constexpr int DT = D / 8;       // 8-wide column tiles of the output
  extern __shared__ __align__(128) uint8_t smem[];
  uint32_t* s_anc = reinterpret_cast<uint32_t*>(smem);
  int* s_parent = reinterpret_cast<int*>(smem + 2048);
  bf16* s_q = reinterpret_cast<bf16*>(smem + 2560);
  bf16* s_k = s_q + BM * D;
  bf16* s_v = s_k + STAGES * BN * D;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks();   // chunk-CTAs that merge through shared memory
  const int crank = (int)cluster.block_rank();
  const int split = blockIdx.x;              // chunk index among num_splits = S * outer
  const int Hq = p.tb.n_q_heads, G = p.G;
  // row tiles of one (sequence, KV head) are neighbours in launch order: they share its K/V through L2
  const int g = blockIdx.y / p.row_tiles, tile = blockIdx.y % p.row_tiles;
  const int b = blockIdx.z;

  const SeqPlan sp = plan_sequence(p, b, split == 0 && blockIdx.y == 0, s_parent, s_anc);
  const SeqInfo& si = sp.info;
  const int rows_total = si.nq * G;
  const int row0 = tile * BM;
  // Uniform over the cluster (depends on the sequence and the row tile only).
  if (!sp.can_write || row0 >= rows_total) return;
  const long long rows_all = (long long)p.total_q * Hq;

  // This thread's two accumulator rows: warp*16 + lane/4 and that + 8.
  uint32_t anc[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int R = row0 + warp * 16 + (lane >> 2) + 8 * i;
    const bool ok = R < rows_total && sp.compute;
    const int node = ok ? si.q0 + R / G : 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) anc[i][w] = ok ? s_anc[4 * node + w] : 0u;
  }

  // Balanced cut of the sequence's T key tiles into num_splits chunks.
  const int L = si.P + si.n;
  const int T = ceil_div(L, BN);
  const int t_base = T / p.num_splits, t_rem = T % p.num_splits;
  const int t_begin = split * t_base + min(split, t_rem);
  const int n_tiles = sp.compute ? t_base + (split < t_rem ? 1 : 0) : 0;

  const bf16* kc = static_cast<const bf16*>(p.tb.k_cache) + (long long)g * D;
  const bf16* vc = static_cast<const bf16*>(p.tb.v_cache) + (long long)g * D;

  auto load_kv_tile = [&](int tile_idx, int stage) {
    bf16* dk = s_k + stage * BN * D;
    bf16* dv = s_v + stage * BN * D;
#pragma unroll
    for (int i = 0; i < BN * CH / NTHREADS; ++i) {
      const int c = tid + i * NTHREADS;
      const int r = c / CH, ch = c % CH;
      const int j = tile_idx * BN + r;
      const bool valid = j < L;
      const long long off = valid ? kv_row_elem_offset(p.tb, b, j) + ch * 8 : 0;
      const int so = r * D + ((ch ^ (r & 7)) * 8);
      cp_async_16(dk + so, kc + off, valid ? 16 : 0);
      cp_async_16(dv + so, vc + off, valid ? 16 : 0);
    }
  };

  // Q tile -> shared memory (rows beyond the sequence's rows are zero-filled).
#pragma unroll
  for (int i = 0; n_tiles > 0 && i < BM * CH / NTHREADS; ++i) {
    const int c = tid + i * NTHREADS;
    const int r = c / CH, ch = c % CH;
    const int R = row0 + r;
    const bool valid = R < rows_total;
    const int node_l = valid ? R / G : 0;
    const int hh = valid ? R - node_l * G : 0;
    const long long off = ((long long)(si.q_off + node_l) * Hq + g * G + hh) * D + ch * 8;
    cp_async_16(s_q + r * D + ((ch ^ (r & 7)) * 8), p.q + (valid ? off : 0), valid ? 16 : 0);
  }
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < n_tiles) load_kv_tile(t_begin + s, s);
    cp_async_commit();
  }

  uint32_t qf[KSTEPS][4];
  float o_acc[DT][4];
#pragma unroll
  for (int d = 0; d < DT; ++d)
#pragma unroll
    for (int e = 0; e < 4; ++e) o_acc[d][e] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};

  for (int it = 0; it < n_tiles; ++it) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    if (it + STAGES - 1 < n_tiles) load_kv_tile(t_begin + it + STAGES - 1, (it + STAGES - 1) % STAGES);
    cp_async_commit();

    if (it == 0) {
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        const int r = warp * 16 + (lane & 15);
        const int ch = 2 * ks + (lane >> 4);
        ldmatrix_x4(qf[ks], s_q + r * D + ((ch ^ (r & 7)) * 8));
      }
    }
    const bf16* sk = s_k + (it % STAGES) * BN * D;
    const bf16* sv = s_v + (it % STAGES) * BN * D;

    // S = Q K^T for 16 rows x 64 keys
    float s_acc[BN / 8][4];
#pragma unroll
    for (int nt = 0; nt < BN / 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) s_acc[nt][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
#pragma unroll
      for (int np = 0; np < BN / 16; ++np) {
        uint32_t kb[4];
        const int r = np * 16 + (lane & 7) + ((lane >> 4) << 3);
        const int ch = 2 * ks + ((lane >> 3) & 1);
        ldmatrix_x4(kb, sk + r * D + ((ch ^ (r & 7)) * 8));
        mma_bf16_16816(s_acc[2 * np], qf[ks], kb[0], kb[1]);
        mma_bf16_16816(s_acc[2 * np + 1], qf[ks], kb[2], kb[3]);
      }
    }

    // scale, tree mask (only tiles that reach past the prefix), online softmax
    const int key0 = (t_begin + it) * BN;
    const bool need_mask = key0 + BN > si.P;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      // bit c of `win`: is key key0 + (lane%4)*2 + c visible to this row
      const uint64_t win = need_mask ? visibility_window(anc[i], key0 - si.P) >> ((lane & 3) * 2) : ~0ull;
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float s2 = s_acc[nt][2 * i + e] * p.scale_log2;
          if (need_mask) s2 = ((win >> (nt * 8 + e)) & 1ull) ? s2 : -INFINITY;
          s_acc[nt][2 * i + e] = s2;
          mx = fmaxf(mx, s2);
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run[i], mx);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      const float corr = fast_exp2(m_run[i] - m_use);
      m_run[i] = m_new;
      l_run[i] *= corr;
#pragma unroll
      for (int d = 0; d < DT; ++d) {
        o_acc[d][2 * i] *= corr;
        o_acc[d][2 * i + 1] *= corr;
      }
      float ls = 0.f;
#pragma unroll
      for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float pe = fast_exp2(s_acc[nt][2 * i + e] - m_use);
          s_acc[nt][2 * i + e] = pe;
          ls += pe;
        }
      }
      l_run[i] += ls;
    }

    // O += P V
#pragma unroll
    for (int kk = 0; kk < BN / 16; ++kk) {
      uint32_t pa[4];
      pa[0] = pack_bf16(s_acc[2 * kk][0], s_acc[2 * kk][1]);
      pa[1] = pack_bf16(s_acc[2 * kk][2], s_acc[2 * kk][3]);
      pa[2] = pack_bf16(s_acc[2 * kk + 1][0], s_acc[2 * kk + 1][1]);
      pa[3] = pack_bf16(s_acc[2 * kk + 1][2], s_acc[2 * kk + 1][3]);
#pragma unroll
      for (int dp = 0; dp < D / 16; ++dp) {
        uint32_t vb[4];
        const int r = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
        const int ch = 2 * dp + (lane >> 4);
        ldmatrix_x4_trans(vb, sv + r * D + ((ch ^ (r & 7)) * 8));
        mma_bf16_16816(o_acc[2 * dp], pa, vb[0], vb[1]);
        mma_bf16_16816(o_acc[2 * dp + 1], pa, vb[2], vb[3]);
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();  // every warp is done with the K/V stages: reuse them as the merge buffer
  if (S > 1) cluster.sync();  // ... in every CTA of the cluster: peers are about to write into them

  // ---- epilogue: every row goes to the shared memory of the cluster CTA that owns it; one cluster
  // barrier; each CTA reduces and stores its rows (with S = 1 this is just a coalescing stage).
  MergeBuf<D> mb(reinterpret_cast<float*>(s_k), BM, S);
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float l = l_run[i];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    const int r = warp * 16 + (lane >> 2) + 8 * i;
    const int c0 = (lane & 3) * 2;
    int slot;
    float* dst = merge_row_dst<D>(cluster, mb, crank, r, &slot);
    if (n_tiles > 0) {
#pragma unroll
      for (int d = 0; d < DT; ++d)
        *reinterpret_cast<float2*>(dst + d * 8 + c0) = make_float2(o_acc[d][2 * i], o_acc[d][2 * i + 1]);
    }
    if ((lane & 3) == 0) merge_push_ml<D>(cluster, mb, crank, r, n_tiles > 0 ? m_run[i] : -INFINITY, n_tiles > 0 ? l : 0.f);
  }
  if (S > 1) cluster.sync(); else __syncthreads();
  merge_reduce_and_store<D, BM>(p, mb, S, crank, split / S, row0, rows_total, g, si.q_off, rows_all, tid, NTHREADS);
}

#endif  // SB_TEST_KERNELS

// ----------------------------------------------------------------------------------------------
// Merge of split partials: out = sum_s w_s out_s, w_s = 2^(lse_s - M) / sum_s 2^(lse_s - M).
// One warp per (node, head) row.
// ----------------------------------------------------------------------------------------------

// One 16-byte load per lane and chunk: a row takes D/8 lanes with bf16 partials, D/4 with fp32 ones, so a
// warp holds one, two or four rows; every lane finds the row's reference maximum itself (the log-sum-exps are
// a few broadcast loads) and then has eight chunks' loads in flight at a time, none of them waiting for a
// weight: a chunk that saw no key for the row did not write its partial, so what was loaded for it is
// dropped by a select instead of being skipped by a branch.
template <int D, bool PB16>
constexpr int merge_rows_per_cta() { return 8 * (32 / (D / (PB16 ? 8 : 4))); }

template <int D, bool PB16>
__global__ void __launch_bounds__(256) attn_merge_kernel(const AttnParams p) {
  constexpr int EPL = PB16 ? 8 : 4;  // elements per lane
  constexpr int LPR = D / EPL;       // lanes per row
  constexpr int RPW = 32 / LPR;      // rows per warp
  constexpr int UN = 8;
  const int b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Sequences whose lengths are bad still own their rows (zero-filled by the empty partials).
  const int o = p.tb.node_offsets[b];
  const int n_raw = p.tb.node_offsets[b + 1] - o;
  const int q0 = p.q_node_begin ? p.q_node_begin[b] : 0;
  const int q_off = p.q_offsets ? p.q_offsets[b] : o;
  const bool rows_ok = n_raw >= 0 && n_raw <= SB_MAX_NODES && n_raw <= p.tb.max_nodes && q0 >= 0 &&
                       q0 <= n_raw && q_off >= 0 && (long long)q_off + (n_raw - q0) <= p.total_q &&
                       o >= 0 && (long long)o + n_raw <= p.tb.total_nodes;
  if (!rows_ok) return;
  const int Hq = p.tb.n_q_heads;
  const int rr = (blockIdx.x * 8 + warp) * RPW + lane / LPR;
  const int col = lane % LPR;
  if (rr >= (n_raw - q0) * Hq) return;
  const long long rows_all = (long long)p.total_q * Hq;
  const long long grow = (long long)q_off * Hq + rr;
  if (!SB_CHECKED_ACCESS(grow, rows_all, &p.status[b])) return;
  float M = -INFINITY;
  for (int s = 0; s < p.outer; ++s) M = fmaxf(M, p.part_lse[s * rows_all + grow]);
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  float denom = 0.f;
  if (M != -INFINITY) {
    for (int s0 = 0; s0 < p.outer; s0 += UN) {
      uint4 raw[UN];
      float w[UN];
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int s = s0 + u;
        if (s < p.outer) {
          const char* src = reinterpret_cast<const char*>(p.part_o) +
                            ((s * rows_all + grow) * D + col * EPL) * (PB16 ? 2 : 4);
          raw[u] = *reinterpret_cast<const uint4*>(src);
        }
      }
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int s = s0 + u;
        const float ls = s < p.outer ? p.part_lse[s * rows_all + grow] : -INFINITY;
        w[u] = ls != -INFINITY ? exp2f(ls - M) : 0.f;
        denom += w[u];
      }
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        if (s0 + u >= p.outer) break;
        const uint32_t q4[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
        const bool live = w[u] != 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (PB16) {
            acc[2 * e] += live ? w[u] * __uint_as_float(q4[e] << 16) : 0.f;
            acc[2 * e + 1] += live ? w[u] * __uint_as_float(q4[e] & 0xffff0000u) : 0.f;
          } else {
            acc[e] += live ? w[u] * __uint_as_float(q4[e]) : 0.f;
          }
        }
      }
    }
  }
  const float inv = denom > 0.f ? 1.f / denom : 0.f;
  bf16* orow = p.out + grow * D + col * EPL;
  if (PB16) {
    uint4 o4;
    o4.x = pack_bf16(acc[0] * inv, acc[1] * inv);
    o4.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    o4.z = pack_bf16(acc[EPL - 4] * inv, acc[EPL - 3] * inv);
    o4.w = pack_bf16(acc[EPL - 2] * inv, acc[EPL - 1] * inv);
    *reinterpret_cast<uint4*>(orow) = o4;
  } else {
    uint2 o2;
    o2.x = pack_bf16(acc[0] * inv, acc[1] * inv);
    o2.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    *reinterpret_cast<uint2*>(orow) = o2;
  }
  if (p.lse && col == 0) p.lse[grow] = denom > 0.f ? (M + log2f(denom)) * kLn2 : 0.f;
}

// ----------------------------------------------------------------------------------------------
// Host side
// ----------------------------------------------------------------------------------------------

static int num_sms() {
  static PerDeviceInt cache;
  return cache.get([]() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
      cudaGetLastError();
      sms = 148;
    }
    return sms;
  }, 148);
}

static sb_status check_batch(const sb_tree_batch* tb) {
  if (!tb || tb->batch < 1 || !tb->k_cache || !tb->v_cache || !tb->prefix_len || !tb->node_offsets ||
      !tb->parent || tb->n_q_heads < 1 || tb->n_kv_heads < 1 || tb->n_q_heads % tb->n_kv_heads != 0 ||
      tb->total_nodes < 0 || tb->max_kv_len < 1)
    return SB_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(tb->k_cache) & 15) || (reinterpret_cast<uintptr_t>(tb->v_cache) & 15))
    return SB_ERR_INVALID_ARG;
  if (tb->head_dim != 64 && tb->head_dim != 128) return SB_ERR_UNSUPPORTED;
  if (tb->n_q_heads / tb->n_kv_heads > 16) return SB_ERR_UNSUPPORTED;
  if (tb->max_nodes < 1 || tb->max_nodes > SB_MAX_NODES) return SB_ERR_UNSUPPORTED;
  if (tb->page_size < 0) return SB_ERR_INVALID_ARG;
  if (tb->page_size > 0) {
    if (tb->page_size < 16 || (tb->page_size & (tb->page_size - 1))) return SB_ERR_UNSUPPORTED;
    if (!tb->page_table || tb->max_pages < 1 || tb->num_pages < 1) return SB_ERR_INVALID_ARG;
  } else if (tb->kv_capacity < 1) {
    return SB_ERR_INVALID_ARG;
  }
  return SB_OK;
}

constexpr int kMaxCluster = 8;  // portable thread-block cluster size


struct SplitPlan {
  int cluster;     // chunk-CTAs merged through distributed shared memory
  int outer;       // clusters per (sequence, KV head, row tile)
  bool two_tiles;  // the two-tiles-per-CTA tcgen05 kernel (no clusters: outer = chunks)
};

#ifdef SB_TEST_KERNELS
// How many clusters of `cluster` CTAs of the mma.sync kernel can be resident at once (0 when the
// query fails).  Cached per (head_dim, cluster size); 8-CTA clusters of full-SM CTAs do not tile
// the 148 SMs evenly, so this is what decides whether a grid runs as one wave.
static int max_active_clusters(int D, int cluster) {
  static PerDeviceInt cache[2][kMaxCluster + 1];
  const int di = D == 64 ? 0 : 1;
  return cache[di][cluster].get([&]() {
    const size_t smem = 2560 + (size_t)BM * D * 2 + 2 * (size_t)STAGES * BN * D * 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster * 64, 1, 1);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    cudaError_t e;
    if (D == 64) {
      cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveClusters(&n, attn_mma_kernel<64>, &cfg);
    } else {
      cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveClusters(&n, attn_mma_kernel<128>, &cfg);
    }
    if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
    return n;
  }, 0);
}
constexpr int kCheckGranule = BN;
#else
static int max_active_clusters(int, int) { return 0; }
constexpr int kCheckGranule = 64;
#endif

// `oversubscribed`: the grid has several waves of CTAs anyway.  Then clusters of 2 are preferred:
// clusters of 8 full-SM CTAs keep only 120 of the 148 SMs busy, clusters of 2 all of them, and the
// extra fp32 partials (one per cluster) cost less than the idle SMs (measured on the long-context
// configuration: 1072 us against 1227 us).
// The tcgen05 kernel also runs clusters of 9 and 10 (beyond the portable 8: allowed per kernel), which the
// single-wave chooser below takes when they fit -- 15 clusters of 9 or 11 of 10 full-SM CTAs on a B200.
constexpr int kMaxClusterTc = 10;
static SplitPlan plan_for(int s, bool oversubscribed, bool wide = false) {
  SplitPlan sp;
  sp.two_tiles = false;
  sp.cluster = 1;
  const int climit = wide ? kMaxClusterTc : kMaxCluster;
  int cmax = oversubscribed ? 2 : climit;
  if (const char* e = test_knob("SB_ATTN_MAX_CLUSTER")) {
    const int v = atoi(e);
    if (v >= 1 && v <= climit) cmax = v;
  }
  for (int c = cmax; c >= 1; --c)
    if (s % c == 0) { sp.cluster = c; break; }
  sp.outer = s / sp.cluster;
  return sp;
}

enum AttnImpl { IMPL_TC = 0, IMPL_MMA = 1, IMPL_SIMPLE = 2 };

// Upper bound of the 128-row query tiles any (sequence, KV head) needs: a sequence has at most
// max_nodes query nodes and never more than there are query rows in the whole batch (a drafter
// block that only queries its newest nodes stays at one tile although its tree is larger).
static int max_row_tiles(const sb_tree_batch* tb, int total_q) {
  const int G = tb->n_q_heads / tb->n_kv_heads;
  const int nq = tb->max_nodes < total_q ? tb->max_nodes : total_q;
  return ceil_div((nq > 0 ? nq : 1) * G, BM);
}

static AttnImpl attn_impl() {
  const char* impl = test_knob("SB_ATTN_IMPL");
  if (impl && strcmp(impl, "simple") == 0) return IMPL_SIMPLE;
  if (impl && strcmp(impl, "mma") == 0) return IMPL_MMA;
  return IMPL_TC;
}

// KV chunks per (sequence, KV head, row tile).  When the caller leaves the choice to us: the
// largest count whose clusters are all resident at once when the batch is small, otherwise
// chunks of a few KV blocks to even out ragged prefix lengths.  The chunks are grouped into
// clusters of the largest divisor <= 8.  `granule` is the kernel's key-block size.
static SplitPlan choose_splits(const sb_tree_batch* tb, int total_q, int num_splits, AttnImpl impl) {
  const int row_tiles = max_row_tiles(tb, total_q);
  const int granule = impl == IMPL_TC ? 128 : kCheckGranule;
  const int max_blocks = ceil_div(tb->max_kv_len, granule);
  const long long base = (long long)tb->batch * tb->n_kv_heads * row_tiles;
  const int sms = num_sms();
  // More (sequence, KV head, row tile) units than SMs and at least two row tiles per KV head: the
  // tcgen05 kernel that gives one CTA two tiles (each K/V block is pulled from L2 once for both).
  // (With three tiles the second CTA of a KV head holds a single one; still faster than three one-tile
  // CTAs on the ragged batch of config 4: 131 us against 154 us.)
  bool two_tiles = impl == IMPL_TC && row_tiles >= 2 && base > sms;
  if (const char* e = test_knob("SB_ATTN_TWO_TILES")) two_tiles = impl == IMPL_TC && row_tiles >= 2 && atoi(e) != 0;
  if (two_tiles) {
    SplitPlan sp;
    sp.two_tiles = true;
    sp.cluster = 1;
    if (num_splits > 0) {
      sp.outer = num_splits < max_blocks ? num_splits : max_blocks;
      return sp;
    }
    // CTAs run in waves; a CTA costs its blocks (two tiles each) plus a fixed start-up and epilogue
    // (about 11 us measured on the long-context configuration: nine block-times), and every chunk beyond
    // the first writes and re-reads a bf16 partial of all rows, here in units of one block-time
    // (1.2 us) at 6 TB/s.
    const long long units = (long long)tb->batch * tb->n_kv_heads * ceil_div(row_tiles, 2);
    const double partial = 2.0 * (double)total_q * tb->n_q_heads * tb->head_dim * 2.0 / 6e12 / 1.2e-6;
    int best = 1;
    double best_cost = 0.0;
    for (int s = 1; s <= 8 && s <= max_blocks; ++s) {
      const long long waves = (units * s + sms - 1) / sms;
      const double cost = (double)waves * (2 * ceil_div(max_blocks, s) + 9) + (s > 1 ? partial * s + 3.0 : 0.0);
      if (s == 1 || cost < best_cost) {
        best = s;
        best_cost = cost;
      }
    }
    sp.outer = best;
    return sp;
  }
  if (num_splits > 0) {
    const int s = num_splits < max_blocks ? num_splits : max_blocks;
    return plan_for(s, base * s > 2LL * sms);
  }
  if (base > sms) {
    if (impl != IMPL_TC) {
      int s = max_blocks / 16;
      if (s > 16) s = 16;
      if (s < 1) s = 1;
      return plan_for(s, true);
    }
    // More tiles than SMs: CTAs run in waves, and every CTA pays a fixed start-up and merge cost
    // worth about five blocks.  Take the chunk count with the fewest waves x (blocks + fixed cost).
    int best = 1;
    long long best_cost = 0;
    for (int s = 1; s <= 8 && s <= max_blocks; ++s) {
      const long long waves = (base * s + sms - 1) / sms;
      const long long cost = waves * (ceil_div(max_blocks, s) + 5 + (s > 1 ? 1 : 0));
      if (s == 1 || cost < best_cost) {
        best = s;
        best_cost = cost;
      }
    }
    return plan_for(best, true);
  }
  // Few tiles: one wave.  Among the chunk counts whose clusters are all resident at once, take the
  // cheapest under: blocks per chunk x 1.2 us, plus 6 us when the chunks of a tile do not fit one
  // cluster (fp32 partials and the merge launch) -- 33 blocks over 8 KV heads: 8 chunks in one
  // cluster of 8 (14.4 us) rather than 15 chunks in 3 clusters of 5 (22.7 us).
  int s_max = (int)(sms / base);
  if (s_max > max_blocks) s_max = max_blocks;
  SplitPlan best = plan_for(1, false);
  double best_cost = 1.2 * max_blocks;
  for (int s = 2; s <= s_max; ++s) {
    const SplitPlan sp = plan_for(s, false, impl == IMPL_TC);
    if (sp.outer > 1 && sp.cluster < 4) continue;  // partial traffic for little gain
    const int fit = impl == IMPL_TC ? attn_tc_max_active_clusters(tb->head_dim, sp.cluster)
                                    : max_active_clusters(tb->head_dim, sp.cluster);
    if (fit > 0 && base * sp.outer > fit) continue;
    const double cost = 1.2 * ceil_div(max_blocks, s) + (sp.outer > 1 ? 6.0 : 0.0);
    if (cost <= best_cost + 1e-9) {  // ties: more chunks (smaller merge slices per CTA)
      best = sp;
      best_cost = cost;
    }
  }
  return best;
}

static size_t workspace_bytes_for(const sb_tree_batch* tb, int total_q, int outer) {
  if (outer <= 1) return 0;
  const size_t rows = (size_t)total_q * tb->n_q_heads;
  const size_t o = (size_t)outer * rows * tb->head_dim * sizeof(float);
  const size_t l = (size_t)outer * rows * sizeof(float);
  return ((o + 255) & ~(size_t)255) + ((l + 255) & ~(size_t)255);
}

#ifdef SB_TEST_KERNELS
template <int D>
static sb_status launch_attn_mma(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  static PerDeviceOnce once;
  if (!once.run([]() {
        const bool ok = cudaFuncSetAttribute(attn_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)attn_mma_smem_bytes<D>()) == cudaSuccess;
        if (!ok) cudaGetLastError();
        return ok;
      }))
    return SB_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = attn_mma_smem_bytes<D>();
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (test_knob("SB_DEBUG")) {
    int max_clusters = -1;
    cudaOccupancyMaxActiveClusters(&max_clusters, attn_mma_kernel<D>, &cfg);
    fprintf(stderr, "[sb] attn_mma<%d> grid (%u,%u,%u) cluster %d outer %d: max active clusters %d\n", D, grid.x,
            grid.y, grid.z, cluster, p.outer, max_clusters);
  }
  if (cudaLaunchKernelEx(&cfg, attn_mma_kernel<D>, p) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}
#endif  // SB_TEST_KERNELS

}  // namespace sb

extern "C" size_t sb_tree_attention_workspace_bytes(const sb_tree_batch* tb, int32_t total_q,
                                                    int32_t num_splits) {
  if (sb::check_batch(tb) != SB_OK || total_q < 0 || num_splits < 0) return 0;
  return sb::workspace_bytes_for(tb, total_q, sb::choose_splits(tb, total_q, num_splits, sb::attn_impl()).outer);
}

extern "C" sb_status sb_tree_attention(const sb_tree_batch* tb, const int32_t* q_node_begin,
                                       const int32_t* q_offsets, int32_t total_q, const void* q, void* out,
                                       float* lse, float scale, int32_t num_splits, void* workspace,
                                       size_t workspace_bytes, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_tree_attention");
  using namespace sb;
  sb_status st = check_batch(tb);
  if (st != SB_OK) return st;
  if (!q || !out || !status || total_q < 1 || num_splits < 0 || !(scale >= 0.f)) return SB_ERR_INVALID_ARG;
  if (q_node_begin && !q_offsets) return SB_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 15))
    return SB_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int D = tb->head_dim;

  AttnParams p;
  p.tb = *tb;
  p.q_node_begin = q_node_begin;
  p.q_offsets = q_offsets;
  p.total_q = total_q;
  p.q = static_cast<const bf16*>(q);
  p.out = static_cast<bf16*>(out);
  p.lse = lse;
  p.scale_log2 = (scale > 0.f ? scale : 1.0f / sqrtf((float)D)) * 1.4426950408889634f;
  p.status = status;
  p.G = tb->n_q_heads / tb->n_kv_heads;
  p.part_o = nullptr;
  p.sort_seqs = 0;
  p.part_bf16 = 0;
  p.part_lse = nullptr;

  const AttnImpl impl = attn_impl();
#ifdef SB_TEST_KERNELS
  if (impl == IMPL_SIMPLE) {
    p.num_splits = 1;
    p.outer = 1;
    p.row_tiles = 1;
    dim3 grid(ceil_div(tb->max_nodes * tb->n_q_heads, 8), tb->batch);
    if (D == 64) attn_simple_kernel<64><<<grid, 256, 0, cs>>>(p);
    else attn_simple_kernel<128><<<grid, 256, 0, cs>>>(p);
    return launch_check();
  }
#endif

  const SplitPlan plan = choose_splits(tb, total_q, num_splits, impl);
  p.num_splits = plan.cluster * plan.outer;
  p.outer = plan.outer;
  if (plan.outer > 1) {
    const size_t need = workspace_bytes_for(tb, total_q, plan.outer);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255))
      return SB_ERR_WORKSPACE;
    const size_t rows = (size_t)total_q * tb->n_q_heads;
    const size_t o = ((size_t)plan.outer * rows * D * sizeof(float) + 255) & ~(size_t)255;
    p.part_o = static_cast<float*>(workspace);
    p.part_lse = reinterpret_cast<float*>(static_cast<char*>(workspace) + o);
  }
  const int row_tiles = max_row_tiles(tb, total_q);
  p.row_tiles = row_tiles;
  p.part_bf16 = plan.two_tiles ? 1 : 0;
  // ragged batches that run in waves start their longest sequences first
  p.sort_seqs = (impl == IMPL_TC && tb->batch > 1 && tb->batch <= 128 &&
                 (long long)tb->batch * tb->n_kv_heads * row_tiles > num_sms()) ? 1 : 0;
  dim3 grid(p.num_splits, (plan.two_tiles ? ceil_div(row_tiles, 2) : row_tiles) * tb->n_kv_heads, tb->batch);
  if (grid.y > 65535 || grid.z > 65535) return SB_ERR_UNSUPPORTED;
  if (plan.two_tiles) st = launch_attn_tc2(p, grid, cs);
  else if (impl == IMPL_TC) st = launch_attn_tc(p, grid, plan.cluster, cs);
#ifdef SB_TEST_KERNELS
  else st = D == 64 ? launch_attn_mma<64>(p, grid, plan.cluster, cs) : launch_attn_mma<128>(p, grid, plan.cluster, cs);
#else
  else st = SB_ERR_UNSUPPORTED;
#endif
  if (st != SB_OK || plan.outer == 1) return st;
  const int rows_max = tb->max_nodes * tb->n_q_heads;
  auto mgrid = [&](int rows_per_cta) { return dim3(ceil_div(rows_max, rows_per_cta), tb->batch); };
  if (p.part_bf16) {
    if (D == 64) attn_merge_kernel<64, true><<<mgrid(merge_rows_per_cta<64, true>()), 256, 0, cs>>>(p);
    else attn_merge_kernel<128, true><<<mgrid(merge_rows_per_cta<128, true>()), 256, 0, cs>>>(p);
  } else {
    if (D == 64) attn_merge_kernel<64, false><<<mgrid(merge_rows_per_cta<64, false>()), 256, 0, cs>>>(p);
    else attn_merge_kernel<128, false><<<mgrid(merge_rows_per_cta<128, false>()), 256, 0, cs>>>(p);
  }
  return launch_check();
}
