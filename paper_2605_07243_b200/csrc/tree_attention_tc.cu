// Tree-masked split-KV attention on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// One CTA owns a 128-row query tile (rows = (node, head-in-group) pairs of one KV head: the tile
// is the M = 128 dimension of the MMA and one row per TMEM lane) and a chunk of the sequence's
// keys, walked in blocks of up to 128 keys:
//
//   loader warps   (2 for K and the Q tile, 1 for V) K and V blocks -> shared memory in the 128-byte-swizzled layouts the
//                  tensor core reads (K, Q, P: K-major; V: MN-major), 16-byte cp.async, 2 stages each;
//   MMA warp       one thread issues  S_j = Q K_j^T  (tcgen05.mma, fp32 accumulator in TMEM, two S
//                  buffers so S_{j+1} runs under the softmax of block j) and  PV_j = P_j V_j;
//   softmax warps  4 warps, thread t owns row t: reads its S row from TMEM (tcgen05.ld), applies the
//                  softmax scale and the tree mask (one 128-bit ancestor set per row, turned into
//                  two 64-bit visibility windows per block; prefix-only blocks skip it), keeps the
//                  running max / sum, writes P_j as bf16 into shared memory for the PV product and
//                  folds PV_{j-1} from TMEM into its fp32 output row held in registers.
//
// All hand-offs are mbarriers (tcgen05.commit on the MMA side); every wait is bounded and reports
// SB_ERR_CUDA instead of spinning forever.  The chunk results of the CTAs of a cluster are merged
// through distributed shared memory exactly as in the mma.sync kernel.
#include <cstdio>
#include <cstdlib>

#include "attention_common.cuh"

namespace sb {

constexpr int TC_BM = 128;           // rows per CTA
constexpr int TC_BN = 128;           // keys per block
constexpr int TC_SOFTMAX_THREADS = 128;
constexpr int TC_MMA_WARP = 4;
constexpr int TC_KLOAD_THREAD0 = 160;  // warps 5,6: K blocks and the Q tile
constexpr int TC_VLOAD_THREAD0 = 224;  // warp 7: V blocks
constexpr int TC_KLOADERS = 64;
constexpr int TC_VLOADERS = 32;
constexpr int TC_THREADS = 256;        // 8 warps = 2 per scheduler: up to 255 registers per thread
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_SMALL_BYTES = 4096;   // ancestor masks, parents, barriers

enum TcBar { K_FULL0, K_FULL1, K_EMPTY0, K_EMPTY1, V_FULL0, V_FULL1, V_EMPTY0, V_EMPTY1, S_FULL0, S_FULL1,
             S_EMPTY0, S_EMPTY1, P_FULL, PV_FULL, PV_EMPTY, TC_NUM_BARS };

template <int D>
constexpr size_t attn_tc_smem_bytes() {
  // small region + Q + 2 K stages + 2 V stages + P, plus slack to align the tiles to 1024 bytes
  return 1024 + TC_SMALL_BYTES + (size_t)TC_BM * D * 2 + 4 * (size_t)TC_BN * D * 2 + (size_t)TC_BM * TC_BN * 2;
}

__device__ inline uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ inline void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait: gives up after two seconds of wall time, or as soon as another thread of the CTA
// has given up, and returns false; the caller then skips its remaining work and the kernel ends.
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t addr = smem_u32(bar);
  unsigned long long t0 = 0;
  for (int it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((it & 63) == 63) {
      if (*abort_flag) return false;
      unsigned long long now;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > 2000000000ull) break;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ inline void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, issued by one thread.
__device__ inline void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1, layout type 2.
__device__ inline uint64_t tc_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, N>>3 at bit 17, M>>4 at bit 24,
// bit 16 = B is MN-major.
__device__ inline uint32_t tc_idesc(int M, int N, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ inline void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ inline void cp_async_16_tc(uint32_t smem_dst, const void* gmem_src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_dst), "l"(gmem_src), "r"(src_bytes));
}

// Byte offset of 16-byte chunk `ch` of row `r` inside a [rows][D] bf16 tile stored as D/64
// column halves of [rows][128 B] with the 128-byte XOR swizzle.
__device__ inline uint32_t sw128_chunk_off(int r, int ch, int rows) {
  return (uint32_t)((ch >> 3) * rows * 128 + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const AttnParams p) {
  constexpr int CH = D / 8;                   // 16-byte chunks per row
  constexpr int TILE_BYTES = TC_BN * D * 2;   // one K or V stage
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint32_t* s_anc = reinterpret_cast<uint32_t*>(base);               // 2048 B
  int* s_parent = reinterpret_cast<int*>(base + 2048);               // 512 B
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(base + 2560);        // TC_NUM_BARS * 8
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(base + 2560 + 256);
  volatile int* s_abort = reinterpret_cast<volatile int*>(base + 2560 + 260);
  uint8_t* sQ = base + TC_SMALL_BYTES;
  uint8_t* sK = sQ + TC_BM * D * 2;
  uint8_t* sV = sK + 2 * TILE_BYTES;
  uint8_t* sP = sV + 2 * TILE_BYTES;

  const int tid = threadIdx.x, warp = tid >> 5;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int split = blockIdx.x;
  const int Hkv = p.tb.n_kv_heads, Hq = p.tb.n_q_heads, G = p.G;
  const int g = blockIdx.y % Hkv, tile = blockIdx.y / Hkv;
  const int b = blockIdx.z;

  if (tid == 0) *s_abort = 0;
  const SeqPlan sp = plan_sequence(p, b, split == 0 && blockIdx.y == 0, s_parent, s_anc);
  const SeqInfo& si = sp.info;
  const int rows_total = si.nq * G;
  const int row0 = tile * TC_BM;
  if (!sp.can_write || row0 >= rows_total) return;  // uniform over the cluster
  const long long rows_all = (long long)p.total_q * Hq;

  // Balanced cut of the sequence's keys, in units of 16, into num_splits chunks.
  const int L = si.P + si.n;
  const int units = ceil_div(L, 16);
  const int u_base = units / p.num_splits, u_rem = units % p.num_splits;
  const int key_begin = 16 * (split * u_base + min(split, u_rem));
  const int chunk_keys = sp.compute ? 16 * (u_base + (split < u_rem ? 1 : 0)) : 0;
  const int nb = ceil_div(chunk_keys, TC_BN);

  if (tid == 0) {
    const int counts[TC_NUM_BARS] = {TC_KLOADERS, TC_KLOADERS, 1, 1, TC_VLOADERS, TC_VLOADERS, 1, 1, 1, 1,
                                     TC_SOFTMAX_THREADS, TC_SOFTMAX_THREADS, TC_SOFTMAX_THREADS, 1, TC_SOFTMAX_THREADS};
    for (int i = 0; i < TC_NUM_BARS; ++i) mbar_init(&s_bar[i], counts[i]);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == TC_MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TC_TMEM_COLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t tmem_pv = tmem + 2 * TC_BN;  // S buffers at columns [0,128) and [128,256), PV after them

  // Row state of the softmax threads (thread t <-> row t <-> TMEM lane t).
  float o_row[D];
  float m_run = -INFINITY, l_run = 0.f;
#pragma unroll
  for (int d = 0; d < D; ++d) o_row[d] = 0.f;

  if (tid < TC_SOFTMAX_THREADS) {
    // ------------------------------------------------------------------ softmax warps
    const int R = row0 + tid;
    const bool row_live = R < rows_total && sp.compute;
    uint32_t anc[4];
    {
      const int node = row_live ? si.q0 + R / G : 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) anc[w] = row_live ? s_anc[4 * node + w] : 0u;
    }
    const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
    float corr_prev = 1.f;  // rescale of o_row that belongs to the PV block still in flight
    bool ok = true;
    for (int j = 0; j < nb && ok; ++j) {
      const int k0 = key_begin + j * TC_BN;
      const int nj = min(TC_BN, chunk_keys - j * TC_BN);  // keys of this block (multiple of 16)
      ok = mbar_wait(&s_bar[S_FULL0 + (j & 1)], (j >> 1) & 1, s_abort);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = tmem + lane_base + (j & 1) * TC_BN;
      // visibility of columns [0,64) and [64,128): tree mask where the block reaches past the
      // prefix, and only the block's own nj columns
      uint64_t win[2];
      const bool need_mask = k0 + TC_BN > si.P;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint64_t w = need_mask ? visibility_window(anc, k0 + 64 * h - si.P) : ~0ull;
        const int cols = nj - 64 * h;
        w &= cols >= 64 ? ~0ull : (cols <= 0 ? 0ull : ((1ull << cols) - 1ull));
        win[h] = w;
      }
      // pass 1: row maximum
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < TC_BN / 32; ++c) {
        if (c * 32 < nj) {
          uint32_t r[32];
          tmem_ld32(t_s + c * 32, r);
          const uint32_t m32 = (uint32_t)(win[c >> 1] >> ((c & 1) * 32));
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, ((m32 >> i) & 1u) ? __uint_as_float(r[i]) : -INFINITY);
        }
      }
      mx *= p.scale_log2;  // scale > 0: max commutes with it (-inf stays -inf)
      const float m_new = fmaxf(m_run, mx);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      const float corr = fast_exp2(m_run - m_use);
      // fold the previous block's PV into the output row (also frees P and the PV accumulator)
      if (j > 0) {
        ok = mbar_wait(&s_bar[PV_FULL], (j - 1) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_pv + lane_base + c * 32, r);
#pragma unroll
          for (int i = 0; i < 32; ++i) o_row[c * 32 + i] = o_row[c * 32 + i] * corr_prev + __uint_as_float(r[i]);
        }
        tc_fence_before();
        mbar_arrive(&s_bar[PV_EMPTY]);
      }
      // pass 2: probabilities -> P (bf16, K-major swizzled), running sum
      float lsum = 0.f;
#pragma unroll
      for (int c = 0; c < TC_BN / 32; ++c) {
        if (c * 32 < nj) {
          uint32_t r[32];
          tmem_ld32(t_s + c * 32, r);
          const uint32_t m32 = (uint32_t)(win[c >> 1] >> ((c & 1) * 32));
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float s0 = ((m32 >> i) & 1u) ? __uint_as_float(r[i]) * p.scale_log2 - m_use : -INFINITY;
            const float s1 = ((m32 >> (i + 1)) & 1u) ? __uint_as_float(r[i + 1]) * p.scale_log2 - m_use : -INFINITY;
            const float p0 = fast_exp2(s0), p1 = fast_exp2(s1);
            lsum += p0 + p1;
            packed[i >> 1] = pack_bf16(p0, p1);
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int ch = c * 4 + q;  // 16-byte chunk (8 keys) of this row
            *reinterpret_cast<uint4*>(sP + sw128_chunk_off(tid, ch, TC_BM)) =
                make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
          }
        }
      }
      l_run = l_run * corr + lsum;
      m_run = m_new;
      corr_prev = corr;
      tc_fence_before();
      mbar_arrive(&s_bar[S_EMPTY0 + (j & 1)]);
      fence_async_smem();
      mbar_arrive(&s_bar[P_FULL]);
    }
    if (ok && nb > 0) {
      ok = mbar_wait(&s_bar[PV_FULL], (nb - 1) & 1, s_abort);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_pv + lane_base + c * 32, r);
#pragma unroll
          for (int i = 0; i < 32; ++i) o_row[c * 32 + i] = o_row[c * 32 + i] * corr_prev + __uint_as_float(r[i]);
        }
      }
    }
    if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
  } else if (warp == TC_MMA_WARP) {
    // ------------------------------------------------------------------ MMA issuer
    if ((tid & 31) == 0 && nb > 0) {
      const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV), p_addr = smem_u32(sP);
      bool ok = true;
      auto issue_s = [&](int j) {
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t idesc = tc_idesc(TC_BM, nj, 0);
        const uint32_t kb = k_addr + (j & 1) * TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t koff = (ks >> 2) * (TC_BM * 128) + (ks & 3) * 32;
          tc_mma(tmem + (j & 1) * TC_BN, tc_smem_desc(q_addr + koff, 16, 1024), tc_smem_desc(kb + koff, 16, 1024), idesc,
                 ks > 0);
        }
        tc_commit(&s_bar[S_FULL0 + (j & 1)]);
        tc_commit(&s_bar[K_EMPTY0 + (j & 1)]);
      };
      ok = mbar_wait(&s_bar[K_FULL0], 0, s_abort);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; j < nb && ok; ++j) {
        if (j + 1 < nb) {
          const int jn = j + 1;
          ok = mbar_wait(&s_bar[K_FULL0 + (jn & 1)], (jn >> 1) & 1, s_abort);
          if (ok && jn >= 2) ok = mbar_wait(&s_bar[S_EMPTY0 + (jn & 1)], ((jn >> 1) - 1) & 1, s_abort);
          if (!ok) break;
          tc_fence_after();
          issue_s(jn);
        }
        ok = mbar_wait(&s_bar[P_FULL], j & 1, s_abort);
        if (ok) ok = mbar_wait(&s_bar[V_FULL0 + (j & 1)], (j >> 1) & 1, s_abort);
        if (ok && j > 0) ok = mbar_wait(&s_bar[PV_EMPTY], (j - 1) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t idesc = tc_idesc(TC_BM, D, 1);
        const uint32_t vb = v_addr + (j & 1) * TILE_BYTES;
        for (int ks = 0; ks < nj / 16; ++ks) {
          const uint32_t aoff = (ks >> 2) * (TC_BM * 128) + (ks & 3) * 32;
          tc_mma(tmem_pv, tc_smem_desc(p_addr + aoff, 16, 1024), tc_smem_desc(vb + ks * 2048, TC_BN * 128, 1024), idesc,
                 ks > 0);
        }
        tc_commit(&s_bar[PV_FULL]);
        tc_commit(&s_bar[V_EMPTY0 + (j & 1)]);
      }
      if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
    }
  } else {
    // ------------------------------------------------------------------ loader warps
    const bool is_k = tid < TC_VLOAD_THREAD0;
    const int lt = tid - (is_k ? TC_KLOAD_THREAD0 : TC_VLOAD_THREAD0);
    const int n_loaders = is_k ? TC_KLOADERS : TC_VLOADERS;
    const bf16* src = static_cast<const bf16*>(is_k ? p.tb.k_cache : p.tb.v_cache) + (long long)g * D;
    const uint32_t dst0 = smem_u32(is_k ? sK : sV);
    auto issue_block = [&](int j) {
      const int nj = min(TC_BN, chunk_keys - j * TC_BN);
      const int k0 = key_begin + j * TC_BN;
      const uint32_t dst = dst0 + (j & 1) * TILE_BYTES;
      for (int c = lt; c < nj * CH; c += n_loaders) {
        const int r = c / CH, ch = c % CH;
        const int key = k0 + r;
        const bool valid = key < L;  // keys past the sequence inside the last unit of 16: zeros
        const long long off = valid ? kv_row_elem_offset(p.tb, b, key) + ch * 8 : 0;
        cp_async_16_tc(dst + sw128_chunk_off(r, ch, TC_BN), src + off, valid ? 16 : 0);
      }
    };
    if (nb > 0) {
      if (is_k) {
        // the query tile travels with the first K block
        const uint32_t qd = smem_u32(sQ);
        for (int c = lt; c < TC_BM * CH; c += n_loaders) {
          const int r = c / CH, ch = c % CH;
          const int R = row0 + r;
          const bool valid = R < rows_total;
          const int node_l = valid ? R / G : 0;
          const int hh = valid ? R - node_l * G : 0;
          const long long off = ((long long)(si.q_off + node_l) * Hq + g * G + hh) * D + ch * 8;
          cp_async_16_tc(qd + sw128_chunk_off(r, ch, TC_BM), p.q + (valid ? off : 0), valid ? 16 : 0);
        }
      }
      issue_block(0);
      asm volatile("cp.async.commit_group;\n" ::);
      if (nb > 1) {
        issue_block(1);
        asm volatile("cp.async.commit_group;\n" ::);
      }
      bool ok = true;
      uint64_t* full = &s_bar[is_k ? K_FULL0 : V_FULL0];
      uint64_t* empty = &s_bar[is_k ? K_EMPTY0 : V_EMPTY0];
      for (int j = 0; j < nb; ++j) {
        if (j + 1 < nb) asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        else asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        fence_async_smem();
        mbar_arrive(&full[j & 1]);
        if (j + 2 < nb) {
          ok = mbar_wait(&empty[j & 1], (j >> 1) & 1, s_abort);
          if (!ok) break;
          issue_block(j + 2);
          asm volatile("cp.async.commit_group;\n" ::);
        }
      }
      asm volatile("cp.async.wait_group 0;\n" ::: "memory");
      if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
    }
  }

  // ---- park (O, m, l) of this chunk, merge over the cluster, store ----------------------------
  constexpr int RS = D + 8;
  float* s_red = reinterpret_cast<float*>(sK);  // the K/V stages are idle once the last PV is folded
  float* s_m = s_red + TC_BM * RS;
  float* s_l = s_m + TC_BM;
  float* s_w = s_l + TC_BM;
  float* s_lse = s_w + TC_BM + 8;
  tc_fence_before();
  __syncthreads();  // every role is done: no async read of the stages is in flight any more
  if (tid < TC_SOFTMAX_THREADS) {
    if (nb > 0) {
#pragma unroll
      for (int d = 0; d < D; d += 4)
        *reinterpret_cast<float4*>(s_red + tid * RS + d) = make_float4(o_row[d], o_row[d + 1], o_row[d + 2], o_row[d + 3]);
    }
    s_m[tid] = m_run;
    s_l[tid] = l_run;
  }
  if (S > 1) cluster.sync(); else __syncthreads();
  if (warp == TC_MMA_WARP) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS));
  }
  cluster_merge_and_store<D, TC_BM>(p, cluster, S, crank, s_red, s_m, s_l, s_w, s_lse, split / S, row0, rows_total, g,
                                    si.q_off, rows_all, tid, TC_THREADS);
  if (S > 1) cluster.sync();
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------

template <int D>
static cudaLaunchConfig_t tc_config(dim3 grid, int cluster, cudaStream_t cs, cudaLaunchAttribute* attr) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = attn_tc_smem_bytes<D>();
  cfg.stream = cs;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cfg;
}

template <int D>
static bool tc_prepare() {
  static bool done = false;
  if (!done) {
    if (cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_tc_smem_bytes<D>()) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    done = true;
  }
  return true;
}

int attn_tc_max_active_clusters(int D, int cluster) {
  static int cache[2][9];
  static bool have[2][9];
  const int di = D == 64 ? 0 : 1;
  if (cluster < 1 || cluster > 8) return 0;
  if (!have[di][cluster]) {
    int n = 0;
    cudaLaunchAttribute attr[1];
    cudaError_t e = cudaErrorUnknown;
    if (D == 64 && tc_prepare<64>()) {
      cudaLaunchConfig_t cfg = tc_config<64>(dim3(cluster * 64, 1, 1), cluster, nullptr, attr);
      e = cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<64>, &cfg);
    } else if (D == 128 && tc_prepare<128>()) {
      cudaLaunchConfig_t cfg = tc_config<128>(dim3(cluster * 64, 1, 1), cluster, nullptr, attr);
      e = cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<128>, &cfg);
    }
    if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
    cache[di][cluster] = n;
    have[di][cluster] = true;
  }
  return cache[di][cluster];
}

template <int D>
static sb_status launch_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  if (!tc_prepare<D>()) return SB_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = tc_config<D>(grid, cluster, cs, attr);
  if (getenv("SB_DEBUG"))
    fprintf(stderr, "[sb] attn_tc<%d> grid (%u,%u,%u) cluster %d outer %d: max active clusters %d\n", D, grid.x, grid.y,
            grid.z, cluster, p.outer, attn_tc_max_active_clusters(D, cluster));
  if (cudaLaunchKernelEx(&cfg, attn_tc_kernel<D>, p) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

sb_status launch_attn_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  return p.tb.head_dim == 64 ? launch_tc<64>(p, grid, cluster, cs) : launch_tc<128>(p, grid, cluster, cs);
}

}  // namespace sb
