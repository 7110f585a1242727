// Tree-masked split-KV attention, two query tiles per CTA (tcgen05 + TMEM + TMA, sm_100a).
//
// The throughput variant of attn_tc_kernel, used when the (sequence, KV head, row tile) units
// outnumber the SMs and a KV head has at least two 128-row tiles (large trees, wide GQA groups).
// There every K/V byte a CTA pulls from L2 is worth one 128-row tile of work, and the shared-memory
// stages (two K, two V) cover less than the load latency.  Here a CTA owns TWO row tiles of the same
// KV head and walks the chunk once: each K/V block serves both tiles, which halves the bytes
// per unit of softmax work and doubles the time a stage has to arrive.
//
// The blocks are processed as "virtual blocks" v = 2 j + t (key block j, tile t):
//   S_v = Q_t K_j^T goes to score buffer v & 1 in tensor memory, so the two tiles alternate
//   buffers; the softmax warps turn it into P_v IN PLACE (packed bf16 over the first half of each
//   thread's score columns), and O_t += P_v V_j accumulates in the tile's own accumulator:
//   tensor memory = 2 score buffers (256 columns) + 2 accumulators (2 D columns).
//   The MMA thread issues S_0, S_1, then PV_v followed by S_{v+2}: the tensor pipe runs its MMAs in
//   order, so S_{v+2} overwrites P_v only after PV_v has read it, and S_{v+1} (the other tile) is
//   computed while the softmax warps work on v.
// Everything else (TMA loaders, visibility windows, lazy reference maximum, bounded waits) is as in
// attn_tc_kernel.  CTAs are not clustered: with more than one KV chunk every CTA writes a bf16
// partial (its rows are rounded to bf16 when they are staged anyway) and attn_merge_kernel merges them.
#include <cstdio>
#include <cstdlib>

#include "tc_common.cuh"

namespace sb {

constexpr int T2_SOFTMAX_THREADS = 256;  // warps 0-3: columns [0,64) of a block, warps 4-7: [64,128)
constexpr int T2_MMA_WARP = 8;
constexpr int T2_KLOAD_WARP = 9;   // lane 0 issues the Q and K loads
constexpr int T2_VLOAD_WARP = 10;  // lane 0 issues the V loads; the warp zeroes rows past the sequence
constexpr int T2_THREADS = 384;
constexpr int T2_TMEM_COLS = 512;
constexpr int T2_SMALL_BYTES = 8192;  // ancestor masks, parents, barriers, softmax exchange

enum T2Bar { K_FULL0, K_FULL1, K_EMPTY0, K_EMPTY1, V_FULL0, V_FULL1, V_EMPTY0, V_EMPTY1, S_FULL0, S_FULL1,
             P_FULL0, P_FULL1, PV_FULL, O_DONE, V_TMA0, V_TMA1, Q_FULL, T2_NUM_BARS };

template <int D>
constexpr size_t attn_tc2_smem_bytes() {
  // small region + 2 Q tiles + 2 K stages + 2 V stages, plus slack to align the tiles to 1024 bytes
  return 1024 + T2_SMALL_BYTES + 2 * (size_t)TC_BM * D * 2 + 4 * (size_t)TC_BN * D * 2;
}

template <int D>
__global__ void __launch_bounds__(T2_THREADS, 1) attn_tc2_kernel(const AttnParams p,
                                                                 const __grid_constant__ CUtensorMap kmap,
                                                                 const __grid_constant__ CUtensorMap vmap,
                                                                 const __grid_constant__ CUtensorMap qmap,
                                                                 const int box_rows, const int q_tma) {
  constexpr int CH = D / 8;                   // 16-byte chunks per row
  constexpr int TILE_BYTES = TC_BN * D * 2;   // one K or V stage
  constexpr int QT_BYTES = TC_BM * D * 2;     // one Q tile
  constexpr int DH = D / 2;                   // output columns per softmax thread
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint32_t* s_anc = reinterpret_cast<uint32_t*>(base);               // 2048 B
  int* s_parent = reinterpret_cast<int*>(base + 2048);               // 512 B
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(base + 2560);        // T2_NUM_BARS * 8
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(base + 2816);
  volatile int* s_abort = reinterpret_cast<volatile int*>(base + 2820);
  float* s_xmax = reinterpret_cast<float*>(base + 3072);             // [2 parities][2 halves][128 rows]
  float* s_xl = reinterpret_cast<float*>(base + 5120);               // [2 tiles][2 halves][128 rows]
  uint8_t* sQ = base + T2_SMALL_BYTES;                               // [2 tiles]
  uint8_t* sK = sQ + 2 * QT_BYTES;
  uint8_t* sV = sK + 2 * TILE_BYTES;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x;
  const int Hq = p.tb.n_q_heads, G = p.G;
  // the tile pairs of one (sequence, KV head) are neighbours in launch order: they share its K/V through L2
  const int pairs = ceil_div(p.row_tiles, 2);
  const int g = blockIdx.y / pairs, pair = blockIdx.y % pairs;
  if (tid == 0) {
    *s_abort = 0;
    const int n = T2_SOFTMAX_THREADS;
    const int counts[T2_NUM_BARS] = {1, 1, 1, 1, 1, 1, 1, 1, 1, 1, n, n, 1, 1, 1, 1, q_tma ? 1 : n};
    for (int i = 0; i < T2_NUM_BARS; ++i) mbar_init(&s_bar[i], counts[i]);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == T2_MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(T2_TMEM_COLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Programmatic dependent launch: everything above is independent of earlier kernels' results.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // grid index z -> sequence (longest first when the grid runs in several waves)
  const int b = p.sort_seqs ? sequence_of_rank(p.tb, blockIdx.z, reinterpret_cast<int*>(s_anc), s_parent) : (int)blockIdx.z;
  const SeqPre pre = plan_lengths(p, b);
  const int rows_total = pre.info.nq * G;
  const int row0 = pair * 2 * TC_BM;                         // first row of tile 0; tile 1 starts 128 rows on
  if (!pre.can_write || row0 >= rows_total) {
    // the designated CTA always owns rows unless the sequence has none; its status is still due
    if (split == 0 && blockIdx.y == 0 && tid == 0) p.status[b] = pre.info.err;
    if (warp == T2_MMA_WARP)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*s_tmem), "r"(T2_TMEM_COLS));
    return;
  }
  const int ntile = row0 + TC_BM < rows_total ? 2 : 1;       // a sequence's last pair may hold one tile
  const long long rows_all = (long long)p.total_q * Hq;

  // Balanced cut of the sequence's 128-key blocks into num_splits chunks (block-aligned, so a
  // TMA box never straddles a page); the sequence's last block is trimmed to a multiple of 16 keys.
  const int L = pre.info.P + pre.info.n;
  const int blocks_total = ceil_div(L, TC_BN);
  const int b_base = blocks_total / p.num_splits, b_rem = blocks_total % p.num_splits;
  const int key_begin = TC_BN * (split * b_base + min(split, b_rem));
  const int nb = pre.info.err == 0 ? b_base + (split < b_rem ? 1 : 0) : 0;
  const int chunk_keys = nb == 0 ? 0 : min(nb * TC_BN, ceil_div(L - key_begin, 16) * 16);
  const int nv = nb * ntile;                                 // virtual blocks: v = j * ntile + t

  const uint32_t tmem = *s_tmem;
  const uint32_t tmem_o = tmem + 2 * TC_BN;                  // accumulator of tile t at tmem_o + t * D

  // One TMA box per page piece of a block: box_rows keys x 64 columns, per 64-column half.  The
  // page ids of a block are looked up separately (page sizes are powers of two >= 16: at most 8
  // pieces), so that a loader can have them before the stage it waits for is free.
  constexpr int MAX_PIECES = TC_BN / 16;
  auto lookup_pages = [&](int j, int (&pg)[MAX_PIECES]) {
    if (p.tb.page_size == 0) return;
    const int nj = min(TC_BN, chunk_keys - j * TC_BN);
    const int k0 = key_begin + j * TC_BN;
    const int pieces = ceil_div(nj, box_rows);
#pragma unroll 1
    for (int i = 0; i < MAX_PIECES; ++i)
      if (i < pieces) {
        const int lp = (k0 + i * box_rows) / p.tb.page_size;
        pg[i] = SB_CHECKED_ACCESS(lp, p.tb.max_pages, &p.status[b]) ? p.tb.page_table[(long long)b * p.tb.max_pages + lp] : 0;
      }
  };
  auto issue_pieces = [&](int j, const int (&pg)[MAX_PIECES], const CUtensorMap* map, uint32_t stage_addr,
                          uint64_t* bar) {
    const int nj = min(TC_BN, chunk_keys - j * TC_BN);
    const int k0 = key_begin + j * TC_BN;
    const int pieces = ceil_div(nj, box_rows);
    mbar_expect_tx(bar, (uint32_t)(pieces * box_rows * D * 2));
#pragma unroll 1
    for (int i = 0; i < MAX_PIECES; ++i) {
      if (i >= pieces) break;
      const int key = k0 + i * box_rows;
      int c2 = key, c3 = b;
      if (p.tb.page_size != 0) {
        int page = pg[i];
        if (page < 0 || page >= p.tb.num_pages) page = 0;  // reported by the designated CTA
        c2 = key & (p.tb.page_size - 1);
        c3 = page;
      }
#pragma unroll
      for (int h = 0; h < D / 64; ++h)
        tma_load_4d(stage_addr + h * (TC_BN * 128) + i * box_rows * 128, map, h * 64, g, c2, c3, bar);
    }
  };
  auto issue_block = [&](int j, const CUtensorMap* map, uint32_t stage_addr, uint64_t* bar) {
    int pg[MAX_PIECES];
    lookup_pages(j, pg);
    issue_pieces(j, pg, map, stage_addr, bar);
  };
  // Only the sequence's last V block can hold rows past its end (stale cache rows that meet zero
  // probabilities but must not be NaN or infinite): it lands on a barrier of its own and is cleaned
  // before the MMA may read it.  Every other V block completes the barrier the MMA warp waits on.
  auto v_needs_fix = [&](int j) { return L - (key_begin + j * TC_BN) < min(TC_BN, chunk_keys - j * TC_BN); };
  auto v_bar = [&](int j) { return &s_bar[(v_needs_fix(j) ? V_TMA0 : V_FULL0) + (j & 1)]; };

  // The first loads go out before anything else: they only need the sequence's lengths.
  if (nb > 0 && lane == 0 && warp == T2_KLOAD_WARP) {
    if (q_tma) {
      mbar_expect_tx(&s_bar[Q_FULL], (uint32_t)(ntile * QT_BYTES));
      for (int t = 0; t < ntile; ++t)
#pragma unroll
        for (int h = 0; h < D / 64; ++h)
          tma_load_3d(smem_u32(sQ) + t * QT_BYTES + h * (TC_BM * 128), &qmap, h * 64, g * G,
                      pre.info.q_off + (pair * 2 + t) * (TC_BM / G), &s_bar[Q_FULL]);
    }
    issue_block(0, &kmap, smem_u32(sK), &s_bar[K_FULL0]);
    if (nb > 1) issue_block(1, &kmap, smem_u32(sK) + TILE_BYTES, &s_bar[K_FULL1]);
  }

  // Only the softmax threads need the tree (ancestor sets, validity): they plan it among themselves
  // while the loaders look up pages and the first S = Q K^T is issued from the lengths alone.
  SeqPlan sp;
  sp.info = pre.info;
  sp.can_write = pre.can_write;
  sp.compute = false;
  const SeqInfo& si = pre.info;

  // Row state of the softmax threads, one set per tile: row = TMEM lane, `half` selects the 64
  // columns of every block and the half of the output row this thread owns.
  constexpr float kRescaleStep = 8.f;  // m_ref follows the row maximum in steps of at least 2^8
  float m_t[2] = {-INFINITY, -INFINITY}, l_t[2] = {0.f, 0.f};  // indexed by constants only
  const int half = (warp >> 2) & 1;
  const int row = (warp & 3) * 32 + lane;
  const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;

  bool softmax_ok = true;
  if (tid < T2_SOFTMAX_THREADS) {
    // ------------------------------------------------------------------ softmax warps
    if (!q_tma && nb > 0) {  // Q tiles as a gather of (node, head) rows
      const uint32_t qd = smem_u32(sQ);
      for (int c = tid; c < ntile * TC_BM * CH; c += T2_SOFTMAX_THREADS) {
        const int r = c / CH, ch = c % CH;   // r in [0, 256): tile r / 128
        const int R = row0 + r;
        const bool valid = R < rows_total;
        const int node_l = valid ? R / G : 0;
        const int hh = valid ? R - node_l * G : 0;
        const long long off = ((long long)(si.q_off + node_l) * Hq + g * G + hh) * D + ch * 8;
        const bool q_ok = valid && SB_CHECKED_ACCESS(off + 7, (long long)p.total_q * Hq * D, &p.status[b]);
        cp_async_16_tc(qd + (r / TC_BM) * QT_BYTES + sw128_chunk_off(r % TC_BM, ch, TC_BM), p.q + (q_ok ? off : 0),
                       q_ok ? 16 : 0);
      }
      asm volatile("cp.async.commit_group;\n" ::);
    }
    sp = plan_tree(p, b, split == 0 && blockIdx.y == 0, pre, s_parent, s_anc, first_threads(T2_SOFTMAX_THREADS));
    if (!q_tma && nb > 0) {
      asm volatile("cp.async.wait_group 0;\n" ::: "memory");
      fence_async_smem();
      mbar_arrive(&s_bar[Q_FULL]);
    }
    // node (index into the ancestor table) of this thread's row in each tile; -1 = no such row
    int node_of[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int R = row0 + t * TC_BM + row;
      node_of[t] = (R < rows_total && sp.compute) ? si.q0 + R / G : -1;
    }
    bool ok = true;
    for (int v = 0; v < nv; ++v) {
      const int j = ntile == 2 ? v >> 1 : v, t = ntile == 2 ? (v & 1) : 0;
      const int k0 = key_begin + j * TC_BN;
      const int nj = min(TC_BN, chunk_keys - j * TC_BN);  // keys of this block (multiple of 16)
      const int my_cols = nj - 64 * half;                 // valid columns among this thread's 64
      // S_v complete also means that every MMA issued before it is: PV_{v-2} is among them, which
      // read the buffer this block's probabilities go to and (with two tiles) last updated this
      // tile's accumulator.
      if (ok) ok = mbar_wait(&s_bar[S_FULL0 + (v & 1)], (v >> 1) & 1, s_abort);
      tc_fence_after();
      uint32_t sr[64];
      const uint32_t s_addr = tmem + lane_base + (v & 1) * TC_BN + 64 * half;
      tmem_ld64(s_addr, sr);
      // visibility of this thread's 64 columns: tree mask where the block reaches past the prefix,
      // and only the block's own nj columns
      uint64_t win = ~0ull;
      if (k0 + TC_BN > si.P) {
        const int node = t == 0 ? node_of[0] : node_of[1];
        uint32_t anc[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) anc[w] = node >= 0 ? s_anc[4 * node + w] : 0u;
        win = visibility_window(anc, k0 + 64 * half - si.P);
      }
      win &= my_cols >= 64 ? ~0ull : (my_cols <= 0 ? 0ull : ((1ull << my_cols) - 1ull));
      if (win != ~0ull) {  // only blocks that touch the tree or the end of the chunk have masked columns
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (!((win >> i) & 1ull)) sr[i] = 0xff800000u;  // -inf
      }
      // row maximum of the raw scores (the softmax scale is positive: it commutes with max)
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 2) mx = max3(mx, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
      mx *= p.scale_log2;
      s_xmax[((v & 1) * 2 + half) * TC_BM + row] = mx;
      softmax_group_sync();
      mx = fmaxf(mx, s_xmax[((v & 1) * 2 + (half ^ 1)) * TC_BM + row]);
      float m_ref = t == 0 ? m_t[0] : m_t[1];
      float l_run = t == 0 ? l_t[0] : l_t[1];
      // lazy reference maximum: both threads of a row take the same decision
      const bool step = mx > m_ref + kRescaleStep || (m_ref == -INFINITY && mx > -INFINITY);
      if (__any_sync(0xffffffffu, step)) {
        const float factor = (step && m_ref != -INFINITY) ? fast_exp2(m_ref - mx) : 1.f;
        if (j > 0) {  // O_t holds blocks 0..j-1: rescale this thread's half-row in tensor memory
          // with two tiles its last update, PV_{v-2}, is complete (see above); with one tile it is
          // PV_{v-1}, whose P this thread delivered: the barrier is in that phase or the next
          if (ntile == 1) {
            if (ok) ok = mbar_wait(&s_bar[PV_FULL], (v - 1) & 1, s_abort);
            tc_fence_after();
          }
          // (rare, and 16 columns at a time: the block's 64 scores stay in registers meanwhile)
#pragma unroll 1
          for (int c = 0; c < DH / 16; ++c) {
            uint32_t r[16];
            tmem_ld16(tmem_o + t * D + lane_base + half * DH + c * 16, r);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st16(tmem_o + t * D + lane_base + half * DH + c * 16, r);
          }
          tmem_wait_st();
        }
        l_run *= factor;
        if (step) m_ref = mx;
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      // probabilities -> packed bf16 pairs, written over the block's scores in tensor memory
      const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
      const unsigned long long negm2 = pack_f32x2(-m_use, -m_use);
      unsigned long long lsum2 = pack_f32x2(0.f, 0.f);
      uint32_t packed[32];
#pragma unroll
      for (int i = 0; i < 64; i += 2) {
        float a0, a1;
        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), scale2, negm2), a0, a1);
        const float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
        lsum2 = add_f32x2(lsum2, pack_f32x2(p0, p1));
        packed[i >> 1] = pack_bf16(p0, p1);
      }
      float lsum, lsum_hi;
      unpack_f32x2(lsum2, lsum, lsum_hi);
      l_run += lsum + lsum_hi;
      if (t == 0) { m_t[0] = m_ref; l_t[0] = l_run; } else { m_t[1] = m_ref; l_t[1] = l_run; }
      tmem_st32(s_addr, packed);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&s_bar[P_FULL0 + (v & 1)]);
    }
#pragma unroll
    for (int t = 0; t < 2; ++t) s_xl[(t * 2 + half) * TC_BM + row] = l_t[t];
    softmax_ok = ok;
  } else if (warp == T2_MMA_WARP) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && nb > 0) {
      // Every operand descriptor is a constant plus a small offset (see tc_common.cuh).
      const uint32_t hi = tc_desc_hi(1024);
      const uint32_t q_lo = tc_desc_lo(smem_u32(sQ), 16), k_lo = tc_desc_lo(smem_u32(sK), 16);
      const uint32_t v_lo = tc_desc_lo(smem_u32(sV), TC_BN * 128);
      const uint32_t idesc_s_full = tc_idesc(TC_BM, TC_BN, 0), idesc_pv = tc_idesc(TC_BM, D, 1);
      bool ok = true;
      auto issue_s = [&](int v) {
        const int j = ntile == 2 ? v >> 1 : v, t = ntile == 2 ? (v & 1) : 0;
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t idesc = nj == TC_BN ? idesc_s_full : tc_idesc(TC_BM, nj, 0);
        const uint32_t qb = q_lo + t * (QT_BYTES >> 4);
        const uint32_t kb = k_lo + (j & 1) * (TILE_BYTES >> 4);
        const uint32_t d = tmem + (v & 1) * TC_BN;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t koff = ((ks >> 2) * (TC_BM * 128) + (ks & 3) * 32) >> 4;
          tc_mma_h(d, qb + koff, kb + koff, hi, idesc, ks > 0);
        }
        tc_commit(&s_bar[S_FULL0 + (v & 1)]);
        if (t == ntile - 1) tc_commit(&s_bar[K_EMPTY0 + (j & 1)]);  // the block's last reader
      };
      // K block j is awaited once, by the first S that reads it (tile 0)
      auto wait_k_for = [&](int v) {
        const int j = ntile == 2 ? v >> 1 : v, t = ntile == 2 ? (v & 1) : 0;
        if (t != 0) return true;
        return mbar_wait(&s_bar[K_FULL0 + (j & 1)], (j >> 1) & 1, s_abort);
      };
      ok = mbar_wait(&s_bar[Q_FULL], 0, s_abort);
      for (int v = 0; v < 2 && v < nv && ok; ++v) {
        ok = wait_k_for(v);
        if (ok) {
          tc_fence_after();
          issue_s(v);
        }
      }
      for (int v = 0; v < nv && ok; ++v) {
        const int j = ntile == 2 ? v >> 1 : v, t = ntile == 2 ? (v & 1) : 0;
        ok = mbar_wait(&s_bar[P_FULL0 + (v & 1)], (v >> 1) & 1, s_abort);
        if (ok && t == 0) ok = mbar_wait(&s_bar[V_FULL0 + (j & 1)], (j >> 1) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t vb = v_lo + (j & 1) * (TILE_BYTES >> 4);
        const uint32_t pb = tmem + (v & 1) * TC_BN;   // P_v sits where S_v was: 32 packed columns per half
        const uint32_t ob = tmem_o + t * D;
        // 16 keys = 8 packed columns of P = 2048 bytes of the V stage per step
        if (nj == TC_BN) {
#pragma unroll
          for (int ks = 0; ks < TC_BN / 16; ++ks)
            tc_mma_ts_h(ob, pb + (ks >> 2) * 64 + (ks & 3) * 8, vb + ks * (2048 >> 4), hi, idesc_pv,
                        (j > 0 || ks > 0) ? 1u : 0u);
        } else {
          for (int ks = 0; ks < nj / 16; ++ks)
            tc_mma_ts_h(ob, pb + (ks >> 2) * 64 + (ks & 3) * 8, vb + ks * (2048 >> 4), hi, idesc_pv,
                        (j > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(&s_bar[PV_FULL]);
        if (t == ntile - 1) tc_commit(&s_bar[V_EMPTY0 + (j & 1)]);
        if (v + 2 < nv) {
          ok = wait_k_for(v + 2);
          if (!ok) break;
          tc_fence_after();
          issue_s(v + 2);
        }
      }
      if (ok) tc_commit(&s_bar[O_DONE]);
      if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
    }
  } else if (warp == T2_KLOAD_WARP) {
    // ------------------------------------------------------------------ K loader (blocks 2..)
    if (lane == 0) {
      bool ok = true;
      int pg[MAX_PIECES];
      if (nb > 2) lookup_pages(2, pg);
      for (int j = 2; j < nb && ok; ++j) {
        ok = mbar_wait(&s_bar[K_EMPTY0 + (j & 1)], ((j >> 1) - 1) & 1, s_abort);
        if (!ok) break;
        issue_pieces(j, pg, &kmap, smem_u32(sK) + (j & 1) * TILE_BYTES, &s_bar[K_FULL0 + (j & 1)]);
        if (j + 1 < nb) lookup_pages(j + 1, pg);  // in flight while the next stage is awaited
      }
      if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
    }
  } else if (warp == T2_VLOAD_WARP) {
    // ------------------------------------------------------------------ V loader
    bool ok = true;
    int pg[MAX_PIECES];
    if (nb > 0 && lane == 0) {
      ok = mbar_wait(&s_bar[K_FULL0], 0, s_abort);
      if (ok) {
        issue_block(0, &vmap, smem_u32(sV), v_bar(0));
        if (nb > 1) issue_block(1, &vmap, smem_u32(sV) + TILE_BYTES, v_bar(1));
        if (nb > 2) lookup_pages(2, pg);
      }
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    for (int j = 0; j < nb && ok; ++j) {
      if (v_needs_fix(j)) {  // warp-uniform; at most once per sequence, so the barrier's phase is 0
        ok = mbar_wait(&s_bar[V_TMA0 + (j & 1)], 0, s_abort);
        if (!ok) break;
        // rows of this block that lie past the end of the sequence: zero them (at most 15)
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const int first_bad = L - (key_begin + j * TC_BN);
        uint8_t* stage = sV + (j & 1) * TILE_BYTES;
        for (int c = lane; c < (nj - first_bad) * CH; c += 32) {
          const int r = first_bad + c / CH, ch = c % CH;
          *reinterpret_cast<uint4*>(stage + sw128_chunk_off(r, ch, TC_BN)) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_bar[V_FULL0 + (j & 1)]);
      }
      if (lane == 0 && j + 2 < nb) {
        ok = mbar_wait(&s_bar[V_EMPTY0 + (j & 1)], (j >> 1) & 1, s_abort);
        if (ok) {
          issue_pieces(j + 2, pg, &vmap, smem_u32(sV) + (j & 1) * TILE_BYTES, v_bar(j + 2));
          if (j + 3 < nb) lookup_pages(j + 3, pg);
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (!ok && lane == 0) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
  }

  // ---- normalise and store ------------------------------------------------------------------------------
  // The softmax threads stage both tiles' rows as [O / l in bf16 (D) | base-2 log-sum-exp | pad | global row]
  // over the idle Q tiles (global row -1: the tile has no such row); then half a warp per row writes whole
  // rows: the output row and its log-sum-exp, or, with several KV chunks, this chunk's bf16 partial for
  // attn_merge_kernel.
  // A tile is staged as soon as its accumulator is final.  With two tiles that is PV_{nv-2} for tile 0 (the
  // barrier is in that phase or the next, since S_{nv-1} has been consumed), so tile 0 is staged while the last
  // PV runs.  By then every S has completed, and with the MMAs every load into the Q tiles and K stages (each
  // was awaited before the MMA that read it).
  constexpr int ROWB = D * 2 + 16;  // bytes per staged row (16-byte multiple)
  if (tid < T2_SOFTMAX_THREADS) {
    bool ok = softmax_ok;
    const bool have = nb > 0 && sp.compute;
    softmax_group_sync();  // both halves' running sums are in s_xl
    for (int t = 0; t < ntile; ++t) {
      if (nb > 0 && ok) {
        ok = t + 1 < ntile ? mbar_wait(&s_bar[PV_FULL], (nv - 2) & 1, s_abort) : mbar_wait(&s_bar[O_DONE], 0, s_abort);
        tc_fence_after();
      }
      uint8_t* stg = sQ + t * (TC_BM * ROWB);  // disjoint per tile; runs a little into the idle K stage
      const float l_tot = s_xl[(t * 2) * TC_BM + row] + s_xl[(t * 2 + 1) * TC_BM + row];
      const float m_ref = t == 0 ? m_t[0] : m_t[1];
      const float inv_l = (have && l_tot > 0.f) ? __fdividef(1.f, l_tot) : 0.f;
      uint8_t* dst = stg + row * ROWB;
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        if (have) tmem_ld32(tmem_o + t * D + lane_base + half * DH + c * 32, r);  // warp-uniform condition
#pragma unroll
        for (int d = 0; d < 32; d += 8) {
          uint4 o4;
          o4.x = pack_bf16(have ? __uint_as_float(r[d]) * inv_l : 0.f, have ? __uint_as_float(r[d + 1]) * inv_l : 0.f);
          o4.y = pack_bf16(have ? __uint_as_float(r[d + 2]) * inv_l : 0.f, have ? __uint_as_float(r[d + 3]) * inv_l : 0.f);
          o4.z = pack_bf16(have ? __uint_as_float(r[d + 4]) * inv_l : 0.f, have ? __uint_as_float(r[d + 5]) * inv_l : 0.f);
          o4.w = pack_bf16(have ? __uint_as_float(r[d + 6]) * inv_l : 0.f, have ? __uint_as_float(r[d + 7]) * inv_l : 0.f);
          *reinterpret_cast<uint4*>(dst + (half * DH + c * 32 + d) * 2) = o4;
        }
      }
      if (half == 0) {
        const int Rr = row0 + t * TC_BM + row;
        const int node_l = Rr / G, hh = Rr - node_l * G;
        const long long grow = (long long)(si.q_off + node_l) * Hq + g * G + hh;
        const bool row_ok = Rr < rows_total && SB_CHECKED_ACCESS(grow, rows_all, &p.status[b]);
        *reinterpret_cast<float*>(dst + D * 2) = (have && l_tot > 0.f) ? m_ref + log2f(l_tot) : -INFINITY;
        *reinterpret_cast<long long*>(dst + D * 2 + 8) = row_ok ? grow : -1ll;
      }
    }
    if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
  }
  tc_fence_before();
  __syncthreads();  // the rows are staged; tensor memory has been read for the last time
  if (warp == T2_MMA_WARP) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(T2_TMEM_COLS));
  }
  for (int t = 0; t < ntile; ++t) {
    const uint8_t* stg = sQ + t * (TC_BM * ROWB);
    const int sub = lane >> 4, col8 = lane & 15;
    if (col8 >= D / 8) continue;
#pragma unroll 3
    for (int r = 2 * warp + sub; r < TC_BM; r += 2 * (T2_THREADS / 32)) {
      const uint8_t* rowp = stg + (size_t)r * ROWB;
      const long long grow = *reinterpret_cast<const long long*>(rowp + D * 2 + 8);
      const float lse2 = *reinterpret_cast<const float*>(rowp + D * 2);
      const uint4 raw = *reinterpret_cast<const uint4*>(rowp + col8 * 16);
      if (grow < 0) continue;
      if (p.outer == 1) {
        *reinterpret_cast<uint4*>(p.out + grow * D + col8 * 8) = raw;
        if (p.lse && col8 == 0) p.lse[grow] = lse2 == -INFINITY ? 0.f : lse2 * kLn2;
      } else {
        // the staged row is bf16 already: partials keep that width (half the bytes of fp32, same values)
        bf16* po = reinterpret_cast<bf16*>(p.part_o) + ((long long)split * rows_all + grow) * D + col8 * 8;
        *reinterpret_cast<uint4*>(po) = raw;
        if (col8 == 0) p.part_lse[(long long)split * rows_all + grow] = lse2;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------

template <int D>
static sb_status launch_tc2(const AttnParams& p, dim3 grid, cudaStream_t cs) {
  static PerDeviceOnce once;
  if (!once.run([]() {
        const bool ok = cudaFuncSetAttribute(attn_tc2_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)attn_tc2_smem_bytes<D>()) == cudaSuccess;
        if (!ok) cudaGetLastError();
        return ok;
      }))
    return SB_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(T2_THREADS);
  cfg.dynamicSmemBytes = attn_tc2_smem_bytes<D>();
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  // the kernel orders itself after its predecessor with griddepcontrol.wait
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = test_knob("SB_NO_PDL") ? 0 : 1;
  if (test_knob("SB_DEBUG"))
    fprintf(stderr, "[sb] attn_tc2<%d> grid (%u,%u,%u) outer %d\n", D, grid.x, grid.y, grid.z, p.outer);
  const int box_rows = p.tb.page_size == 0 ? TC_BN : (p.tb.page_size < TC_BN ? p.tb.page_size : TC_BN);
  CUtensorMap kmap, vmap, qmap;
  if (!make_kv_map(&kmap, p.tb, p.tb.k_cache, box_rows) || !make_kv_map(&vmap, p.tb, p.tb.v_cache, box_rows))
    return SB_ERR_CUDA;
  const int q_tma = (TC_BM % p.G == 0) ? 1 : 0;
  if (q_tma) {
    if (!make_q_map(&qmap, p)) return SB_ERR_CUDA;
  } else {
    qmap = kmap;  // unused by the kernel in this mode
  }
  if (cudaLaunchKernelEx(&cfg, attn_tc2_kernel<D>, p, kmap, vmap, qmap, box_rows, q_tma) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

// grid = (chunks, KV heads x tile pairs, sequences); p.num_splits = p.outer = chunks
sb_status launch_attn_tc2(const AttnParams& p, dim3 grid, cudaStream_t cs) {
  return p.tb.head_dim == 64 ? launch_tc2<64>(p, grid, cs) : launch_tc2<128>(p, grid, cs);
}

}  // namespace sb
