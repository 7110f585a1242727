// Tree-masked split-KV attention on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// One CTA owns a 128-row query tile (rows = (node, head-in-group) pairs of one KV head: the tile
// is the M = 128 dimension of the MMA and one row per TMEM lane) and a chunk of the sequence's
// keys, walked in blocks of up to 128 keys:
//
//   loader warps   one thread per operand issues TMA tile loads (cp.async.bulk.tensor, 128-byte swizzle,
//                  no multicast) of the K and V blocks straight into the shared-memory layouts the
//                  tensor core reads (K, Q, P: K-major; V: MN-major), 2 stages each, completion by
//                  mbarrier transaction count; paged caches load one box per page piece, the page ids
//                  of the next block being fetched while its stage is still busy.  A V block lands
//                  on the barrier the MMA warp waits on, except the one whose rows pass the end of
//                  the sequence: those rows are zeroed first (P is 0 there, but 0 * garbage must stay 0).
//                  The Q tile is one TMA box {64 columns, G heads, 128/G nodes} per column half when
//                  G divides 128, else a 16-byte cp.async gather by the softmax warps;
//   MMA warp       one thread issues  S_j = Q K_j^T  (tcgen05.mma, fp32 accumulator in TMEM, two S
//                  buffers) and  O += P_j V_j  with P_j read from TMEM and O accumulated in TMEM;
//                  operand descriptors are constant halves plus an offset (two adds per MMA);
//   softmax warps  8 warps, two threads per row (TMEM lane), each owning 64 of a block's 128 columns:
//                  read S once from TMEM into registers (tcgen05.ld; the S buffer is released at
//                  once), apply the softmax scale and the tree mask (one 128-bit ancestor set per
//                  row, turned into a 64-bit visibility window per block half; prefix-only blocks
//                  skip it), exchange the row maximum through shared memory, and write
//                  P_j = 2^(s - m_ref) as packed bf16 back into TMEM (tcgen05.st, two P buffers).
//                  m_ref is a lazily updated reference maximum: it moves (and O and the running
//                  sum are rescaled, tcgen05.ld/st) only when a block's maximum exceeds it by more
//                  than 8 in the base-2 domain, so P never exceeds 2^8 and the rescale is rare.
//
// All hand-offs are mbarriers (tcgen05.commit on the MMA side); every wait is bounded and reports
// SB_ERR_CUDA instead of spinning forever.  The chunk results of the CTAs of a cluster are merged
// through distributed shared memory: every CTA stages its rows normalised in bf16 with (m, l), sends
// each owner CTA its slice with one bulk shared-to-shared copy, and the owner reduces and stores.
// Grids that run in several waves take their sequences longest first (attention_common.cuh).
#include <cstdio>
#include <cstdlib>

#include "tc_common.cuh"

namespace sb {

constexpr int TC_SOFTMAX_THREADS = 256;  // warps 0-3: columns [0,64) of a block, warps 4-7: [64,128)
constexpr int TC_MMA_WARP = 8;
constexpr int TC_KLOAD_WARP = 9;     // lane 0 issues the Q and K loads
constexpr int TC_VLOAD_WARP = 10;    // lane 0 issues the V loads; the warp zeroes rows past the sequence
constexpr int TC_THREADS = 384;      // 12 warps (warp 11 only takes part in the barriers)
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_SMALL_BYTES = 8192; // ancestor masks, parents, barriers, softmax exchange
constexpr int TC_MAX_CLUSTER = 10;          // chunks merged in one cluster (9 and 10 are beyond the portable size)
constexpr int TC_MERGE_SLOTS = TC_BM + 8;  // receive slots: S * ceil(128 / S) <= 135 for S <= 10

enum TcBar { K_FULL0, K_FULL1, K_EMPTY0, K_EMPTY1, V_FULL0, V_FULL1, V_EMPTY0, V_EMPTY1, S_FULL0, S_FULL1,
             S_EMPTY0, S_EMPTY1, P_FULL, PV_FULL, V_TMA0, V_TMA1, Q_FULL, MERGE_BAR, ACK_BAR, TC_NUM_BARS };

template <int D>
constexpr size_t attn_tc_smem_bytes() {
  // small region + Q + 2 K stages + 2 V stages + the merge receive buffer (bf16 rows + m, l), plus
  // slack to align the tiles to 1024 bytes
  return 1024 + TC_SMALL_BYTES + (size_t)TC_BM * D * 2 + 4 * (size_t)TC_BN * D * 2 + (size_t)TC_MERGE_SLOTS * (D * 2 + 16);
}


// FAST: the common single-wave case fixed at compile time -- contiguous cache (one 128-row TMA box per
// block, no page table), Q tile by TMA, all chunks of a tile in one cluster (no fp32 partials), grid
// index z = sequence.  The general instantiation decides all of that at run time (paged caches, a
// gathered Q tile, partials for attn_merge_kernel, sequences taken longest first).  Code that is
// never executed still costs a kernel this short: an untaken branch to the sequence ranking alone
// was 0.1 us per launch, and knowing the cluster size (CS = 1..10, the chunks of a tile) at compile
// time another 0.4 us.  CS = 0 is the general instantiation; 9 and 10 are beyond the portable cluster size.
template <int D, int CS>
__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const AttnParams p,
                                                                const __grid_constant__ CUtensorMap kmap,
                                                                const __grid_constant__ CUtensorMap vmap,
                                                                const __grid_constant__ CUtensorMap qmap,
                                                                const int box_rows_arg, const int q_tma_arg) {
  constexpr bool FAST = CS > 0;
  const int box_rows = FAST ? TC_BN : box_rows_arg;
  const int q_tma = FAST ? 1 : q_tma_arg;
  const int page_size = FAST ? 0 : p.tb.page_size;
  constexpr int CH = D / 8;                   // 16-byte chunks per row
  constexpr int TILE_BYTES = TC_BN * D * 2;   // one K or V stage
  constexpr int DH = D / 2;                   // output columns per softmax thread
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint32_t* s_anc = reinterpret_cast<uint32_t*>(base);               // 2048 B
  int* s_parent = reinterpret_cast<int*>(base + 2048);               // 512 B
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(base + 2560);        // TC_NUM_BARS * 8
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(base + 2816);
  volatile int* s_abort = reinterpret_cast<volatile int*>(base + 2820);
  float* s_xmax = reinterpret_cast<float*>(base + 3072);             // [2 parities][2 halves][128 rows]
  float* s_xl = reinterpret_cast<float*>(base + 5120);               // [2 halves][128 rows]
  uint8_t* sQ = base + TC_SMALL_BYTES;
  uint8_t* sK = sQ + TC_BM * D * 2;
  uint8_t* sV = sK + 2 * TILE_BYTES;
  uint8_t* sRcv = sV + 2 * TILE_BYTES;  // merge receive buffer: written by cluster peers only

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = FAST ? CS : (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int split = blockIdx.x;
  const int Hq = p.tb.n_q_heads, G = p.G;
  // row tiles of one (sequence, KV head) are neighbours in launch order: they share its K/V through L2
  const int g = blockIdx.y / p.row_tiles, tile = blockIdx.y % p.row_tiles;
  if (tid == 0) {
    *s_abort = 0;
    const int n = TC_SOFTMAX_THREADS;
    const int counts[TC_NUM_BARS] = {1, 1, 1, 1, 1, 1, 1, 1, 1, 1, n, n, n, 1, 1, 1, q_tma ? 1 : n, 1, S};
    for (int i = 0; i < TC_NUM_BARS; ++i) mbar_init(&s_bar[i], counts[i]);
    // the merge barrier is armed at once: cluster peers may deliver their rows at any time
    if (S > 1) {
      const int rp = ceil_div(TC_BM, S);
      const int mine = max(0, min(TC_BM, (crank + 1) * rp) - crank * rp);
      mbar_expect_tx(&s_bar[MERGE_BAR], (uint32_t)(S * mine * (D * 2 + 16)));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == TC_MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TC_TMEM_COLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Non-blocking half of a cluster barrier: "my barriers are initialised".  The matching wait sits
  // just before this CTA first touches a peer's barrier, microseconds later.
  if (S > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  // Programmatic dependent launch: everything above is independent of earlier kernels' results and
  // may overlap their tail; from here on their memory is complete and visible.  Dependents of this
  // kernel are released right away, so at most two consecutive grids are ever in flight.
  // A caller may vouch that the kernel just before does not write the index arrays: then the sequence
  // lengths (one trip to the L2 cache, on the way to the first load) are fetched before the wait.
  const bool lengths_early = p.tb.index_arrays_settled != 0 && !(!FAST && p.sort_seqs);
  if (!lengths_early) asm volatile("griddepcontrol.wait;" ::: "memory");

  // grid index z -> sequence (longest first when the grid runs in several waves)
  const int b = (!FAST && p.sort_seqs) ? sequence_of_rank(p.tb, blockIdx.z, reinterpret_cast<int*>(s_anc), s_parent)
                                       : (int)blockIdx.z;
  const SeqPre pre = plan_lengths(p, b);
  // A second vouch, for the committed prefix's cache rows (positions below prefix_len): the K blocks of this
  // CTA's first two stages that lie wholly inside the prefix are requested before the wait as well, so that
  // they are on their way from HBM while the predecessor finishes (Q, a fresh product of that predecessor,
  // comes from L2 and is faster anyway).  Contiguous single-wave variant only.
  const bool kv_early = FAST && lengths_early && p.tb.prefix_rows_settled != 0;
  if (lengths_early && !kv_early) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!kv_early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int rows_total = pre.info.nq * G;
  const int row0 = tile * TC_BM;
  if (!pre.can_write || row0 >= rows_total) {  // uniform over the cluster
    if (kv_early) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    // the designated CTA always owns rows unless the sequence has none; its status is still due
    if (split == 0 && blockIdx.y == 0 && tid == 0) p.status[b] = pre.info.err;
    if (warp == TC_MMA_WARP)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*s_tmem), "r"(TC_TMEM_COLS));
    if (S > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // pairs with the arrive above
    return;
  }
  const long long rows_all = (long long)p.total_q * Hq;

  // Balanced cut of the sequence's 128-key blocks into num_splits chunks (block-aligned, so a
  // TMA box never straddles a page); the sequence's last block is trimmed to a multiple of 16 keys.
  const int L = pre.info.P + pre.info.n;
  const int blocks_total = ceil_div(L, TC_BN);
  const int b_base = blocks_total / p.num_splits, b_rem = blocks_total % p.num_splits;
  const int key_begin = TC_BN * (split * b_base + min(split, b_rem));
  const int nb = pre.info.err == 0 ? b_base + (split < b_rem ? 1 : 0) : 0;
  const int chunk_keys = nb == 0 ? 0 : min(nb * TC_BN, ceil_div(L - key_begin, 16) * 16);

  const uint32_t tmem = *s_tmem;
  // TMEM columns: S buffers [0,128) and [128,256), O [256,256+D), P buffers (packed bf16) [384,448), [448,512)
  const uint32_t tmem_o = tmem + 2 * TC_BN;
  const uint32_t tmem_p = tmem + 3 * TC_BN;

  // One TMA box per page piece of a block: box_rows keys x 64 columns, per 64-column half.  The
  // page ids of a block are looked up separately (page sizes are powers of two >= 16: at most 8
  // pieces), so that a loader can have them in registers before the stage it waits for is free.
  constexpr int MAX_PIECES = TC_BN / 16;
  auto lookup_pages = [&](int j, int (&pg)[MAX_PIECES]) {
    if (FAST || page_size == 0) return;
    const int nj = min(TC_BN, chunk_keys - j * TC_BN);
    const int k0 = key_begin + j * TC_BN;
    const int pieces = ceil_div(nj, box_rows);
#pragma unroll 1
    for (int i = 0; i < MAX_PIECES; ++i)
      if (i < pieces) {
        const int lp = (k0 + i * box_rows) / (FAST ? 1 : page_size);
        pg[i] = SB_CHECKED_ACCESS(lp, p.tb.max_pages, &p.status[b]) ? p.tb.page_table[(long long)b * p.tb.max_pages + lp] : 0;
      }
  };
  auto issue_pieces = [&](int j, const int (&pg)[MAX_PIECES], const CUtensorMap* map, uint32_t stage_addr,
                          uint64_t* bar) {
    const int nj = min(TC_BN, chunk_keys - j * TC_BN);
    const int k0 = key_begin + j * TC_BN;
    if (FAST) {  // one box of 128 rows per column half (rows past the cache read as zero)
      mbar_expect_tx(bar, (uint32_t)(TC_BN * D * 2));
#pragma unroll
      for (int h = 0; h < D / 64; ++h) tma_load_4d(stage_addr + h * (TC_BN * 128), map, h * 64, g, k0, b, bar);
      return;
    }
    const int pieces = ceil_div(nj, box_rows);
    mbar_expect_tx(bar, (uint32_t)(pieces * box_rows * D * 2));
#pragma unroll 1
    for (int i = 0; i < MAX_PIECES; ++i) {
      if (i >= pieces) break;
      const int key = k0 + i * box_rows;
      int c2 = key, c3 = b;
      if (page_size != 0) {
        int page = pg[i];
        if (page < 0 || page >= p.tb.num_pages) page = 0;  // reported by the designated CTA
        c2 = key & (page_size - 1);
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
  // A V block whose rows reach past the end of the sequence holds stale cache rows there; they
  // meet zero probabilities, but must not be NaN or infinite: such a block (only the last one of
  // the sequence can be) lands on a barrier of its own and is cleaned before the MMA may read it.
  // Every other V block completes the barrier the MMA warp waits on directly.
  auto v_needs_fix = [&](int j) { return L - (key_begin + j * TC_BN) < min(TC_BN, chunk_keys - j * TC_BN); };
  auto v_bar = [&](int j) { return &s_bar[(v_needs_fix(j) ? V_TMA0 : V_FULL0) + (j & 1)]; };
  // The first loads go out before anything else: they only need the sequence's lengths.  Only
  // the K side (Q, K blocks 0 and 1) is requested at once; the V blocks, needed a softmax later,
  // follow when K block 0 has landed, so they do not queue in front of it in the memory system.
  if (nb > 0 && lane == 0 && warp == TC_KLOAD_WARP) {
    bool k0e = false, k1e = false;
    if (kv_early) {
      if (key_begin + TC_BN <= pre.info.P) {
        issue_block(0, &kmap, smem_u32(sK), &s_bar[K_FULL0]);
        k0e = true;
      }
      if (nb > 1 && key_begin + 2 * TC_BN <= pre.info.P) {
        issue_block(1, &kmap, smem_u32(sK) + TILE_BYTES, &s_bar[K_FULL1]);
        k1e = true;
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    if (q_tma) {
      mbar_expect_tx(&s_bar[Q_FULL], (uint32_t)(TC_BM * D * 2));
#pragma unroll
      for (int h = 0; h < D / 64; ++h)
        tma_load_3d(smem_u32(sQ) + h * (TC_BM * 128), &qmap, h * 64, g * G, pre.info.q_off + tile * (TC_BM / G),
                    &s_bar[Q_FULL]);
    }
    if (!k0e) issue_block(0, &kmap, smem_u32(sK), &s_bar[K_FULL0]);
    if (nb > 1 && !k1e) issue_block(1, &kmap, smem_u32(sK) + TILE_BYTES, &s_bar[K_FULL1]);
  } else if (kv_early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }

  const SeqPlan sp = plan_tree(p, b, split == 0 && blockIdx.y == 0, pre, s_parent, s_anc);
  const SeqInfo& si = sp.info;

  // Row state of the softmax threads: row = TMEM lane, `half` selects the 64 columns of every block
  // and the half of the output row this thread owns.
  constexpr float kRescaleStep = 8.f;  // m_ref follows the row maximum in steps of at least 2^8
  float o_row[DH];
  float m_ref = -INFINITY, l_run = 0.f;
  const int half = (warp >> 2) & 1;
  const int row = (warp & 3) * 32 + lane;

  if (tid < TC_SOFTMAX_THREADS) {
    // ------------------------------------------------------------------ softmax warps
    if (!q_tma && nb > 0) {  // Q tile as a gather of (node, head) rows
      const uint32_t qd = smem_u32(sQ);
      for (int c = tid; c < TC_BM * CH; c += TC_SOFTMAX_THREADS) {
        const int r = c / CH, ch = c % CH;
        const int R = row0 + r;
        const bool valid = R < rows_total;
        const int node_l = valid ? R / G : 0;
        const int hh = valid ? R - node_l * G : 0;
        const long long off = ((long long)(si.q_off + node_l) * Hq + g * G + hh) * D + ch * 8;
        const bool q_ok = valid && SB_CHECKED_ACCESS(off + 7, (long long)p.total_q * Hq * D, &p.status[b]);
        cp_async_16_tc(qd + sw128_chunk_off(r, ch, TC_BM), p.q + (q_ok ? off : 0), q_ok ? 16 : 0);
      }
      asm volatile("cp.async.commit_group;\n" ::);
      asm volatile("cp.async.wait_group 0;\n" ::: "memory");
      fence_async_smem();
      mbar_arrive(&s_bar[Q_FULL]);
    }
    const int R = row0 + row;
    const bool row_live = R < rows_total && sp.compute;
    uint32_t anc[4];
    {
      const int node = row_live ? si.q0 + R / G : 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) anc[w] = row_live ? s_anc[4 * node + w] : 0u;
    }
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    bool ok = true;
    // The trip count and the named barrier inside are uniform over the 256 threads: after a failed
    // wait the remaining waits return at once (abort flag) and the loop just runs out.
    for (int j = 0; j < nb; ++j) {
      const int k0 = key_begin + j * TC_BN;
      const int nj = min(TC_BN, chunk_keys - j * TC_BN);  // keys of this block (multiple of 16)
      const int my_cols = nj - 64 * half;                 // valid columns among this thread's 64
      if (ok) ok = mbar_wait(&s_bar[S_FULL0 + (j & 1)], (j >> 1) & 1, s_abort);
      tc_fence_after();
      uint32_t sr[64];
      tmem_ld64(tmem + lane_base + (j & 1) * TC_BN + 64 * half, sr);
      tc_fence_before();
      mbar_arrive(&s_bar[S_EMPTY0 + (j & 1)]);  // S is in registers: the buffer may be refilled
      // visibility of this thread's 64 columns: tree mask where the block reaches past the prefix,
      // and only the block's own nj columns
      uint64_t win = k0 + TC_BN > si.P ? visibility_window(anc, k0 + 64 * half - si.P) : ~0ull;
      win &= my_cols >= 64 ? ~0ull : (my_cols <= 0 ? 0ull : ((1ull << my_cols) - 1ull));
      // row maximum of the raw scores (the softmax scale is positive: it commutes with max)
      if (win != ~0ull) {  // only blocks that touch the tree or the end of the chunk have masked columns
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (!((win >> i) & 1ull)) sr[i] = 0xff800000u;  // -inf
      }
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 2) mx = max3(mx, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
      mx *= p.scale_log2;
      s_xmax[((j & 1) * 2 + half) * TC_BM + row] = mx;
      softmax_group_sync();
      mx = fmaxf(mx, s_xmax[((j & 1) * 2 + (half ^ 1)) * TC_BM + row]);
      // lazy reference maximum: both threads of a row take the same decision
      const bool step = mx > m_ref + kRescaleStep || (m_ref == -INFINITY && mx > -INFINITY);
      bool pv_waited = false;
      if (__any_sync(0xffffffffu, step)) {
        const float factor = (step && m_ref != -INFINITY) ? fast_exp2(m_ref - mx) : 1.f;
        if (j > 0) {  // O holds blocks 0..j-1: rescale this thread's half-row in tensor memory
          if (ok) ok = mbar_wait(&s_bar[PV_FULL], (j - 1) & 1, s_abort);
          pv_waited = true;
          tc_fence_after();
          // (rare, and 16 columns at a time: the block's 64 scores stay in registers meanwhile)
#pragma unroll 1
          for (int c = 0; c < DH / 16; ++c) {
            uint32_t r[16];
            tmem_ld16(tmem_o + lane_base + half * DH + c * 16, r);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st16(tmem_o + lane_base + half * DH + c * 16, r);
          }
          tmem_wait_st();
        }
        l_run *= factor;
        if (step) m_ref = mx;
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
      // probabilities -> packed bf16 pairs, written to the block's P buffer in tensor memory
      // p = 2^(s * scale - m_ref): the argument and the running sum use packed two-lane arithmetic
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
      lsum += lsum_hi;
      l_run += lsum;
      // Every PV phase is waited for, in order (a parity wait must never lag a whole phase), and
      // late: PV_{j-1} done also means PV_{j-2} has consumed the P buffer about to be overwritten.
      if (j > 0 && !pv_waited) {
        if (ok) ok = mbar_wait(&s_bar[PV_FULL], (j - 1) & 1, s_abort);
        tc_fence_after();
      }
      tmem_st32(tmem_p + lane_base + (j & 1) * 64 + half * 32, packed);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&s_bar[P_FULL]);
    }
#pragma unroll
    for (int d = 0; d < DH; ++d) o_row[d] = 0.f;
    if (nb > 0) {
      if (ok) ok = mbar_wait(&s_bar[PV_FULL], (nb - 1) & 1, s_abort);
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_o + lane_base + half * DH + c * 32, r);
#pragma unroll
        for (int i = 0; i < 32; ++i) o_row[c * 32 + i] = __uint_as_float(r[i]);
      }
    }
    s_xl[half * TC_BM + row] = l_run;
    if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
  } else if (warp == TC_MMA_WARP) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && nb > 0) {
      // Every operand descriptor is a constant plus a small offset: the halves are formed once, so
      // that each MMA costs the issuing thread a couple of integer adds.
      const uint32_t hi = tc_desc_hi(1024);
      const uint32_t q_lo = tc_desc_lo(smem_u32(sQ), 16), k_lo = tc_desc_lo(smem_u32(sK), 16);
      const uint32_t v_lo = tc_desc_lo(smem_u32(sV), TC_BN * 128);
      const uint32_t idesc_s_full = tc_idesc(TC_BM, TC_BN, 0), idesc_pv = tc_idesc(TC_BM, D, 1);
      bool ok = true;
      auto issue_s = [&](int j) {
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t idesc = nj == TC_BN ? idesc_s_full : tc_idesc(TC_BM, nj, 0);
        const uint32_t kb = k_lo + (j & 1) * (TILE_BYTES >> 4);
        const uint32_t d = tmem + (j & 1) * TC_BN;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t koff = ((ks >> 2) * (TC_BM * 128) + (ks & 3) * 32) >> 4;
          tc_mma_h(d, q_lo + koff, kb + koff, hi, idesc, ks > 0);
        }
        tc_commit(&s_bar[S_FULL0 + (j & 1)]);
        tc_commit(&s_bar[K_EMPTY0 + (j & 1)]);
      };
      ok = mbar_wait(&s_bar[Q_FULL], 0, s_abort);
      if (ok) ok = mbar_wait(&s_bar[K_FULL0], 0, s_abort);
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
        if (!ok) break;
        tc_fence_after();
        const int nj = min(TC_BN, chunk_keys - j * TC_BN);
        const uint32_t vb = v_lo + (j & 1) * (TILE_BYTES >> 4);
        const uint32_t pb = tmem_p + (j & 1) * 64;
        // 16 keys = 8 packed columns of P = 2048 bytes of the V stage per step
        if (nj == TC_BN) {
#pragma unroll
          for (int ks = 0; ks < TC_BN / 16; ++ks)
            tc_mma_ts_h(tmem_o, pb + ks * 8, vb + ks * (2048 >> 4), hi, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
        } else {
          for (int ks = 0; ks < nj / 16; ++ks)
            tc_mma_ts_h(tmem_o, pb + ks * 8, vb + ks * (2048 >> 4), hi, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(&s_bar[PV_FULL]);
        tc_commit(&s_bar[V_EMPTY0 + (j & 1)]);
      }
      if (!ok) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
    }
  } else if (warp == TC_KLOAD_WARP) {
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
  } else if (warp == TC_VLOAD_WARP) {
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

  // ---- merge the cluster's chunks and store -------------------------------------------------------
  // Row r of the tile is owned by cluster CTA r / rows_per.  Every CTA stages its 128 rows as
  // [O / l in bf16 (D) | m | l | pad] (normalised, so bf16 has the range and O(2^-9) relative error
  // against a 1e-2 tolerance), then sends each owner its slice with ONE bulk asynchronous
  // shared-to-shared copy credited to the owner's mbarrier.  The receive buffer is written by
  // peers only and its barrier was armed at kernel start, so nothing has to be awaited before
  // sending.  The owner reduces its rows over the S sources and stores them; a CTA leaves once
  // every owner has acknowledged that its slice has arrived.
  constexpr int ROWB = D * 2 + 16;                  // bytes per staged row (16-byte multiple)
  uint8_t* stg = sQ;                                // [128][ROWB]: Q and the K stages are idle by now
  const int rows_per = ceil_div(TC_BM, S);
  const int my_first = crank * rows_per;
  const int my_rows = max(0, min(TC_BM, my_first + rows_per) - my_first);
  // No CTA-wide barrier here: a softmax thread has seen the last PV complete, and the tensor pipe runs a
  // thread's MMAs in order, so every MMA has read its operands and every K/V/Q load (each landed before the
  // MMA that used it) is done -- the staging area below (the Q tile and the head of K stage 0) is free.
  if (tid < TC_SOFTMAX_THREADS) {
    const bool have = nb > 0 && sp.compute;
    softmax_group_sync();  // both halves' running sums are in s_xl
    const float l_tot = s_xl[row] + s_xl[TC_BM + row];
    const float inv_l = (have && l_tot > 0.f) ? __fdividef(1.f, l_tot) : 0.f;
    uint8_t* dst = stg + row * ROWB;
#pragma unroll
    for (int d = 0; d < DH; d += 8) {
      uint4 v;
      v.x = pack_bf16(o_row[d] * inv_l, o_row[d + 1] * inv_l);
      v.y = pack_bf16(o_row[d + 2] * inv_l, o_row[d + 3] * inv_l);
      v.z = pack_bf16(o_row[d + 4] * inv_l, o_row[d + 5] * inv_l);
      v.w = pack_bf16(o_row[d + 6] * inv_l, o_row[d + 7] * inv_l);
      *reinterpret_cast<uint4*>(dst + (half * DH + d) * 2) = v;
    }
    if (half == 0) {
      *reinterpret_cast<float*>(dst + D * 2) = (have && l_tot > 0.f) ? m_ref : -INFINITY;
      *reinterpret_cast<float*>(dst + D * 2 + 4) = (have && l_tot > 0.f) ? l_tot : 0.f;
    }
  }
  bool merge_ok = true;
  tc_fence_before();
  if (S > 1) {
    fence_async_smem();  // the staged rows are read by the bulk-copy engine
    __syncthreads();     // rows staged; every role is done and every read of tensor memory is over
    if (warp == TC_MMA_WARP) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS));
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // every peer's barriers exist (long since)
    if (tid < S) {       // thread c sends owner c its slice
      const int c = tid;
      const int first = c * rows_per;
      const int n = max(0, min(TC_BM, first + rows_per) - first);
      if (n > 0)
        dsmem_bulk_copy(mapa_u32(smem_u32(sRcv + (size_t)crank * rows_per * ROWB), c), smem_u32(stg + (size_t)first * ROWB),
                        (uint32_t)(n * ROWB), mapa_u32(smem_u32(&s_bar[MERGE_BAR]), c));
    }
    merge_ok = mbar_wait(&s_bar[MERGE_BAR], 0, s_abort);
    // Every source's slice has landed here: tell each source that its staging rows are free.  The
    // last warp does it (it owns the fewest rows of the reduction below, often none), and the arrive
    // carries no data, so it needs no release ordering.
    if (warp == TC_THREADS / 32 - 1 && lane < S) mbar_arrive_remote_relaxed(mapa_u32(smem_u32(&s_bar[ACK_BAR]), lane));
  } else {
    __syncthreads();
    if (warp == TC_MMA_WARP) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS));
    }
  }
  {
    // One row per half-warp, eight columns per lane (D <= 128).  Every lane reads all S (m, l)
    // pairs itself (broadcast loads) and forms the weights redundantly, then loads its columns
    // from all S sources at once: no serial chain over the sources and no shuffles.
    const uint8_t* src = S > 1 ? sRcv : stg;  // [source][row in my slice][ROWB]
    const int sub = lane >> 4, col8 = lane & 15;
    for (int t = 2 * warp + sub; t < my_rows; t += 2 * (TC_THREADS / 32)) {
      const int Rr = row0 + my_first + t;
      if (Rr >= rows_total) continue;
      const bool has_cols = col8 < D / 8;
      constexpr int SRC = FAST ? CS : TC_MAX_CLUSTER;  // sources: known at compile time in the common case
      float w[SRC];
      uint4 raw[SRC];
      float M = -INFINITY, Lsum = 0.f;
      {
        float mc[SRC], lc[SRC];
#pragma unroll
        for (int c = 0; c < SRC; ++c) {
          const uint8_t* rowp = src + ((size_t)(c < S ? c : 0) * rows_per + t) * ROWB;
          mc[c] = c < S ? *reinterpret_cast<const float*>(rowp + D * 2) : -INFINITY;
          lc[c] = c < S ? *reinterpret_cast<const float*>(rowp + D * 2 + 4) : 0.f;
          raw[c] = (c < S && has_cols) ? *reinterpret_cast<const uint4*>(rowp + col8 * 16) : make_uint4(0u, 0u, 0u, 0u);
          M = fmaxf(M, mc[c]);
        }
#pragma unroll
        for (int c = 0; c < SRC; ++c) {
          w[c] = mc[c] == -INFINITY ? 0.f : fast_exp2(mc[c] - M) * lc[c];  // 2^(m_c - M) * l_c
          Lsum += w[c];
        }
      }
      const float inv = Lsum > 0.f ? __fdividef(1.f, Lsum) : 0.f;
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
      for (int c = 0; c < SRC; ++c) {
        const uint32_t q4[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          acc[2 * e] += w[c] * __uint_as_float(q4[e] << 16);
          acc[2 * e + 1] += w[c] * __uint_as_float(q4[e] & 0xffff0000u);
        }
      }
      const int node_l = Rr / G, hh = Rr - node_l * G;
      const long long grow = (long long)(si.q_off + node_l) * Hq + g * G + hh;
      const float lse2 = Lsum > 0.f ? M + log2f(Lsum) : -INFINITY;
      if (has_cols && SB_CHECKED_ACCESS(grow, rows_all, &p.status[b])) {
        if (FAST || p.outer == 1) {
          uint4 packed;
          packed.x = pack_bf16(acc[0] * inv, acc[1] * inv);
          packed.y = pack_bf16(acc[2] * inv, acc[3] * inv);
          packed.z = pack_bf16(acc[4] * inv, acc[5] * inv);
          packed.w = pack_bf16(acc[6] * inv, acc[7] * inv);
          *reinterpret_cast<uint4*>(p.out + grow * D + col8 * 8) = packed;
          if (p.lse && col8 == 0) p.lse[grow] = lse2 == -INFINITY ? 0.f : lse2 * kLn2;
        } else {
          const int outer_idx = split / S;
          float* po = p.part_o + (outer_idx * rows_all + grow) * D + col8 * 8;
          *reinterpret_cast<float4*>(po) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
          *reinterpret_cast<float4*>(po + 4) = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
          if (col8 == 0) p.part_lse[outer_idx * rows_all + grow] = lse2;
        }
      }
    }
  }
  if (S > 1) {
    // do not leave while a peer's copy may still be reading the staged rows
    if (merge_ok) merge_ok = mbar_wait(&s_bar[ACK_BAR], 0, s_abort);
    if (!merge_ok && tid == 0) atomicMax(&p.status[b], (int)SB_ERR_CUDA);
  }
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
  // the kernel orders itself after its predecessor with griddepcontrol.wait
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = test_knob("SB_NO_PDL") ? 1 : 2;
  return cfg;
}

template <int D>
static bool tc_prepare() {
  static PerDeviceOnce once;  // kernel attributes belong to a device: a process may drive several
  return once.run([]() {
    bool all = true;
#define SB_TC_PREPARE(cs_)                                                                                       \
  all = all && cudaFuncSetAttribute(attn_tc_kernel<D, cs_>, cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                                    (int)attn_tc_smem_bytes<D>()) == cudaSuccess;
    SB_TC_PREPARE(0) SB_TC_PREPARE(1) SB_TC_PREPARE(2) SB_TC_PREPARE(3) SB_TC_PREPARE(4)
    SB_TC_PREPARE(5) SB_TC_PREPARE(6) SB_TC_PREPARE(7) SB_TC_PREPARE(8) SB_TC_PREPARE(9) SB_TC_PREPARE(10)
#undef SB_TC_PREPARE
    // clusters of 9 and 10 CTAs are beyond the portable size: allowed per kernel
    all = all && cudaFuncSetAttribute(attn_tc_kernel<D, 0>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    all = all && cudaFuncSetAttribute(attn_tc_kernel<D, 9>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    all = all && cudaFuncSetAttribute(attn_tc_kernel<D, 10>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    if (!all) cudaGetLastError();
    return all;
  });
}

int attn_tc_max_active_clusters(int D, int cluster) {
  static PerDeviceInt cache[2][TC_MAX_CLUSTER + 1];
  const int di = D == 64 ? 0 : 1;
  if (cluster < 1 || cluster > TC_MAX_CLUSTER) return 0;
  return cache[di][cluster].get([&]() {
    int n = 0;
    cudaLaunchAttribute attr[2];
    cudaError_t e = cudaErrorUnknown;
    if (D == 64 && tc_prepare<64>()) {
      cudaLaunchConfig_t cfg = tc_config<64>(dim3(cluster * 64, 1, 1), cluster, nullptr, attr);
      e = cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<64, 0>, &cfg);
    } else if (D == 128 && tc_prepare<128>()) {
      cudaLaunchConfig_t cfg = tc_config<128>(dim3(cluster * 64, 1, 1), cluster, nullptr, attr);
      e = cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<128, 0>, &cfg);
    }
    if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
    return n;
  }, 0);
}

template <int D>
static sb_status launch_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  if (!tc_prepare<D>()) return SB_ERR_CUDA;
  cudaLaunchAttribute attr[2];
  cudaLaunchConfig_t cfg = tc_config<D>(grid, cluster, cs, attr);
  if (test_knob("SB_DEBUG"))
    fprintf(stderr, "[sb] attn_tc<%d> grid (%u,%u,%u) cluster %d outer %d: max active clusters %d\n", D, grid.x, grid.y,
            grid.z, cluster, p.outer, attn_tc_max_active_clusters(D, cluster));
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
  const bool fast = p.tb.page_size == 0 && q_tma && p.outer == 1 && !p.sort_seqs;
  cudaError_t le = cudaErrorInvalidValue;
  switch (fast ? cluster : 0) {
#define SB_TC_LAUNCH(cs_) \
  case cs_: le = cudaLaunchKernelEx(&cfg, attn_tc_kernel<D, cs_>, p, kmap, vmap, qmap, box_rows, q_tma); break;
    SB_TC_LAUNCH(0) SB_TC_LAUNCH(1) SB_TC_LAUNCH(2) SB_TC_LAUNCH(3) SB_TC_LAUNCH(4)
    SB_TC_LAUNCH(5) SB_TC_LAUNCH(6) SB_TC_LAUNCH(7) SB_TC_LAUNCH(8) SB_TC_LAUNCH(9) SB_TC_LAUNCH(10)
#undef SB_TC_LAUNCH
    default: break;
  }
  if (le != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

sb_status launch_attn_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  return p.tb.head_dim == 64 ? launch_tc<64>(p, grid, cluster, cs) : launch_tc<128>(p, grid, cluster, cs);
}

}  // namespace sb
