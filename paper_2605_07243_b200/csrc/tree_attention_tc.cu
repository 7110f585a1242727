// Tree-masked split-KV attention on the 5th-generation tensor cores (tcgen05 + TMEM), sm_100a.
//
// One CTA owns a 128-row query tile (rows = (node, head-in-group) pairs of one KV head: the tile
// is the M = 128 dimension of the MMA and one row per TMEM lane) and a chunk of the sequence's
// keys, walked in blocks of up to 128 keys:
//
//   loader warps   one thread per operand issues TMA tile loads (cp.async.bulk.tensor, 128-byte swizzle,
//                  no multicast) of the K and V blocks straight into the shared-memory layouts the
//                  tensor core reads (K, Q, P: K-major; V: MN-major), 2 stages each, completion by
//                  mbarrier transaction count; paged caches load one box per page piece.  V rows past
//                  the end of the sequence are zeroed (P is 0 there, but 0 * garbage must stay 0).
//                  The Q tile is one TMA box {64 columns, G heads, 128/G nodes} per column half when
//                  G divides 128, else a 16-byte cp.async gather by the softmax warps;
//   MMA warp       one thread issues  S_j = Q K_j^T  (tcgen05.mma, fp32 accumulator in TMEM, two S
//                  buffers) and  O += P_j V_j  with P_j read from TMEM and O accumulated in TMEM;
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
// through distributed shared memory exactly as in the mma.sync kernel.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>

#include "attention_common.cuh"

namespace sb {

constexpr int TC_BM = 128;           // rows per CTA
constexpr int TC_BN = 128;           // keys per block
constexpr int TC_SOFTMAX_THREADS = 256;  // warps 0-3: columns [0,64) of a block, warps 4-7: [64,128)
constexpr int TC_MMA_WARP = 8;
constexpr int TC_KLOAD_WARP = 9;     // lane 0 issues the Q and K loads
constexpr int TC_VLOAD_WARP = 10;    // lane 0 issues the V loads; the warp zeroes rows past the sequence
constexpr int TC_THREADS = 384;      // 12 warps (warp 11 only takes part in the barriers)
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_SMALL_BYTES = 8192; // ancestor masks, parents, barriers, softmax exchange
constexpr int TC_MERGE_SLOTS = TC_BM + 8;  // receive slots: S * ceil(128 / S) <= 135 for S <= 8

enum TcBar { K_FULL0, K_FULL1, K_EMPTY0, K_EMPTY1, V_FULL0, V_FULL1, V_EMPTY0, V_EMPTY1, S_FULL0, S_FULL1,
             S_EMPTY0, S_EMPTY1, P_FULL, PV_FULL, V_TMA0, V_TMA1, Q_FULL, MERGE_BAR, ACK_BAR, TC_NUM_BARS };

template <int D>
constexpr size_t attn_tc_smem_bytes() {
  // small region + Q + 2 K stages + 2 V stages + the merge receive buffer (bf16 rows + m, l), plus
  // slack to align the tiles to 1024 bytes
  return 1024 + TC_SMALL_BYTES + (size_t)TC_BM * D * 2 + 4 * (size_t)TC_BN * D * 2 + (size_t)TC_MERGE_SLOTS * (D * 2 + 16);
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
// Shared-memory matrix descriptor, 128-byte swizzle: start address (bits 0-13), leading (16-29) and
// stride (32-45) byte offsets, all in 16-byte units, descriptor version 1 (bit 46), layout type 2
// (bits 61-63) -- kept as two 32-bit halves.  Only the low half depends on the address, and a byte
// offset inside the tile is added to it as offset >> 4 (shared memory addresses stay below 2^18,
// so the 14-bit field cannot overflow): the issuing thread forms each operand with one add.
__device__ inline uint32_t tc_desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr >> 4) & 0x3FFF) | (((lbo_bytes >> 4) & 0x3FFF) << 16);
}
__device__ inline uint32_t tc_desc_hi(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFF) | (1u << 14) | (2u << 29);
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
__device__ inline void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// TMA tile load of one box of a rank-4 tensor (d, kv head, row in page, page) into shared memory.
__device__ inline void tma_load_4d(uint32_t smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                   uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ inline void tma_load_3d(uint32_t smem_dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Address of `smem_addr` (a shared::cta address of this CTA's window) in CTA `rank` of the cluster.
__device__ inline uint32_t mapa_u32(uint32_t smem_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// Bulk asynchronous copy from this CTA's shared memory into a cluster peer's; the bytes are
// credited to the peer's mbarrier.  Sizes and addresses are multiples of 16 bytes.
__device__ inline void dsmem_bulk_copy(uint32_t dst_cluster_addr, uint32_t src_cta_addr, uint32_t bytes,
                                       uint32_t mbar_cluster_addr) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   dst_cluster_addr),
               "r"(src_cta_addr), "r"(bytes), "r"(mbar_cluster_addr)
               : "memory");
}
// Arrive on an mbarrier that lives in a cluster peer's shared memory.
__device__ inline void mbar_arrive_remote(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ inline void softmax_group_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// 32 consecutive 32-bit columns of this thread's TMEM lane <- registers.
__device__ inline void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ inline void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Two 32-column loads in flight, one wait.
__device__ inline void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
#pragma unroll
  for (int h = 0; h < 2; ++h)
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        : "=r"(r[32 * h + 0]), "=r"(r[32 * h + 1]), "=r"(r[32 * h + 2]), "=r"(r[32 * h + 3]), "=r"(r[32 * h + 4]),
          "=r"(r[32 * h + 5]), "=r"(r[32 * h + 6]), "=r"(r[32 * h + 7]), "=r"(r[32 * h + 8]), "=r"(r[32 * h + 9]),
          "=r"(r[32 * h + 10]), "=r"(r[32 * h + 11]), "=r"(r[32 * h + 12]), "=r"(r[32 * h + 13]), "=r"(r[32 * h + 14]),
          "=r"(r[32 * h + 15]), "=r"(r[32 * h + 16]), "=r"(r[32 * h + 17]), "=r"(r[32 * h + 18]), "=r"(r[32 * h + 19]),
          "=r"(r[32 * h + 20]), "=r"(r[32 * h + 21]), "=r"(r[32 * h + 22]), "=r"(r[32 * h + 23]), "=r"(r[32 * h + 24]),
          "=r"(r[32 * h + 25]), "=r"(r[32 * h + 26]), "=r"(r[32 * h + 27]), "=r"(r[32 * h + 28]), "=r"(r[32 * h + 29]),
          "=r"(r[32 * h + 30]), "=r"(r[32 * h + 31])
        : "r"(taddr + 32 * h));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// D[tmem] (+)= A * B, bf16 inputs, fp32 accumulate, issued by one thread; the shared memory
// descriptors are given as (low, high) halves.  First form: A and B in shared memory.  Second form:
// A is read from tensor memory (row = lane, bf16 pairs along columns).
__device__ inline void tc_mma_h(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t hi, uint32_t idesc,
                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 ad, bd;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 ad, {%1, %3};\n\tmov.b64 bd, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %4, p;\n\t}\n" ::"r"(d_tmem),
      "r"(alo), "r"(blo), "r"(hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ inline void tc_mma_ts_h(uint32_t d_tmem, uint32_t a_tmem, uint32_t blo, uint32_t hi, uint32_t idesc,
                                   uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 bd;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 bd, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}\n" ::"r"(d_tmem),
      "r"(a_tmem), "r"(blo), "r"(hi), "r"(idesc), "r"(accumulate)
      : "memory");
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
__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const AttnParams p,
                                                                const __grid_constant__ CUtensorMap kmap,
                                                                const __grid_constant__ CUtensorMap vmap,
                                                                const __grid_constant__ CUtensorMap qmap,
                                                                const int box_rows, const int q_tma) {
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
  const int S = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int split = blockIdx.x;
  const int Hq = p.tb.n_q_heads, G = p.G;
  // row tiles of one (sequence, KV head) are neighbours in launch order: they share its K/V through L2
  const int g = blockIdx.y / p.row_tiles, tile = blockIdx.y % p.row_tiles;
  const int b = blockIdx.z;
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
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const SeqPre pre = plan_lengths(p, b);
  const int rows_total = pre.info.nq * G;
  const int row0 = tile * TC_BM;
  if (!pre.can_write || row0 >= rows_total) {  // uniform over the cluster
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
    if (p.tb.page_size == 0) return;
    const int nj = min(TC_BN, chunk_keys - j * TC_BN);
    const int k0 = key_begin + j * TC_BN;
    const int pieces = ceil_div(nj, box_rows);
#pragma unroll 1
    for (int i = 0; i < MAX_PIECES; ++i)
      if (i < pieces) pg[i] = p.tb.page_table[(long long)b * p.tb.max_pages + (k0 + i * box_rows) / p.tb.page_size];
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
    if (q_tma) {
      mbar_expect_tx(&s_bar[Q_FULL], (uint32_t)(TC_BM * D * 2));
#pragma unroll
      for (int h = 0; h < D / 64; ++h)
        tma_load_3d(smem_u32(sQ) + h * (TC_BM * 128), &qmap, h * 64, g * G, pre.info.q_off + tile * (TC_BM / G),
                    &s_bar[Q_FULL]);
    }
    issue_block(0, &kmap, smem_u32(sK), &s_bar[K_FULL0]);
    if (nb > 1) issue_block(1, &kmap, smem_u32(sK) + TILE_BYTES, &s_bar[K_FULL1]);
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
        cp_async_16_tc(qd + sw128_chunk_off(r, ch, TC_BM), p.q + (valid ? off : 0), valid ? 16 : 0);
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
#pragma unroll
          for (int c = 0; c < DH / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem_o + lane_base + half * DH + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st32(tmem_o + lane_base + half * DH + c * 32, r);
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
  tc_fence_before();
  __syncthreads();  // every role is done: no async access to Q/K/V stages is in flight any more
  if (warp == TC_MMA_WARP) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS));
  }
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
  if (S > 1) {
    fence_async_smem();  // the staged rows are read by the bulk-copy engine
    __syncthreads();
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
    // every source's slice has landed here: tell each source that its staging rows are free
    if (tid < S) mbar_arrive_remote(mapa_u32(smem_u32(&s_bar[ACK_BAR]), tid));
  } else {
    __syncthreads();
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
      float w[8];
      uint4 raw[8];
      float M = -INFINITY, Lsum = 0.f;
      {
        float mc[8], lc[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint8_t* rowp = src + ((size_t)(c < S ? c : 0) * rows_per + t) * ROWB;
          mc[c] = c < S ? *reinterpret_cast<const float*>(rowp + D * 2) : -INFINITY;
          lc[c] = c < S ? *reinterpret_cast<const float*>(rowp + D * 2 + 4) : 0.f;
          raw[c] = (c < S && has_cols) ? *reinterpret_cast<const uint4*>(rowp + col8 * 16) : make_uint4(0u, 0u, 0u, 0u);
          M = fmaxf(M, mc[c]);
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          w[c] = mc[c] == -INFINITY ? 0.f : fast_exp2(mc[c] - M) * lc[c];  // 2^(m_c - M) * l_c
          Lsum += w[c];
        }
      }
      const float inv = Lsum > 0.f ? __fdividef(1.f, Lsum) : 0.f;
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
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
      if (has_cols) {
        if (p.outer == 1) {
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

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
    else
      cudaGetLastError();
  }
  return fn;
}

// Rank-4 view (d, kv head, row, page) of a K or V cache; a contiguous cache is one "page" of
// kv_capacity rows per sequence.  Box = 64 columns x 1 head x box_rows rows, 128-byte swizzle,
// out-of-range rows read as zero.
static bool make_kv_map(CUtensorMap* map, const sb_tree_batch& tb, const void* cache, int box_rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t D = (cuuint64_t)tb.head_dim, H = (cuuint64_t)tb.n_kv_heads;
  const cuuint64_t rows = tb.page_size == 0 ? (cuuint64_t)tb.kv_capacity : (cuuint64_t)tb.page_size;
  const cuuint64_t pages = tb.page_size == 0 ? (cuuint64_t)tb.batch : (cuuint64_t)tb.num_pages;
  const cuuint64_t dims[4] = {D, H, rows, pages};
  const cuuint64_t strides[3] = {D * 2, H * D * 2, rows * H * D * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(cache), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Rank-3 view (d, query head, query row) of Q; box = 64 columns x G heads x 128/G rows lands in
// shared memory as the tile's 128 packed (node, head-in-group) rows.
static bool make_q_map(CUtensorMap* map, const AttnParams& p) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t D = (cuuint64_t)p.tb.head_dim, H = (cuuint64_t)p.tb.n_q_heads;
  const cuuint64_t dims[3] = {D, H, (cuuint64_t)p.total_q};
  const cuuint64_t strides[2] = {D * 2, H * D * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)p.G, (cuuint32_t)(TC_BM / p.G)};
  const cuuint32_t elem[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(p.q), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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
  cfg.numAttrs = getenv("SB_NO_PDL") ? 1 : 2;
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
    cudaLaunchAttribute attr[2];
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
  cudaLaunchAttribute attr[2];
  cudaLaunchConfig_t cfg = tc_config<D>(grid, cluster, cs, attr);
  if (getenv("SB_DEBUG"))
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
  if (cudaLaunchKernelEx(&cfg, attn_tc_kernel<D>, p, kmap, vmap, qmap, box_rows, q_tma) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

sb_status launch_attn_tc(const AttnParams& p, dim3 grid, int cluster, cudaStream_t cs) {
  return p.tb.head_dim == 64 ? launch_tc<64>(p, grid, cluster, cs) : launch_tc<128>(p, grid, cluster, cs);
}

}  // namespace sb
