// sb_shift_project: the layer-wise shift between the drafter's decoder layers (Sec. 3.1): position
// k's state concatenated with position k-1's state of the same block, projected back by W_shift --
// a weight-streaming GEMM with a few dozen rows (one row per drafted position), HBM-bound on the
// weights (2 d x d_out bf16), on the tcgen05 tensor cores.
//
//   out[r] = W_a h[r] + W_b h[prev(r)],  W_shift = [W_a | W_b],  prev(r) = r - 1 inside a block, r at
//   its first position.  The shift is applied on the OUTPUT side: Z_a = H W_a^T and Z_b = H W_b^T
//   are plain GEMMs over the same H, and out[r] = Z_a[r] + Z_b[prev(r)].
//
//   shift_gemm_kernel  : operands swapped, so that the 128 rows of an MMA are output features and
//                        its N columns the (padded) positions: D[128 features][R] = W_tile H^T.
//                        One CTA per (feature tile, half a|b, K split): a TMA producer lane streams
//                        128 x 64 weight tiles and R x 64 activation slabs through a ring of stages
//                        (128-byte swizzle, mbarrier transaction counts), one lane issues the MMAs
//                        (accumulator in tensor memory), four warps write the fp32 partial
//                        [part][R][d_out] (feature-contiguous, coalesced).
//   shift_finish_kernel: sums the K splits, adds Z_b of the previous position, rounds to bf16.
//                        Launched as a programmatic dependent of the GEMM.
// (Reducing the parts of a feature tile inside a thread-block cluster over distributed shared memory,
// without a second kernel, was measured slower: 22.7 us against 17.1 us.)
#include <cstdlib>

#include "tc_common.cuh"

namespace sb {

constexpr int SG_THREADS = 192;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int SG_MAX_STAGES = 12;
constexpr int SG_BK = 64;        // K elements per stage (one 128-byte swizzled row)
constexpr int SG_BM = 128;       // output features per CTA
// The GEMM's CTAs report a wait that gave up by storing this value in the word after the partials;
// the finishing kernel turns it into status[0] and clears it, so no launch is spent on zeroing (a
// workspace whose stale contents equal this value by chance would raise one false error).
constexpr int SG_ERR_MAGIC = 0x5b0e7706;
__device__ inline void tma_load_2d(uint32_t smem_dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

// grid (d_out / 128, parts); part = half * ksplit + ks.  k_per = K elements of one split.
__global__ void __launch_bounds__(SG_THREADS, 1) shift_gemm_kernel(const __grid_constant__ CUtensorMap wmap,
                                                                   const __grid_constant__ CUtensorMap xmap,
                                                                   int n_rows, int r_pad, int d, int d_out, int ksplit,
                                                                   int k_per, int tmem_cols, int stages,
                                                                   float* __restrict__ part, int* __restrict__ err_flag) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* s_full = reinterpret_cast<uint64_t*>(base);        // [stages]
  uint64_t* s_empty = s_full + SG_MAX_STAGES;                   // [stages]
  uint64_t* s_done = s_empty + SG_MAX_STAGES;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(base + 256);
  volatile int* s_abort = reinterpret_cast<volatile int*>(base + 260);
  uint8_t* tiles = base + 1024;
  const int a_bytes = SG_BM * SG_BK * 2;                        // 16 KB
  const int b_bytes = r_pad * SG_BK * 2;
  const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int feat0 = blockIdx.x * SG_BM;
  const int part_id = blockIdx.y;
  const int half = part_id / ksplit, ks_id = part_id % ksplit;
  const int nk = k_per / SG_BK;
  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < stages; ++i) { mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 1); }
    mbar_init(s_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();     // the activations may come from the kernel just before
  pdl_release();  // the finishing kernel may start its prologue
  const uint32_t tmem = *s_tmem;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      for (int ks = 0; ks < nk && ok; ++ks) {
        const int st = ks % stages;
        if (ks >= stages) ok = mbar_wait(&s_empty[st], ((ks / stages) - 1) & 1, s_abort);
        if (!ok) break;
        const uint32_t sa = smem_u32(tiles + (size_t)st * stage_bytes);
        const int k0 = ks_id * k_per + ks * SG_BK;
        mbar_expect_tx(&s_full[st], (uint32_t)(a_bytes + b_bytes));
        tma_load_2d(sa, &wmap, half * d + k0, feat0, &s_full[st]);   // weights: [128 features][64 k]
        tma_load_2d(sa + a_bytes, &xmap, k0, 0, &s_full[st]);        // activations: [r_pad rows][64 k]
      }
      if (!ok) *err_flag = SG_ERR_MAGIC;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t hi = tc_desc_hi(1024);
      const uint32_t idesc = tc_idesc(SG_BM, r_pad, 0);
      bool ok = true;
      for (int ks = 0; ks < nk && ok; ++ks) {
        const int st = ks % stages;
        ok = mbar_wait(&s_full[st], (ks / stages) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(tiles + (size_t)st * stage_bytes);
        const uint32_t a_lo = tc_desc_lo(sa, 16), b_lo = tc_desc_lo(sa + a_bytes, 16);
#pragma unroll
        for (int k4 = 0; k4 < SG_BK / 16; ++k4)
          tc_mma_h(tmem, a_lo + ((k4 * 32) >> 4), b_lo + ((k4 * 32) >> 4), hi, idesc, (ks > 0 || k4 > 0) ? 1u : 0u);
        tc_commit(&s_empty[st]);
      }
      if (ok) tc_commit(s_done);
      if (!ok) *err_flag = SG_ERR_MAGIC;
    }
  } else {
    // ------------------------------------------------------------------ epilogue: fp32 partial, feature-contiguous
    const bool ok = mbar_wait(s_done, 0, s_abort);
    tc_fence_after();
    if (ok) {
      const int q = warp & 3;                                   // TMEM lane quarter this warp may read
      const int feat = feat0 + q * 32 + lane;
      const uint32_t lane_base = ((uint32_t)(q * 32)) << 16;
      float* dst = part + (size_t)part_id * n_rows * d_out + feat;
      for (int c0 = 0; c0 < r_pad; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(tmem + lane_base + c0, v);
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (c0 + i < n_rows) dst[(size_t)(c0 + i) * d_out] = __uint_as_float(v[i]);
      }
    } else if (lane == 0) {
      *err_flag = SG_ERR_MAGIC;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols));
  }
}

// out[r][f] = bf16( sum_ks part[0 * ksplit + ks][r][f] + sum_ks part[1 * ksplit + ks][prev(r)][f] ), 4 features
// per thread; thread 0 of the grid turns the GEMM's error word into status[0] and clears it.
__global__ void __launch_bounds__(256) shift_finish_kernel(const float* __restrict__ part, int n_rows, int d_out,
                                                           int ksplit, int halves, int block_k, bf16* __restrict__ out,
                                                           int* __restrict__ err_word, int* __restrict__ status) {
  const int f4 = blockIdx.x * blockDim.x + threadIdx.x;  // group of 4 features
  const int r = blockIdx.y;
  pdl_wait();  // the partials are complete from here on
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    status[0] = *err_word == SG_ERR_MAGIC ? (int)SB_ERR_CUDA : (int)SB_OK;
    *err_word = 0;
  }
  if (f4 * 4 >= d_out) return;
  const int prev = (block_k > 0 && r % block_k != 0) ? r - 1 : r;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int h = 0; h < halves; ++h) {
    const int row = h == 0 ? r : prev;
    for (int ks = 0; ks < ksplit; ++ks) {
      const float4 v = *reinterpret_cast<const float4*>(part + ((size_t)(h * ksplit + ks) * n_rows + row) * d_out + f4 * 4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
  }
  uint2 o;
  o.x = pack_bf16(acc.x, acc.y);
  o.y = pack_bf16(acc.z, acc.w);
  *reinterpret_cast<uint2*>(out + (size_t)r * d_out + f4 * 4) = o;
}

struct ShiftPlan {
  int halves, ksplit, k_per, r_pad, tmem_cols, stages;
  size_t smem, ws_bytes;
};

static bool shift_plan(int n_rows, int d, int d_out, int block_k, ShiftPlan* pl) {
  if (n_rows < 1 || n_rows > 128 || d < SG_BK || d % SG_BK != 0 || d_out < SG_BM || d_out % SG_BM != 0 || block_k < 0)
    return false;
  pl->halves = block_k > 0 ? 2 : 1;
  const int tiles = d_out / SG_BM, ksteps = d / SG_BK;
  pl->r_pad = ((n_rows + 15) / 16) * 16;
  int cols = 32;
  while (cols < pl->r_pad) cols *= 2;
  pl->tmem_cols = cols;
  const size_t stage = (size_t)SG_BM * SG_BK * 2 + (((size_t)pl->r_pad * SG_BK * 2 + 1023) & ~(size_t)1023);
  // Enough CTAs and bytes in flight to pull the weights at HBM rate.  With few rows a stage is small:
  // two CTAs share an SM (about 110 KB each) and the K dimension is split until about 256 CTAs
  // exist (measured 17.1 us against 18.3 us for 128 CTAs with deeper rings on 4096 x 8192 weights);
  // with many rows one CTA per SM and a ring as deep as shared memory allows.
  const bool two_per_sm = stage <= 24 * 1024;
  int cta_target = two_per_sm ? 320 : 160;
  size_t budget = two_per_sm ? 110 * 1024 : 200 * 1024;
  if (const char* e = getenv("SB_SHIFT_CTAS")) cta_target = atoi(e);
  if (const char* e = getenv("SB_SHIFT_SMEM_KB")) budget = (size_t)atoi(e) * 1024;
  int ks = 1;
  while (ks < 8 && tiles * pl->halves * ks * 2 <= cta_target && ksteps % (ks * 2) == 0) ks *= 2;
  pl->ksplit = ks;
  pl->k_per = d / ks;
  int stages = (int)((budget - 2048) / stage);
  if (stages > SG_MAX_STAGES) stages = SG_MAX_STAGES;
  if (stages > pl->k_per / SG_BK) stages = pl->k_per / SG_BK;
  if (stages < 1) return false;
  pl->stages = stages;
  pl->smem = 1024 + 1024 + stages * stage;
  pl->ws_bytes = (size_t)pl->halves * ks * n_rows * d_out * sizeof(float);
  return true;
}

static bool make_2d_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {(cuuint32_t)SG_BK, box_rows};
  const cuuint32_t elem[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace sb

extern "C" size_t sb_shift_project_workspace_bytes(int32_t n_rows, int32_t d, int32_t d_out, int32_t block_k) {
  sb::ShiftPlan pl;
  if (!sb::shift_plan(n_rows, d, d_out, block_k, &pl)) return 0;
  return ((pl.ws_bytes + 255) & ~(size_t)255) + 256;  // partials + the error word
}

extern "C" sb_status sb_shift_project(const void* h, const void* w, int32_t n_rows, int32_t d, int32_t d_out,
                                      int32_t block_k, void* out, void* workspace, size_t workspace_bytes,
                                      int32_t* status, void* stream) {
  using namespace sb;
  if (!h || !w || !out || !status) return SB_ERR_INVALID_ARG;
  ShiftPlan pl;
  if (!shift_plan(n_rows, d, d_out, block_k, &pl)) return SB_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(h) & 15) || (reinterpret_cast<uintptr_t>(w) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 7))
    return SB_ERR_INVALID_ARG;
  const size_t need = sb_shift_project_workspace_bytes(n_rows, d, d_out, block_k);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  static bool prepared = false;
  if (!prepared) {
    if (cudaFuncSetAttribute(shift_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) {
      cudaGetLastError();
      return SB_ERR_CUDA;
    }
    prepared = true;
  }
  if (pl.smem > 200 * 1024) return SB_ERR_UNSUPPORTED;
  CUtensorMap wmap, xmap;
  if (!make_2d_map(&wmap, w, (uint64_t)pl.halves * d, (uint64_t)d_out, SG_BM) ||
      !make_2d_map(&xmap, h, (uint64_t)d, (uint64_t)n_rows, (uint32_t)pl.r_pad))
    return SB_ERR_CUDA;
  int* err_word = reinterpret_cast<int*>(static_cast<char*>(workspace) + ((pl.ws_bytes + 255) & ~(size_t)255));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d_out / SG_BM, pl.halves * pl.ksplit);
  cfg.blockDim = dim3(SG_THREADS);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the kernel orders itself (pdl_wait)
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = getenv("SB_NO_PDL") ? 0 : 1;
  if (cudaLaunchKernelEx(&cfg, shift_gemm_kernel, wmap, xmap, (int)n_rows, pl.r_pad, (int)d, (int)d_out, pl.ksplit,
                         pl.k_per, pl.tmem_cols, pl.stages, static_cast<float*>(workspace), err_word) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  return launch_dependent(shift_finish_kernel, dim3(ceil_div(d_out / 4, 256), n_rows), dim3(256), cs,
                          static_cast<const float*>(workspace), (int)n_rows, (int)d_out, pl.ksplit, pl.halves,
                          (int)block_k, static_cast<bf16*>(out), err_word, status);
}
