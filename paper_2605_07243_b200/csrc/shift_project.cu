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

// grid (d_out / 128, parts); part = half * ksplit + ks.  k_per = K elements of one split.  "half" is the
// segment of the concatenated input (a | b of the shift; context | embedding | query of the fused
// input): its weights start at column half * d and its activations at row half * x_seg_rows of xmap
// (0 when every segment multiplies the same rows).
__global__ void __launch_bounds__(SG_THREADS, 1) shift_gemm_kernel(const __grid_constant__ CUtensorMap wmap,
                                                                   const __grid_constant__ CUtensorMap xmap,
                                                                   int n_rows, int r_pad, int d, int d_out, int ksplit,
                                                                   int k_per, int tmem_cols, int stages, int x_seg_rows,
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
  pdl_release();  // the finishing kernel may start its prologue
  const uint32_t tmem = *s_tmem;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The weights are requested before the dependency wait: they are model constants, never the
    // output of the kernel just before, so the first ring of weight tiles streams while that
    // kernel (the normalisation, or the previous call's finishing kernel) is still running.  The
    // activations, which may be its output, are requested after the wait.
    if (lane == 0) {
      const int pre = stages < nk ? stages : nk;
      for (int ks = 0; ks < pre; ++ks) {
        mbar_expect_tx(&s_full[ks], (uint32_t)(a_bytes + b_bytes));
        tma_load_2d(smem_u32(tiles + (size_t)ks * stage_bytes), &wmap, half * d + ks_id * k_per + ks * SG_BK, feat0,
                    &s_full[ks]);
      }
      pdl_wait();
      for (int ks = 0; ks < pre; ++ks)
        tma_load_2d(smem_u32(tiles + (size_t)ks * stage_bytes) + a_bytes, &xmap, ks_id * k_per + ks * SG_BK,
                    half * x_seg_rows, &s_full[ks]);
      bool ok = true;
      for (int ks = pre; ks < nk && ok; ++ks) {
        const int st = ks % stages;
        ok = mbar_wait(&s_empty[st], ((ks / stages) - 1) & 1, s_abort);
        if (!ok) break;
        const uint32_t sa = smem_u32(tiles + (size_t)st * stage_bytes);
        const int k0 = ks_id * k_per + ks * SG_BK;
        mbar_expect_tx(&s_full[st], (uint32_t)(a_bytes + b_bytes));
        tma_load_2d(sa, &wmap, half * d + k0, feat0, &s_full[st]);   // weights: [128 features][64 k]
        tma_load_2d(sa + a_bytes, &xmap, k0, half * x_seg_rows, &s_full[st]);  // activations: [r_pad rows][64 k]
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
      if (!ok) {
        pdl_wait();
        *err_flag = SG_ERR_MAGIC;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: fp32 partial, feature-contiguous
    const bool ok = mbar_wait(s_done, 0, s_abort);
    tc_fence_after();
    pdl_wait();  // the partials may still be read by the previous call's finishing kernel (long done by now)
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
  pdl_release();  // the next call's kernels may set themselves up (and request their weights)
  pdl_wait();     // the partials are complete from here on
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

// n_rows = columns of the MMA (rows of the activation operand), segments = pieces of the concatenated input.
static bool shift_plan(int n_rows, int d, int d_out, int segments, ShiftPlan* pl, int split_like = 0) {
  if (n_rows < 1 || n_rows > 128 || d < SG_BK || d % SG_BK != 0 || d_out < SG_BM || d_out % SG_BM != 0 || segments < 1 ||
      segments > 3)
    return false;
  pl->halves = segments;
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
  if (const char* e = test_knob("SB_SHIFT_CTAS")) cta_target = atoi(e);
  if (const char* e = test_knob("SB_SHIFT_SMEM_KB")) budget = (size_t)atoi(e) * 1024;
  int ks = 1;
  // split_like: choose the K split as a problem of that many segments would (the same partial sums, hence the
  // same bits, whether or not a cached segment is left out)
  const int split_segments = split_like > 0 ? split_like : pl->halves;
  while (ks < 8 && tiles * split_segments * ks * 2 <= cta_target && ksteps % (ks * 2) == 0) ks *= 2;
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

// Launches the GEMM of a plan (programmatic dependent of whatever precedes it in the stream).
static sb_status launch_shift_gemm(const ShiftPlan& pl, const CUtensorMap& wmap, const CUtensorMap& xmap, int n_cols,
                                   int d, int d_out, int x_seg_rows, float* part, int* err_word, cudaStream_t cs) {
  static PerDeviceOnce once;
  if (!once.run([]() {
        const bool ok = cudaFuncSetAttribute(shift_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) == cudaSuccess;
        if (!ok) cudaGetLastError();
        return ok;
      }))
    return SB_ERR_CUDA;
  if (pl.smem > 200 * 1024) return SB_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d_out / SG_BM, pl.halves * pl.ksplit);
  cfg.blockDim = dim3(SG_THREADS);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the kernel orders itself (pdl_wait)
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = test_knob("SB_NO_PDL") ? 0 : 1;
  if (cudaLaunchKernelEx(&cfg, shift_gemm_kernel, wmap, xmap, n_cols, pl.r_pad, d, d_out, pl.ksplit, pl.k_per,
                         pl.tmem_cols, pl.stages, x_seg_rows, part, err_word) != cudaSuccess) {
    cudaGetLastError();
    return SB_ERR_CUDA;
  }
  return launch_check();
}

// ---- the drafter's fused per-position input (Sec. 3.1, the equation for h^(0)) ----------------------
//
//   h0[s * K + k] = W_fuse [ norm(c_s), norm(e_s), norm(q_k) ] = Z_c[s] + Z_e[s] + Z_q[k]:
// the context feature and the embedding are shared by the K positions of a block (the prefix
// broadcast) and the query term does not depend on the start, so the GEMM has max(S, K) columns, not
// S * K, and each third of W_fuse is streamed once.  Z_q is the same for every call with the same
// weights: the caller may keep it (q_term) and have later calls stream two thirds of W_fuse only.

// Row (seg, i) of X [3][r_pad][d]: norm(x)[j] = g[j] x[j] / sqrt(mean x^2 + eps) in bf16; rows past the
// segment's count are zero.  One CTA per row.
__global__ void __launch_bounds__(256) fuse_norm_kernel(const bf16* __restrict__ c, const bf16* __restrict__ e,
                                                        const bf16* __restrict__ q, const float* __restrict__ gain_c,
                                                        const float* __restrict__ gain_e,
                                                        const float* __restrict__ gain_q, float eps, int n_starts,
                                                        int block_k, int d, int r_pad, int segments,
                                                        bf16* __restrict__ x) {
  __shared__ float s_part[8];
  const int seg = blockIdx.x / r_pad, i = blockIdx.x % r_pad;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_release();  // the GEMM may set itself up and request weights; it waits for this grid before it loads X
  pdl_wait();     // the inputs may come from the kernel just before
  const int count = seg == 2 ? block_k : n_starts;
  bf16* dst = x + ((size_t)seg * r_pad + i) * d;
  if (i >= count) {
    for (int j = tid * 8; j < d; j += 256 * 8) *reinterpret_cast<uint4*>(dst + j) = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const bf16* src = (seg == 0 ? c : seg == 1 ? e : q) + (size_t)i * d;
  const float* g = seg == 0 ? gain_c : seg == 1 ? gain_e : gain_q;
  float ss = 0.f;
  for (int j = tid * 8; j < d; j += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(src + j);
    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float a = __uint_as_float(w4[t] << 16), b = __uint_as_float(w4[t] & 0xffff0000u);
      ss += a * a + b * b;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) s_part[warp] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += s_part[w];
  const float inv = rsqrtf(tot / (float)d + eps);
  for (int j = tid * 8; j < d; j += 256 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(src + j);
    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
    float y[8];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      y[2 * t] = __uint_as_float(w4[t] << 16) * inv;
      y[2 * t + 1] = __uint_as_float(w4[t] & 0xffff0000u) * inv;
    }
    if (g) {
      const float4 g0 = *reinterpret_cast<const float4*>(g + j), g1 = *reinterpret_cast<const float4*>(g + j + 4);
      y[0] *= g0.x; y[1] *= g0.y; y[2] *= g0.z; y[3] *= g0.w;
      y[4] *= g1.x; y[5] *= g1.y; y[6] *= g1.z; y[7] *= g1.w;
    }
    uint4 o;
    o.x = pack_bf16(y[0], y[1]); o.y = pack_bf16(y[2], y[3]); o.z = pack_bf16(y[4], y[5]); o.w = pack_bf16(y[6], y[7]);
    *reinterpret_cast<uint4*>(dst + j) = o;
  }
}

// out[s * K + k][f] = bf16( (Z_c[s][f] + Z_e[s][f]) + Z_q[k][f] ), each Z the sum of its K splits; Z_q is
// read from q_term when the caller holds it, else formed here and (by the rows of start 0) stored there.
__global__ void __launch_bounds__(256) fuse_finish_kernel(const float* __restrict__ part, int n_cols, int d_out,
                                                          int ksplit, int block_k, int q_term_valid,
                                                          float* __restrict__ q_term, bf16* __restrict__ out,
                                                          int* __restrict__ err_word, int* __restrict__ status) {
  const int f4 = blockIdx.x * blockDim.x + threadIdx.x;  // group of 4 features
  const int r = blockIdx.y, s = r / block_k, k = r % block_k;
  pdl_release();  // the next call's kernels may set themselves up (and request their weights)
  pdl_wait();     // the partials are complete from here on
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    status[0] = *err_word == SG_ERR_MAGIC ? (int)SB_ERR_CUDA : (int)SB_OK;
    *err_word = 0;
  }
  if (f4 * 4 >= d_out) return;
  auto seg_sum = [&](int seg, int row) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int ks = 0; ks < ksplit; ++ks) {
      const float4 v = *reinterpret_cast<const float4*>(part + ((size_t)(seg * ksplit + ks) * n_cols + row) * d_out + f4 * 4);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    return a;
  };
  const float4 zc = seg_sum(0, s), ze = seg_sum(1, s);
  float4 zq;
  if (q_term_valid) {
    zq = *reinterpret_cast<const float4*>(q_term + (size_t)k * d_out + f4 * 4);
  } else {
    zq = seg_sum(2, k);
    if (s == 0 && q_term) *reinterpret_cast<float4*>(q_term + (size_t)k * d_out + f4 * 4) = zq;
  }
  uint2 o;
  o.x = pack_bf16((zc.x + ze.x) + zq.x, (zc.y + ze.y) + zq.y);
  o.y = pack_bf16((zc.z + ze.z) + zq.z, (zc.w + ze.w) + zq.w);
  *reinterpret_cast<uint2*>(out + (size_t)r * d_out + f4 * 4) = o;
}

struct FusePlan {
  ShiftPlan gemm;
  int n_cols, segments;
  size_t part_bytes, x_off, total;
};

static bool fuse_plan(int n_starts, int block_k, int d, int d_out, int q_term_valid, FusePlan* fp) {
  if (n_starts < 1 || n_starts > 128 || block_k < 1 || block_k > 128 || n_starts * block_k > 65535) return false;
  fp->n_cols = n_starts > block_k ? n_starts : block_k;
  fp->segments = q_term_valid ? 2 : 3;
  if (!shift_plan(fp->n_cols, d, d_out, fp->segments, &fp->gemm, 2)) return false;
  fp->part_bytes = (fp->gemm.ws_bytes + 255) & ~(size_t)255;
  fp->x_off = fp->part_bytes + 256;  // the error word sits between the partials and X
  fp->total = fp->x_off + (((size_t)3 * fp->gemm.r_pad * d * sizeof(bf16) + 255) & ~(size_t)255);
  return true;
}

}  // namespace sb

extern "C" size_t sb_shift_project_workspace_bytes(int32_t n_rows, int32_t d, int32_t d_out, int32_t block_k) {
  sb::ShiftPlan pl;
  if (block_k < 0 || !sb::shift_plan(n_rows, d, d_out, block_k > 0 ? 2 : 1, &pl)) return 0;
  return ((pl.ws_bytes + 255) & ~(size_t)255) + 256;  // partials + the error word
}

extern "C" sb_status sb_shift_project(const void* h, const void* w, int32_t n_rows, int32_t d, int32_t d_out,
                                      int32_t block_k, void* out, void* workspace, size_t workspace_bytes,
                                      int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_shift_project");
  using namespace sb;
  if (!h || !w || !out || !status) return SB_ERR_INVALID_ARG;
  ShiftPlan pl;
  if (block_k < 0 || !shift_plan(n_rows, d, d_out, block_k > 0 ? 2 : 1, &pl)) return SB_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(h) & 15) || (reinterpret_cast<uintptr_t>(w) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 7))
    return SB_ERR_INVALID_ARG;
  const size_t need = sb_shift_project_workspace_bytes(n_rows, d, d_out, block_k);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  CUtensorMap wmap, xmap;
  if (!make_2d_map(&wmap, w, (uint64_t)pl.halves * d, (uint64_t)d_out, SG_BM) ||
      !make_2d_map(&xmap, h, (uint64_t)d, (uint64_t)n_rows, (uint32_t)pl.r_pad))
    return SB_ERR_CUDA;
  int* err_word = reinterpret_cast<int*>(static_cast<char*>(workspace) + ((pl.ws_bytes + 255) & ~(size_t)255));
  sb_status st = launch_shift_gemm(pl, wmap, xmap, n_rows, d, d_out, 0, static_cast<float*>(workspace), err_word, cs);
  if (st != SB_OK) return st;
  return launch_dependent(shift_finish_kernel, dim3(ceil_div(d_out / 4, 256), n_rows), dim3(256), cs,
                          static_cast<const float*>(workspace), (int)n_rows, (int)d_out, pl.ksplit, pl.halves,
                          (int)block_k, static_cast<bf16*>(out), err_word, status);
}

extern "C" size_t sb_fuse_project_workspace_bytes(int32_t n_starts, int32_t block_k, int32_t d, int32_t d_out,
                                                  int32_t q_term_valid) {
  sb::FusePlan fp;
  if (!sb::fuse_plan(n_starts, block_k, d, d_out, q_term_valid, &fp)) return 0;
  return fp.total;
}

extern "C" sb_status sb_fuse_project(const void* c, const void* e, const void* q, const float* gain_c,
                                     const float* gain_e, const float* gain_q, float eps, const void* w,
                                     int32_t n_starts, int32_t block_k, int32_t d, int32_t d_out, float* q_term,
                                     int32_t q_term_valid, void* out, void* workspace, size_t workspace_bytes,
                                     int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_fuse_project");
  using namespace sb;
  if (!c || !e || !q || !w || !out || !status || (q_term_valid && !q_term) || !(eps >= 0.f)) return SB_ERR_INVALID_ARG;
  FusePlan fp;
  if (!fuse_plan(n_starts, block_k, d, d_out, q_term_valid, &fp)) return SB_ERR_UNSUPPORTED;
  auto misaligned = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
  if (misaligned(c, 16) || misaligned(e, 16) || misaligned(q, 16) || misaligned(w, 16) || misaligned(out, 8) ||
      (gain_c && misaligned(gain_c, 16)) || (gain_e && misaligned(gain_e, 16)) || (gain_q && misaligned(gain_q, 16)) ||
      (q_term && misaligned(q_term, 16)))
    return SB_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < fp.total || misaligned(workspace, 256)) return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  float* part = reinterpret_cast<float*>(ws);
  int* err_word = reinterpret_cast<int*>(ws + fp.part_bytes);
  bf16* x = reinterpret_cast<bf16*>(ws + fp.x_off);
  const int r_pad = fp.gemm.r_pad;
  CUtensorMap wmap, xmap;
  if (!make_2d_map(&wmap, w, (uint64_t)3 * d, (uint64_t)d_out, SG_BM) ||
      !make_2d_map(&xmap, x, (uint64_t)d, (uint64_t)3 * r_pad, (uint32_t)r_pad))
    return SB_ERR_CUDA;
  sb_status st = launch_dependent(fuse_norm_kernel, dim3(fp.segments * r_pad), dim3(256), cs, static_cast<const bf16*>(c),
                                  static_cast<const bf16*>(e), static_cast<const bf16*>(q), gain_c, gain_e, gain_q, eps,
                                  (int)n_starts, (int)block_k, (int)d, r_pad, fp.segments, x);
  if (st != SB_OK) return st;
  st = launch_shift_gemm(fp.gemm, wmap, xmap, fp.n_cols, d, d_out, r_pad, part, err_word, cs);
  if (st != SB_OK) return st;
  return launch_dependent(fuse_finish_kernel, dim3(ceil_div(d_out / 4, 256), n_starts * block_k), dim3(256), cs,
                          static_cast<const float*>(part), fp.n_cols, (int)d_out, fp.gemm.ksplit, (int)block_k,
                          (int)q_term_valid, q_term, static_cast<bf16*>(out), err_word, status);
}
