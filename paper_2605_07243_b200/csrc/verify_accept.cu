// sb_verify_accept: greedy verification of a draft tree (App. A.5; Alg. 1 "(prefix, bonus) <- verify").
//
//   row_argmax_kernel : streams the [nodes][vocab] logits once; every (row, vocab chunk) CTA keeps the
//                       best (value, id) under the order "value descending, id ascending" with NaN
//                       read as -inf, and writes one partial per chunk.
//   accept_kernel     : one CTA per sequence: finishes the argmax, marks the edges whose drafted
//                       token equals the target's choice at the parent, finds the deepest node whose
//                       whole root path matches, and writes path, tokens and the bonus token.
#include "common.cuh"

namespace sb {

struct Best {
  float v;
  int i;
};

// Total order of the argmax: larger value first, then smaller id.
__device__ inline bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

__device__ inline Best warp_best(Best x) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, x.v, s);
    const int oi = __shfl_xor_sync(0xffffffffu, x.i, s);
    if (better(ov, oi, x.v, x.i)) { x.v = ov; x.i = oi; }
  }
  return x;
}

constexpr int ARGMAX_THREADS = 256;

template <typename T>
__device__ inline float logit_to_float(T x);
template <>
__device__ inline float logit_to_float<float>(float x) { return score_of(x); }
template <>
__device__ inline float logit_to_float<uint16_t>(uint16_t x) { return score_of(bf16_bits_to_float(x)); }

// T = uint16_t (bf16 bits) or float.  VEC elements per 16-byte load.
template <typename T>
__global__ void __launch_bounds__(ARGMAX_THREADS) row_argmax_kernel(const T* __restrict__ logits,
                                                                    long long row_stride, int vocab,
                                                                    int chunk, int n_chunks, bool vec_ok,
                                                                    float* __restrict__ part_val,
                                                                    int* __restrict__ part_idx) {
  constexpr int VEC = 16 / sizeof(T);
  const int row = blockIdx.y, c = blockIdx.x;
  const T* base = logits + (long long)row * row_stride;
  const int begin = c * chunk;
  const int end = min(vocab, begin + chunk);
  pdl_release();  // the path kernel may start its prologue
  Best best = {-INFINITY, 0x7fffffff};
  if (vec_ok) {
    // four independent running maxima (one per load slot modulo 4): the compare-select chain of a single
    // maximum is a serial dependency of 64 steps per sweep; ids still ascend inside each of the four
    Best acc[4] = {{-INFINITY, 0x7fffffff}, {-INFINITY, 0x7fffffff}, {-INFINITY, 0x7fffffff}, {-INFINITY, 0x7fffffff}};
    // chunk is a multiple of VEC and rows are 16-byte aligned
    const int n_vec = max(0, (end - begin) / VEC);
    const uint4* vb = reinterpret_cast<const uint4*>(base + begin);
    // All of a thread's loads of one sweep are issued before any is used: a chunk of up to
    // UNROLL * 256 vectors (32 KB) costs one trip to memory.
    constexpr int UNROLL = 8;
    for (int t0 = threadIdx.x; t0 < n_vec; t0 += UNROLL * ARGMAX_THREADS) {
      uint4 raw[UNROLL];
#pragma unroll
      for (int q = 0; q < UNROLL; ++q)
        if (t0 + q * ARGMAX_THREADS < n_vec) raw[q] = __ldg(vb + t0 + q * ARGMAX_THREADS);
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        if (t0 + q * ARGMAX_THREADS < n_vec) {
          const T* e = reinterpret_cast<const T*>(&raw[q]);
#pragma unroll
          for (int u = 0; u < VEC; ++u) {
            const float x = logit_to_float<T>(e[u]);
            const int id = begin + (t0 + q * ARGMAX_THREADS) * VEC + u;
            if (x > acc[q & 3].v) { acc[q & 3].v = x; acc[q & 3].i = id; }  // ids ascend inside a slot: strict keeps the first
          }
        }
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
      if (better(acc[a].v, acc[a].i, best.v, best.i)) best = acc[a];
    for (int id = begin + n_vec * VEC + threadIdx.x; id < end; id += ARGMAX_THREADS) {
      const float x = logit_to_float<T>(base[id]);
      if (x > best.v) { best.v = x; best.i = id; }
    }
  } else {
    for (int id = begin + threadIdx.x; id < end; id += ARGMAX_THREADS) {
      const float x = logit_to_float<T>(base[id]);
      if (x > best.v) { best.v = x; best.i = id; }
    }
  }
  best = warp_best(best);
  __shared__ float s_v[ARGMAX_THREADS / 32];
  __shared__ int s_i[ARGMAX_THREADS / 32];
  if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = best.v; s_i[threadIdx.x >> 5] = best.i; }
  __syncthreads();
  if (threadIdx.x < 32) {
    Best x = {-INFINITY, 0x7fffffff};
    if (threadIdx.x < ARGMAX_THREADS / 32) { x.v = s_v[threadIdx.x]; x.i = s_i[threadIdx.x]; }
    x = warp_best(x);
    if (threadIdx.x == 0) {
      // Every thread keeps the first of its maxima by strict compares over ascending ids, so a chunk
      // that holds nothing above -inf (NaN counts as -inf) records no id at all: its first element wins.
      if (x.i == 0x7fffffff && begin < end) x.i = begin;
      // (checked build: gridDim.y rows of n_chunks partials each were sized by the host)
      if (SB_CHECKED_ACCESS((long long)row * n_chunks + c, (long long)gridDim.y * n_chunks, nullptr)) {
        part_val[(long long)row * n_chunks + c] = x.v;
        part_idx[(long long)row * n_chunks + c] = x.i;
      }
    }
  }
}

__global__ void __launch_bounds__(SB_MAX_NODES) accept_kernel(int n_chunks, const float* __restrict__ part_val,
                                                              const int* __restrict__ part_idx,
                                                              const int* __restrict__ node_offsets,
                                                              const int* __restrict__ parent,
                                                              const int* __restrict__ tok, int total_nodes,
                                                              int max_depth, int* __restrict__ amax,
                                                              int* __restrict__ accept_len,
                                                              int* __restrict__ path_nodes,
                                                              int* __restrict__ out_tokens,
                                                              int* __restrict__ bonus, int* __restrict__ status) {
  __shared__ int s_parent[SB_MAX_NODES], s_amax[SB_MAX_NODES], s_tok[SB_MAX_NODES];
  __shared__ int s_bad, s_best;
  const int b = blockIdx.x, i = threadIdx.x;
  const int o = node_offsets[b];
  const int n = node_offsets[b + 1] - o;
  int* path = path_nodes + (long long)b * (max_depth + 1);
  int* otok = out_tokens + (long long)b * (max_depth + 1);
  for (int t = i; t <= max_depth; t += blockDim.x) { path[t] = -1; otok[t] = -1; }
  if (i == 0) { s_bad = 0; s_best = -1; accept_len[b] = 0; bonus[b] = -1; }
  __syncthreads();
  pdl_wait();  // the chunk partials of the scan kernel are complete from here on
  if (n < 1 || n > SB_MAX_NODES || o < 0 || (long long)o + n > total_nodes) {
    if (i == 0) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  if (i < n) {
    // finish the row argmax over the chunk partials
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = 0; c < n_chunks; ++c) {
      const float v = part_val[(long long)(o + i) * n_chunks + c];
      const int id = part_idx[(long long)(o + i) * n_chunks + c];
      if (better(v, id, bv, bi)) { bv = v; bi = id; }
    }
    s_amax[i] = bi;
    if (SB_CHECKED_ACCESS(o + i, total_nodes, &status[b])) amax[o + i] = bi;
    const int p = parent[o + i];
    s_parent[i] = p;
    s_tok[i] = tok[o + i];
    if (i == 0 ? p != -1 : (p < 0 || p >= i)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (i == 0) status[b] = SB_ERR_INVALID_TREE;
    return;
  }
  if (i < n) {
    // walk to the root: accepted iff every edge on the way matches
    bool acc = true;
    int depth = 0;
    for (int a = i; a > 0; a = s_parent[a]) {
      acc = acc && s_tok[a] == s_amax[s_parent[a]];
      ++depth;
    }
    if (acc && depth <= max_depth) atomicMax(&s_best, (depth << 8) | (SB_MAX_NODES - 1 - i));
  }
  __syncthreads();
  if (i == 0) {
    const int depth = s_best >> 8;
    int node = SB_MAX_NODES - 1 - (s_best & 255);
    accept_len[b] = depth;
    bonus[b] = s_amax[node];
    otok[depth] = s_amax[node];
    for (int t = depth; t >= 0; --t) {
      if (!SB_CHECKED_ACCESS(t, max_depth + 1, &status[b]) || !SB_CHECKED_ACCESS(node, n, &status[b])) break;
      path[t] = node;
      if (t > 0) otok[t - 1] = s_tok[node];
      node = s_parent[node];
    }
    status[b] = SB_OK;
  }
}

static int argmax_chunks(int total_nodes, int vocab, int vec) {
  int nc = ceil_div(4 * 148, total_nodes > 0 ? total_nodes : 1);
  const int max_nc = ceil_div(vocab, 4096);
  if (nc > max_nc) nc = max_nc;
  if (nc < 1) nc = 1;
  (void)vec;
  return nc;
}

}  // namespace sb

extern "C" size_t sb_verify_accept_workspace_bytes(int32_t total_nodes, int32_t vocab) {
  if (total_nodes < 1 || vocab < 1) return 0;
  const size_t nc = (size_t)sb::argmax_chunks(total_nodes, vocab, 8);
  return 2 * (((size_t)total_nodes * nc * 4 + 255) & ~(size_t)255);
}

extern "C" sb_status sb_verify_accept(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                                      int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                                      const int32_t* parent, const int32_t* tok, int32_t max_depth,
                                      int32_t* amax, int32_t* accept_len, int32_t* path_nodes,
                                      int32_t* out_tokens, int32_t* bonus, void* workspace,
                                      size_t workspace_bytes, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_verify_accept");
  using namespace sb;
  if (!logits || !node_offsets || !parent || !tok || !amax || !accept_len || !path_nodes || !out_tokens ||
      !bonus || !status || batch < 1 || total_nodes < 1 || vocab < 1 || row_stride < vocab)
    return SB_ERR_INVALID_ARG;
  if (dtype != SB_BF16 && dtype != SB_F32) return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH) return SB_ERR_UNSUPPORTED;
  const size_t need = sb_verify_accept_workspace_bytes(total_nodes, vocab);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int esz = dtype == SB_BF16 ? 2 : 4;
  const int vec = 16 / esz;
  const int nc = argmax_chunks(total_nodes, vocab, vec);
  int chunk = ceil_div(vocab, nc);
  chunk = ceil_div(chunk, vec) * vec;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(logits) & 15) == 0 && (row_stride * esz) % 16 == 0;
  float* part_val = static_cast<float*>(workspace);
  int* part_idx = reinterpret_cast<int*>(static_cast<char*>(workspace) + need / 2);
  if (total_nodes > 65535) return SB_ERR_UNSUPPORTED;
  dim3 grid(nc, total_nodes);
  if (dtype == SB_BF16)
    row_argmax_kernel<uint16_t><<<grid, ARGMAX_THREADS, 0, cs>>>(static_cast<const uint16_t*>(logits),
                                                                 row_stride, vocab, chunk, nc, vec_ok,
                                                                 part_val, part_idx);
  else
    row_argmax_kernel<float><<<grid, ARGMAX_THREADS, 0, cs>>>(static_cast<const float*>(logits), row_stride,
                                                              vocab, chunk, nc, vec_ok, part_val, part_idx);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  return launch_dependent(accept_kernel, dim3(batch), dim3(SB_MAX_NODES), cs, nc, part_val, part_idx, node_offsets,
                          parent, tok, total_nodes, max_depth, amax, accept_len, path_nodes, out_tokens, bonus,
                          status);
}

// ---------------------------------------------------------------------------------------------------
// sb_verify_accept_static: the same two kernels, with their scratch in a fixed array of the library
// image instead of a caller workspace -- for callers that have no way to allocate device memory.
// ---------------------------------------------------------------------------------------------------

// In host code this name is only a handle for the runtime, not a device address: the address each
// device uses comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_accept_scratch[SB_STATIC_SCRATCH_BYTES];

extern "C" sb_status sb_verify_accept_static(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                                             int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                                             const int32_t* parent, const int32_t* tok, int32_t max_depth,
                                             int32_t* amax, int32_t* accept_len, int32_t* path_nodes,
                                             int32_t* out_tokens, int32_t* bonus, int32_t* status, void* stream) {
  sb::TraceRange trace_range("sb_verify_accept_static");
  using namespace sb;
  if (!logits || !node_offsets || !parent || !tok || !amax || !accept_len || !path_nodes || !out_tokens ||
      !bonus || !status || batch < 1 || total_nodes < 1 || vocab < 1 || row_stride < vocab)
    return SB_ERR_INVALID_ARG;
  if (dtype != SB_BF16 && dtype != SB_F32) return SB_ERR_INVALID_ARG;
  if (max_depth < 0 || max_depth > SB_MAX_DEPTH || total_nodes > 65535) return SB_ERR_UNSUPPORTED;
  const size_t need = sb_verify_accept_workspace_bytes(total_nodes, vocab);
  if (need > (size_t)SB_STATIC_SCRATCH_BYTES) return SB_ERR_WORKSPACE;  // larger than the fixed array

  // Device address of the array, looked up once per device with that device current.
  // (Atomic slots: two host threads may make a device's first call at once; both then store the same
  // address.  The address holds for the life of the device's primary context.)
  static std::atomic<void*> scratch_of_device[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return SB_ERR_CUDA;
  if (dev >= kMaxDevices) return SB_ERR_UNSUPPORTED;
  void* ptr = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!ptr) {
    if (cudaGetSymbolAddress(&ptr, g_accept_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return SB_ERR_CUDA;
    }
    scratch_of_device[dev].store(ptr, std::memory_order_release);
  }
  char* scratch = static_cast<char*>(ptr);

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int esz = dtype == SB_BF16 ? 2 : 4;
  const int vec = 16 / esz;
  const int nc = argmax_chunks(total_nodes, vocab, vec);
  int chunk = ceil_div(vocab, nc);
  chunk = ceil_div(chunk, vec) * vec;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(logits) & 15) == 0 && (row_stride * esz) % 16 == 0;
  float* part_val = reinterpret_cast<float*>(scratch);
  int* part_idx = reinterpret_cast<int*>(scratch + need / 2);
  dim3 grid(nc, total_nodes);
  if (dtype == SB_BF16)
    row_argmax_kernel<uint16_t><<<grid, ARGMAX_THREADS, 0, cs>>>(static_cast<const uint16_t*>(logits),
                                                                 row_stride, vocab, chunk, nc, vec_ok,
                                                                 part_val, part_idx);
  else
    row_argmax_kernel<float><<<grid, ARGMAX_THREADS, 0, cs>>>(static_cast<const float*>(logits), row_stride,
                                                              vocab, chunk, nc, vec_ok, part_val, part_idx);
  sb_status st = launch_check();
  if (st != SB_OK) return st;
  return launch_dependent(accept_kernel, dim3(batch), dim3(SB_MAX_NODES), cs, nc, part_val, part_idx, node_offsets,
                          parent, tok, total_nodes, max_depth, amax, accept_len, path_nodes, out_tokens, bonus,
                          status);
}
