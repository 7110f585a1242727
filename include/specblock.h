/*
 * specblock.h -- C ABI of the SpecBlock draft-and-verify hot path for NVIDIA B200 (sm_100a).
 *
 * One verifier iteration of SpecBlock (Algorithm 1) grows a draft tree by block
 * expansions, scores every tree node with one parallel target forward, commits the
 * longest accepted root-to-node path plus one bonus token, and keeps the committed
 * positions' keys/values in the cache.  This library holds the device steps of that
 * iteration that do not need model weights:
 *
 *   sb_tree_ancestors  ancestor bitmask / depth of every tree node      (Sec. 3.1, App. A.2, Fig. 4)
 *   sb_tree_attention  tree-masked attention over prefix KV + ancestors (Sec. 3.1, App. A.2, the verify step of Alg. 1)
 *   sb_tree_expand     per-row top-k + bucket-driven branching          (Sec. 3.2, App. A.5, the attach step of Alg. 1)
 *   sb_rank_features   15-dim summary of each draft distribution        (Sec. 3.2, App. B)
 *   sb_tree_expand_features  both of the above from one pass over the scores
 *   sb_verifier_signal verifier-derived update signal s = sum (1 - r)   (Sec. 3.4, Alg. 2)
 *   sb_verify_sample   stochastic (temperature > 0) tree verification   (Sec. 4.1, Sec. 4.2)
 *   sb_shift_project   layer-wise shift projection between drafter layers (Sec. 3.1)
 *   sb_fuse_project    the drafter's fused per-position input h^(0)      (Sec. 3.1, the paragraph on the block forward)
 *   sb_verify_accept   greedy longest accepted path + bonus token       (App. A.5, the verify and return steps of Alg. 1)
 *   sb_kv_compact      move the accepted path's K/V behind the prefix   (Sec. 3.1, App. A.2: committed positions stay in the cache)
 *   sb_path_rows       the accepted path in the drafter's row numbering  (App. A.2)
 *
 * Conventions that hold for every call
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *     The library never allocates or frees device memory, enqueues its kernels on `stream` (a
 *     cudaStream_t passed as void*, NULL = legacy default stream) and returns without synchronising.
 *     It keeps no state between calls, with three small exceptions: per device, kernel attributes and
 *     occupancy figures are set up or looked up on the first call that needs them (so that first
 *     call on a device should come before any stream capture); sb_verify_accept_static uses a fixed
 *     scratch array inside the library image, whose device address it looks up once per device (valid
 *     for the life of the device's primary context); and the status word of the projection calls
 *     is written by their kernels, i.e. after the call has returned.  One process may drive several
 *     devices: all of this is kept per device, for the device that is current during the call.
 *   - The return value reports what the host can see (null pointers, unsupported shapes,
 *     a workspace that is too small, a failed launch).  Data-dependent problems (a parent
 *     index that is not smaller than its child, a prefix longer than the cache, a page id
 *     outside the pool) are written to the caller's `status` device array, one int32 per
 *     sequence (0 = ok, else an sb_status value).  The outputs of a sequence with a bad tree or bad
 *     lengths are zero-filled; with a page id outside the pool (SB_ERR_BOUNDS from the page table)
 *     the sequence's outputs are unspecified -- every read is redirected to page 0, so nothing is
 *     read outside the pool, and the other sequences' outputs are unaffected.  No kernel traps,
 *     spins without bound or reads outside the described arrays.
 *   - bf16 = IEEE-754 binary32 truncated to its upper 16 bits (round-to-nearest-even on
 *     conversion).  All accumulation is fp32.
 *   - Tree node i of sequence b lives at logical cache position prefix_len[b] + i: the
 *     forward that produced the tree's K/V appended them behind the prefix in node order.
 */
#ifndef SPECBLOCK_H_
#define SPECBLOCK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SB_MAX_NODES 128 /* nodes per tree: one 128-bit ancestor mask per node            */
#define SB_MAX_DEPTH 32  /* longest accepted path (drafted tokens) handled by accept/compact */
#define SB_KMAX 16       /* widest per-row top-k kept by sb_tree_expand (paper's widest map entry is 10) */

typedef enum sb_status {
  SB_OK = 0,
  SB_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, Hq % Hkv != 0 ...        */
  SB_ERR_UNSUPPORTED = 2,  /* head_dim / page_size / limits outside what is built        */
  SB_ERR_WORKSPACE = 3,    /* workspace smaller than the *_workspace_bytes query         */
  SB_ERR_INVALID_TREE = 4, /* per-sequence: parent[i] not in {-1} U [0,i), too many nodes */
  SB_ERR_BOUNDS = 5,       /* per-sequence: prefix+nodes beyond cache, page id outside pool */
  SB_ERR_CUDA = 6          /* a CUDA runtime call or launch failed                       */
} sb_status;

typedef enum sb_dtype { SB_BF16 = 0, SB_F32 = 1 } sb_dtype;

/*
 * A ragged batch of draft trees over ONE layer's KV cache.
 *
 * Cache layouts (bf16, K and V separate, same shape):
 *   page_size == 0 : contiguous  [batch][kv_capacity][n_kv_heads][head_dim]
 *   page_size  > 0 : paged pool  [num_pages][page_size][n_kv_heads][head_dim]; logical position
 *                    j of sequence b is row (j % page_size) of pool page
 *                    page_table[b*max_pages + j / page_size].
 * Tree: node_offsets is the exclusive scan of the per-sequence node counts N_b (N_b <=
 * SB_MAX_NODES); parent[node_offsets[b] + i] is the LOCAL index of node i's parent, -1 when the
 * node hangs directly off the prefix.  A valid tree has parent[i] in {-1} U [0, i).
 * The three host integers at the end only size grids and bound loops; the kernels re-check
 * the device values against them and flag SB_ERR_INVALID_TREE / SB_ERR_BOUNDS instead of
 * trusting them.
 * index_arrays_settled: the attention kernel starts as a programmatic dependent of whatever
 * precedes it in the stream and normally reads nothing before that work has completed.  A caller
 * who knows that the kernel enqueued IMMEDIATELY before the call does not write this batch's index
 * arrays (prefix_len, node_offsets, q_node_begin, q_offsets -- e.g. the previous layer's attention
 * call of the same verify forward) may set this to 1: the sequence lengths are then fetched while
 * that kernel is still running (about half a microsecond per call).  Q, K, V, the parents and the
 * page table are always read after it has completed.  0 is always correct.
 * prefix_rows_settled (only with index_arrays_settled = 1): the same vouch for the cache rows of
 * the committed prefix -- the kernel enqueued immediately before does not write K or V at positions
 * below prefix_len[b] (a projection that appends the tree's rows, or the previous layer's
 * attention, qualifies).  Key blocks that lie wholly inside the prefix may then be requested
 * before that kernel has completed; rows from prefix_len on, Q, V, the parents and the page table
 * are still read afterwards.  Used by the contiguous-cache single-wave kernel; 0 is always correct.
 */
typedef struct sb_tree_batch {
  int32_t batch;      /* B >= 1                                                     */
  int32_t n_q_heads;  /* Hq                                                         */
  int32_t n_kv_heads; /* Hkv, Hq % Hkv == 0, group size G = Hq/Hkv <= 16            */
  int32_t head_dim;   /* D in {64, 128}                                             */
  const void* k_cache;
  const void* v_cache;
  int32_t page_size;         /* 0 = contiguous, else a power of two >= 16           */
  int32_t max_pages;         /* paged: row length of page_table                     */
  int64_t kv_capacity;       /* contiguous: positions per sequence                  */
  int32_t num_pages;         /* paged: pages in the pool                            */
  int32_t total_nodes;       /* host copy of node_offsets[B]                        */
  const int32_t* page_table; /* [B][max_pages], paged only                          */
  const int32_t* prefix_len; /* [B]  P_b >= 0                                       */
  const int32_t* node_offsets; /* [B+1]                                             */
  const int32_t* parent;     /* [total_nodes]                                       */
  int32_t max_nodes;         /* host upper bound on N_b (<= SB_MAX_NODES)           */
  int32_t max_kv_len;        /* host upper bound on P_b + N_b                       */
  int32_t index_arrays_settled; /* 0, or 1: see below                                */
  int32_t prefix_rows_settled;  /* 0, or 1: see below (needs index_arrays_settled)   */
} sb_tree_batch;

/*
 * sb_tree_ancestors -- ancestor set and depth of every node (App. A.2; Fig. 4).
 *   anc(i) = {i} U anc(parent[i]), anc(-1) = {}; depth(i) = |anc(i)| - 1.  Bit a of the 128-bit
 *   mask anc_mask[node][4] (little-endian 32-bit words) is set iff a is in anc(i).  The
 *   position id the figure prints for a node is prefix_len + depth.
 *   node_offsets [B+1], parent [total]; outputs anc_mask uint32 [total][4], depth int32 [total],
 *   status int32 [B].  anc_mask or depth may be NULL.  Invalid trees: status = SB_ERR_INVALID_TREE,
 *   that sequence's outputs zero.
 */
sb_status sb_tree_ancestors(int32_t batch, const int32_t* node_offsets, const int32_t* parent,
                            int32_t max_nodes, uint32_t* anc_mask, int32_t* depth,
                            int32_t* status, void* stream);

/*
 * sb_tree_attention -- tree-masked attention of one layer (Sec. 3.1, the paragraph on
 * dependence inside a block; App. A.2: prefix fully visible, earlier draft positions visible only
 * along the branch path, causal inside the block; the verify step of Alg. 1).
 *
 *   For sequence b, query node i in [q_node_begin[b], N_b), query head h (KV head g = h / G):
 *     visible keys = {0..P_b-1} U {P_b + a : a in anc(i)}
 *     s_j = scale * <q[i,h,:], k[j,g,:]>,  lse = ln sum_j exp(s_j),
 *     out[i,h,:] = sum_j exp(s_j - lse) v[j,g,:]
 *
 *   q, out : bf16 [total_q][Hq][D]; sequence b's first query row is q_offsets[b] (NULL: the
 *            rows follow node_offsets, which requires q_node_begin == NULL).
 *   q_node_begin : [B] first node that has a query row (earlier nodes are cached context
 *            only, e.g. blocks drafted by an earlier forward), or NULL = 0.
 *   lse    : fp32 [total_q][Hq] natural-log sum-exp, or NULL.
 *   scale  : 0 means 1/sqrt(D).
 *   num_splits : how many KV chunks each (sequence, KV head, query tile) is cut into;
 *            0 = chosen from the grid size.  Chunks are merged by log-sum-exp; a chunk in which
 *            a row sees no key contributes nothing.
 *   workspace : scratch of at least sb_tree_attention_workspace_bytes(...) bytes, 256-byte
 *            aligned; contents need no initialisation and are garbage afterwards.  Calls
 *            that may overlap on the GPU need distinct workspaces.
 *   status : int32 [B].
 */
sb_status sb_tree_attention(const sb_tree_batch* tb, const int32_t* q_node_begin,
                            const int32_t* q_offsets, int32_t total_q, const void* q, void* out,
                            float* lse, float scale, int32_t num_splits, void* workspace,
                            size_t workspace_bytes, int32_t* status, void* stream);

/* Bytes of workspace sb_tree_attention needs for this batch / num_splits (0 = auto). Host only. */
size_t sb_tree_attention_workspace_bytes(const sb_tree_batch* tb, int32_t total_q,
                                         int32_t num_splits);

/*
 * sb_tree_expand -- attach candidates of one batched drafter forward to the tree
 * (Sec. 3.2, branching driven by the rank bucket; App. A.5 maps b(.); the attach loop of Alg. 1
 * over starting points and positions).
 *
 *   Rows r = i*block_k + k (start i, position k), scores fp32 [n_rows][row_stride >= vocab].
 *   (1) per row the SB_KMAX best ids by (score descending, id ascending; NaN counts as -inf)
 *       -> topk_tok int32 [n_rows][SB_KMAX], topk_val fp32 [n_rows][SB_KMAX] (ranks beyond vocab: -1 / -inf);
 *   (2) b_r = bmap[bucket[r]] (bucket in 0..3; bmap host array of 4 entries, each 0..SB_KMAX);
 *   (3) rows in order: row (i,0) attaches under start_parent[i] (an existing node id, or -1);
 *       row (i,k>0) attaches under the rank-0 node created for row (i,k-1); when that node does
 *       not exist the row and the rest of its block emit nothing;
 *   (4) ranks 0..b_r-1 become nodes n_nodes, n_nodes+1, ... with tok, parent,
 *       depth = depth[parent]+1 (0 under -1), node_row = r, node_rank = rank, until
 *       node_budget nodes exist (emission stops for good).
 *   n_nodes : device int32 scalar, in = nodes already in the arrays, out = new count.
 *   tok/parent/depth/node_row/node_rank : int32 arrays of capacity node_budget.
 *   workspace : sb_tree_expand_workspace_bytes(n_rows, vocab) bytes.
 *   status : int32 [1].
 */
sb_status sb_tree_expand(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                         int32_t block_k, const uint8_t* bucket, const int32_t* bmap /*host[4]*/,
                         const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                         int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                         int32_t* node_rank, int32_t* topk_tok, float* topk_val, void* workspace,
                         size_t workspace_bytes, int32_t* status, void* stream);
size_t sb_tree_expand_workspace_bytes(int32_t n_rows, int32_t vocab);

/*
 * sb_rank_features -- the rank head's 15-dimensional summary psi(p) of every draft distribution
 * (Sec. 3.2, the rank head; App. B, its distribution summary).
 *
 *   scores fp32 [n_rows][row_stride >= vocab] are the drafter's logits; p = softmax(row), NaN read
 *   as -inf.  features fp32 [n_rows][15], in the order the appendix lists them:
 *     [0..9]   natural-log probabilities of the ten most likely tokens, most likely first
 *              (-inf where the vocabulary has fewer than ten tokens);
 *     [10..12] logit gaps between the top token and the tokens of rank 2, 3 and 5 (+inf where
 *              that rank does not exist);
 *     [13]     probability of the top token;   [14] entropy -sum p ln p in nats.
 *   A row without any finite score is reported as the uniform distribution.
 *   The scores are streamed once (the same scan as sb_tree_expand's top-k, which also yields the
 *   chunk maxima and the two exponential sums); accuracy is that of fp32 sums over the row.
 *   workspace : sb_rank_features_workspace_bytes(n_rows, vocab) bytes, 256-byte aligned.
 */
sb_status sb_rank_features(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                           float* features, void* workspace, size_t workspace_bytes, void* stream);
size_t sb_rank_features_workspace_bytes(int32_t n_rows, int32_t vocab);

/*
 * sb_tree_expand_features -- sb_tree_expand and sb_rank_features of the same scores in ONE pass over them:
 * the scan that finds the per-chunk top-16 also accumulates the chunk statistics of psi(p), and both
 * finishing kernels follow it.  Arguments as sb_tree_expand plus features fp32 [n_rows][15] as
 * sb_rank_features; results identical to the two separate calls, except that node_row counts the rows from
 * row_base (node_row = row_base + r), like child_row.
 *   child_row int32 [node_budget] or NULL: for every row of this call that emits nodes under an existing
 *   node, child_row[that node] = row_base + row -- the row of the drafter's scores that proposed the node's
 *   children, as sb_verifier_signal and sb_verify_sample want it (row_base = rows of the earlier blocks when
 *   the blocks' scores lie one after the other in one matrix).  Entries of nodes without children are left
 *   as they are (initialise the array to -1); if several rows attach under one node, one of them is recorded.
 *   workspace : sb_rank_features_workspace_bytes(n_rows, vocab) bytes, 256-byte aligned.
 */
sb_status sb_tree_expand_features(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                                  int32_t block_k, const uint8_t* bucket, const int32_t* bmap /*host[4]*/,
                                  const int32_t* start_parent, int32_t node_budget, int32_t* n_nodes,
                                  int32_t* tok, int32_t* parent, int32_t* depth, int32_t* node_row,
                                  int32_t* node_rank, int32_t* topk_tok, float* topk_val, float* features,
                                  int32_t* child_row, int32_t row_base, void* workspace, size_t workspace_bytes,
                                  int32_t* status, void* stream);

/*
 * sb_shift_project -- the layer-wise shift between consecutive decoder layers of the drafter
 * (Sec. 3.1, the paragraph on dependence inside a block, the equation for h-tilde): position k's state is
 * concatenated with position k-1's state of the same block and projected back by W_shift.
 *
 *   h   bf16 [n_rows][d]: rows r = i * block_k + k are the block_k positions of block i.
 *   w   bf16 [d_out][2 d] row-major: W_shift acting on the concatenation [h_k , h_{k-1}].
 *   out bf16 [n_rows][d_out]: out[r] = w[:, :d] h[r] + w[:, d:] h[prev(r)], prev(r) = r - 1 inside a
 *       block and r at its first position (the convention h_0 = h_1); fp32 accumulation.
 *   block_k = 0: plain projection out = h w^T with w [d_out][d] (e.g. W_cond of the block forward).
 *   Limits: n_rows <= 128, d a multiple of 64, d_out a multiple of 128, h and w 16-byte aligned.
 *   workspace: sb_shift_project_workspace_bytes(...) bytes, 256-byte aligned (fp32 partials of the
 *   K splits and one word that outlives the call: hand the same workspace to every call, or a zeroed
 *   one).  status int32 [1]: SB_OK, or SB_ERR_CUDA if a bounded device wait gave up.
 *   HBM-bound on the weights: 2 * d * d_out * 2 bytes are read once.
 *   Ordering: the kernels are programmatic dependents of whatever precedes the call in the stream.
 *   h (and every output) is touched only after that work has completed, but the first tiles of w
 *   are requested earlier: w must not be written by the ONE kernel enqueued immediately before the
 *   call (weights updated earlier in the stream are seen as usual).
 */
sb_status sb_shift_project(const void* h, const void* w, int32_t n_rows, int32_t d, int32_t d_out,
                           int32_t block_k, void* out, void* workspace, size_t workspace_bytes,
                           int32_t* status, void* stream);
size_t sb_shift_project_workspace_bytes(int32_t n_rows, int32_t d, int32_t d_out, int32_t block_k);

/*
 * sb_fuse_project -- the per-position input of a drafter block (Sec. 3.1, the paragraph on the block
 * forward, the equation for h^(0)): the context feature c_s of start s, the embedding e_s of its last committed
 * token and the learnable query q_k of draft depth k are normalised, concatenated and projected by
 * W_fuse.  c_s and e_s are shared by the block_k positions of a block (the prefix broadcast).
 *
 *   c, e bf16 [n_starts][d];  q bf16 [block_k][d];  w bf16 [d_out][3 d] row-major, acting on
 *   [norm(c) , norm(e) , norm(q)].  the normalisation is not specified further by the paper; here it is
 *   norm(x)[j] = gain[j] * x[j] / sqrt(mean_j x[j]^2 + eps), gains fp32 [d] or NULL for ones (the
 *   normalised rows are rounded to bf16, the type of the tensor-core operand).
 *   out bf16 [n_starts * block_k][d_out], row s * block_k + k; fp32 accumulation.
 *   Since out[s, k] = w_c norm(c_s) + w_e norm(e_s) + w_q norm(q_k), the GEMM has
 *   max(n_starts, block_k) columns and every third of w is read once.  The last term does not
 *   depend on the start or on the call: with q_term_valid = 0 it is computed and, if q_term is not
 *   NULL, stored there (fp32 [block_k][d_out]); with q_term_valid = 1 it is read from q_term and only
 *   the first 2 d columns of w are streamed.  Both ways give bit-identical outputs.
 *   Limits: n_starts, block_k <= 128, d a multiple of 64, d_out a multiple of 128, pointers 16-byte
 *   aligned (out 8).  workspace: sb_fuse_project_workspace_bytes(...) bytes, 256-byte aligned (the
 *   normalised rows, fp32 partials and one word that outlives the call, as for sb_shift_project).
 *   status int32 [1]: SB_OK, or SB_ERR_CUDA if a bounded device wait gave up.
 *   HBM-bound on the weights: (3 or 2) * d * d_out * 2 bytes.  Ordering as for sb_shift_project: c, e, q,
 *   the gains and q_term are read after the preceding work has completed, the first tiles of w before.
 */
sb_status sb_fuse_project(const void* c, const void* e, const void* q, const float* gain_c,
                          const float* gain_e, const float* gain_q, float eps, const void* w,
                          int32_t n_starts, int32_t block_k, int32_t d, int32_t d_out, float* q_term,
                          int32_t q_term_valid, void* out, void* workspace, size_t workspace_bytes,
                          int32_t* status, void* stream);
size_t sb_fuse_project_workspace_bytes(int32_t n_starts, int32_t block_k, int32_t d, int32_t d_out,
                                       int32_t q_term_valid);

/*
 * sb_verify_sample -- verification at temperature T > 0 by multi-candidate rejection sampling over
 * the draft tree (Sec. 4.1 evaluates temperature 0 and 1.0; Sec. 4.2 mentions rejection sampling against the
 * target).  The paper names the procedure without listing it; the steps are:
 *
 *   a = root (node 0), depth 0, p = softmax(logits[a] / T).  Repeat:
 *     children of a = the nodes c with parent[c] == a, in increasing index (emission order);
 *     stop if there are none or depth == max_depth;
 *     q = softmax(scores[child_row[a]] / T), the draft distribution that proposed them;
 *     for each child c in order, x = tok[c]: accept c iff u_accept[c] < p(x) / q(x)
 *       (q(x) = 0: iff p(x) > 0).  Accepted: a = c, depth += 1, p = softmax(logits[c] / T), next round.
 *       Rejected: p <- max(p - q, 0) renormalised (unchanged if nothing remains); q(x) <- 0 and q
 *       renormalised (siblings are distinct tokens: drawn without replacement).
 *     stop if every child was rejected.
 *   bonus = the smallest v whose inclusive prefix sum of p exceeds u_bonus * sum(p) (p is the residual
 *   distribution when the walk stopped on a rejection).
 *
 *   logits [total_nodes][row_stride >= vocab] bf16 or fp32 (target), scores fp32
 *   [n_rows][score_stride >= vocab] (drafter, over the same vocabulary), child_row int32 [total_nodes]
 *   as for sb_verifier_signal, u_accept fp32 [total_nodes] and u_bonus fp32 [batch] uniform in [0, 1)
 *   supplied by the caller (the library draws no random numbers).  NaN counts as -inf; a row without a
 *   finite value is flat.  Outputs as sb_verify_accept (accept_len = depth reached, path_nodes,
 *   out_tokens = accepted tokens then the bonus, bonus).
 *   status int32 [batch]: SB_OK, SB_ERR_INVALID_TREE, or SB_ERR_BOUNDS when an inner node of the walk
 *   has no valid child_row (outputs of that sequence: accept_len 0, -1 elsewhere).
 *   workspace: sb_verify_sample_workspace_bytes(batch, vocab, total_nodes, n_rows) bytes, 256-byte aligned (vocab
 *   floats per sequence for the residual distribution after a rejection, and the per-chunk softmax statistics of
 *   every target and draft row, which a first pair of kernels computes over the whole GPU).
 *   Probabilities and sums are fp32; a decision whose two sides differ by less than about 1e-5
 *   relative may fall either way.
 */
sb_status sb_verify_sample(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                           const float* scores, int64_t score_stride, int32_t n_rows, int32_t batch,
                           int32_t total_nodes, const int32_t* node_offsets, const int32_t* parent,
                           const int32_t* tok, const int32_t* child_row, float temperature,
                           const float* u_accept, const float* u_bonus, int32_t max_depth, int32_t* accept_len,
                           int32_t* path_nodes, int32_t* out_tokens, int32_t* bonus, void* workspace,
                           size_t workspace_bytes, int32_t* status, void* stream);
size_t sb_verify_sample_workspace_bytes(int32_t batch, int32_t vocab, int32_t total_nodes, int32_t n_rows);

/*
 * sb_verifier_signal -- one iteration's term of the verifier-derived update signal
 * s = sum over rejected positions of (1 - r), r = the drafter's probability of the token the
 * target chose there (Sec. 3.4, the verifier-derived signal; Alg. 2 line 2).
 *
 *   A verify iteration rejects at most one position per sequence: the one right after the last
 *   accepted node best = path_nodes[b][accept_len[b]], where the target chose bonus[b] (all three
 *   as sb_verify_accept leaves them on the device).
 *   child_row int32 [total_nodes]: for every tree node the row of `scores` (drafter logits, fp32
 *       [n_rows][row_stride >= vocab]) that predicted the token following it, or -1 when nothing
 *       was drafted after it.
 *   r = softmax(scores[child_row[best]])[bonus]; NaN scores read as -inf, a row without a finite
 *       score as flat, a token outside [0, vocab) as probability 0 (not in the drafter's vocabulary).
 *   r_prob fp32 [batch]: out, r, or -1 when nothing was rejected (child_row = -1) or on an error.
 *   signal fp32 [batch]: in/out, signal[b] += 1 - r; the caller zeroes it at the start of a query
 *       and reads the query-level s after its last iteration.
 *   status int32 [batch]: SB_OK, or SB_ERR_BOUNDS when accept_len, the path node or the row index
 *       is out of range (r_prob = -1, signal untouched).
 *   One pass over one score row per sequence (vocab * 4 bytes); fp32 sums.  No workspace.
 */
sb_status sb_verifier_signal(const float* scores, int64_t row_stride, int32_t n_rows, int32_t vocab,
                             int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                             const int32_t* child_row, const int32_t* path_nodes, const int32_t* accept_len,
                             const int32_t* bonus, int32_t max_depth, float* r_prob, float* signal,
                             int32_t* status, void* stream);

/*
 * sb_verify_accept -- greedy (temperature 0) verification (App. A.5: the longest accepted
 * prefix is what gets committed; the verify step of Alg. 1 returns it with a bonus token; case study:
 * accepted tokens plus one bonus token are committed).
 *
 *   logits [total_nodes][row_stride >= vocab] (bf16 or fp32): the target's next-token scores
 *   at every tree node.  amax[i] = smallest id attaining the row maximum (NaN counts as -inf).
 *   Node 0 of each sequence is the root (last committed token, parent -1; any other parent of
 *   -1 is SB_ERR_INVALID_TREE).  Node i>0 is accepted iff tok[i] == amax[parent[i]] and its
 *   parent is accepted.  best = accepted node of greatest depth (ties: smallest index).
 *   accept_len[b] = depth(best) (drafted tokens accepted; the committed count is accept_len+1);
 *   path_nodes[b][0..accept_len] = root..best (rest -1); out_tokens[b][0..accept_len-1] = their
 *   tokens (root excluded), out_tokens[b][accept_len] = bonus[b] = amax[best] (rest -1).
 *   Row length of path_nodes/out_tokens is max_depth+1, max_depth <= SB_MAX_DEPTH; a deeper
 *   accepted path is cut at max_depth.
 *   workspace : sb_verify_accept_workspace_bytes(total_nodes, vocab) bytes.
 */
sb_status sb_verify_accept(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                           int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                           const int32_t* parent, const int32_t* tok, int32_t max_depth,
                           int32_t* amax, int32_t* accept_len, int32_t* path_nodes,
                           int32_t* out_tokens, int32_t* bonus, void* workspace,
                           size_t workspace_bytes, int32_t* status, void* stream);
size_t sb_verify_accept_workspace_bytes(int32_t total_nodes, int32_t vocab);

/*
 * sb_verify_accept_static -- sb_verify_accept for callers that cannot provide scratch memory.
 * (The paper has no counterpart for this call; it exists for integration reasons only.)
 *
 *   Some hosts of this library never get to call cudaMalloc themselves: a plugin that runs inside
 *   another runtime's pre-sized memory arena, a process whose device memory was carved up once at
 *   start-up, or code that runs where an allocation would synchronise the device at a bad moment.
 *   For them this variant takes no workspace: the per-chunk argmax partials live in a fixed
 *   SB_STATIC_SCRATCH_BYTES array that is part of the library image (every GPU that loads the
 *   library holds these bytes until the process exits).  Arguments, results and status words are
 *   exactly those of sb_verify_accept; inputs and outputs are still the caller's buffers.
 *
 *   - The call allocates and frees nothing, on the host or on the device.
 *   - Problems whose scratch need (sb_verify_accept_workspace_bytes) exceeds SB_STATIC_SCRATCH_BYTES
 *     are refused with SB_ERR_WORKSPACE; use sb_verify_accept with your own workspace for those.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it
 *     (nothing in it has to start at zero: every partial is rewritten before it is read).  Two
 *     calls that can overlap on the GPU -- different streams, or graph branches -- race on it;
 *     serialise them or use sb_verify_accept with separate workspaces.
 */
#define SB_STATIC_SCRATCH_BYTES (256 * 1024)
sb_status sb_verify_accept_static(const void* logits, sb_dtype dtype, int64_t row_stride, int32_t vocab,
                                  int32_t batch, int32_t total_nodes, const int32_t* node_offsets,
                                  const int32_t* parent, const int32_t* tok, int32_t max_depth,
                                  int32_t* amax, int32_t* accept_len, int32_t* path_nodes,
                                  int32_t* out_tokens, int32_t* bonus, int32_t* status, void* stream);

/*
 * sb_kv_compact -- keep the committed positions' K/V, drop the rest (Sec. 3.1 / App. A.2: later
 * forwards see every committed position's cached keys and values as the verified prefix).
 *
 *   For every layer l < n_layers (layer l's cache starts layer_stride_elems bf16 elements after
 *   layer l-1's; tb->k_cache / v_cache are layer 0), K and V, sequence b, j = 0..accept_len[b]:
 *       cache[P_b + j] <- cache[P_b + path_nodes[b][j]]          (in place)
 *   new_len[b] = P_b + accept_len[b] + 1.  Positions >= new_len[b] are unspecified afterwards.
 *   path_nodes int32 [B][max_depth+1] and accept_len int32 [B] as written by sb_verify_accept.
 *   A path that is not strictly increasing from node 0, or leaves the tree, sets
 *   SB_ERR_INVALID_TREE for that sequence and moves nothing.
 */
sb_status sb_kv_compact(const sb_tree_batch* tb, int32_t n_layers, int64_t layer_stride_elems,
                        const int32_t* path_nodes, const int32_t* accept_len, int32_t max_depth,
                        int32_t* new_len, int32_t* status, void* stream);

/*
 * sb_path_rows -- the accepted path in the drafter's own row numbering (App. A.2: a committed
 * position keeps the keys and values that its own draft forward produced).
 *
 *   A draft forward has one cache row per block position, shared by the sibling tokens attached at
 *   that position, so the drafter's cache is committed by rows, not by tree nodes.  For sequence b
 *   with accepted path nodes p_0 = 0, p_1, ..., p_a (a = accept_len[b]):
 *       path_rows[b][0] = 0
 *       path_rows[b][j] = 1 + node_row[node_offsets[b] + p_j] - row_begin[b],   j = 1..a
 *   -- node_row, the tree array written by sb_tree_expand / sb_tree_expand_features, names the row
 *   whose distribution proposed a node (counted from the call's row_base, so that the rows of an
 *   iteration's blocks are numbered through); entries past a are -1.
 *   Slot 0 stands for the last committed position, whose row lies just before this iteration's
 *   rows: with a drafter cache that holds row r of the iteration at position Pd + r,
 *   sb_kv_compact over a batch with prefix_len = Pd - 1 and node_offsets = {0, 1 + rows} and the
 *   path (path_rows, accept_len) moves the accepted rows to Pd .. Pd + a - 1 and returns
 *   new_len = Pd + a.
 *   row_begin int32 [batch] or NULL (= 0): first row of each sequence in node_row's numbering.
 *   status[b]: SB_ERR_INVALID_TREE when accept_len[b] is outside [0, max_depth], a path node lies
 *   outside the sequence's tree or has no row (the root, or a row before row_begin[b]), or the rows
 *   do not increase along the path; path_rows[b] is then 0 followed by -1.
 *   All pointers device; path_nodes, path_rows int32 [batch][max_depth+1]; max_depth <= SB_MAX_DEPTH.
 */
sb_status sb_path_rows(int32_t batch, const int32_t* node_offsets, const int32_t* node_row,
                       const int32_t* row_begin, const int32_t* path_nodes, const int32_t* accept_len,
                       int32_t max_depth, int32_t* path_rows, int32_t* status, void* stream);

/* Text for a status code (static storage). */
const char* sb_status_string(sb_status s);
/* Library version, major*10000 + minor*100 + patch. */
int32_t sb_version(void);
/* Kernels launched by this library in this process since load (host counter, for benchmarks). */
int64_t sb_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECBLOCK_H_ */
