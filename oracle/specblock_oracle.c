/*
 * specblock_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what the SpecBlock draft-and-verify device steps
 * compute, written from the paper's definitions.  It exists to check the CUDA library and to
 * be timed as a CPU baseline; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.  It shares no code with the CUDA path, includes no CUDA header, and takes HOST
 * pointers only.  OpenMP pragmas spread independent rows over cores; they change no
 * arithmetic and no order of operations inside a row.
 *
 * Pin status of each function (what, other than itself, it is checked against):
 *   sbo_tree_ancestors  : the printed attention-mask example (Fig. 4) and its position ids.
 *   sbo_tree_attention  : Fig. 4 visibility through a uniform-score read-out; a library
 *                         scaled-dot-product attention on root-to-node paths and on chain trees;
 *                         closed forms (single key, equal scores, equal values).
 *   sbo_row_argmax / sbo_row_topk : numpy argmax / stable argsort.
 *   sbo_verify_accept   : exhaustive comparison with an independent recurrence on all small
 *                         trees; planted paths; the case-study tree (4 accepted + bonus).
 *   sbo_kv_compact      : numpy fancy-index gather; attention over the compacted cache.
 *   sbo_path_rows       : a hand-worked two-block tree; numpy fancy indexing on random paths.
 *   sbo_rank_features   : scipy log_softmax / entropy; closed forms (uniform row, one dominant token).
 *   sbo_verifier_signal : scipy softmax; closed forms (flat row, one raised token); probabilities of
 *                         all tokens of a row sum to one; the sum over iterations of a query.
 *   sbo_verify_sample   : the textbook identity of speculative sampling -- with the candidate drawn from
 *                         the draft distribution (one candidate, and two drawn without replacement) the
 *                         committed token is distributed exactly as the target -- checked by exact
 *                         integration over the uniforms (acceptance thresholds and bonus intervals found
 *                         by bisection on the oracle); T -> 0 reduces to greedy acceptance.  The paper
 *                         names the procedure only (rejection sampling): the order in which siblings
 *                         are tried and the treatment of the draft distribution after a rejection are
 *                         readings -- for those PARITY IS UNPINNED by the paper.
 *   sbo_shift_project   : numpy matmul on the explicitly concatenated input; W = [I, 0] returns the input,
 *                         W = [0, I] the previous position's state (the first position its own).
 *   sbo_fuse_project    : numpy (mean-square, concatenate, matmul) on a non-square W; closed forms for
 *                         W = [I, 0, 0] with constant and two-valued inputs; invariance under
 *                         rescaling an input when eps = 0; the difference between two positions of a
 *                         block does not depend on the start.  "norm" is not specified by the paper:
 *                         the RMS norm is a reading -- for the choice of norm PARITY IS UNPINNED.
 *   sbo_tree_expand     : hand-derived trees for the two printed branching maps; chain special
 *                         case; structural invariants.  The attach point of siblings, the cut
 *                         order at the node budget and the treatment of b = 0 are readings of
 *                         text the paper leaves open: for those rules PARITY IS UNPINNED.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SBO_MAX_NODES 128
#define SBO_KMAX 16

/* ---- exact widening of the storage types ------------------------------------------------ */

static double bf16_to_f64(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* NaN takes part in max/top-k as -infinity. */
static double score_of(double x) { return isnan(x) ? -INFINITY : x; }

/* ---- tree: ancestors and depth (App. A.2, Fig. 4) ----------------------------------------- */

/* 0 when parent[i] is -1 or an earlier node for every i and n <= 128, else 1. */
static int tree_is_valid(const int32_t* parent, int n) {
  if (n < 0 || n > SBO_MAX_NODES) return 0;
  for (int i = 0; i < n; ++i)
    if (parent[i] < -1 || parent[i] >= i) return 0;
  return 1;
}

/*
 * anc(i) = {i} U anc(parent[i]), anc(-1) = {}.  Writes, per node, a 128-bit set as four 32-bit
 * words (bit a of word a/32) and depth = |anc| - 1.  Returns 0, or 1 for an invalid tree (outputs
 * zeroed).
 */
int sbo_tree_ancestors(const int32_t* parent, int n, uint32_t* anc_mask, int32_t* depth) {
  if (anc_mask) memset(anc_mask, 0, sizeof(uint32_t) * 4 * (size_t)(n > 0 ? n : 0));
  if (depth) memset(depth, 0, sizeof(int32_t) * (size_t)(n > 0 ? n : 0));
  if (!tree_is_valid(parent, n)) return 1;
  for (int i = 0; i < n; ++i) {
    int d = -1;
    for (int a = i; a != -1; a = parent[a]) { /* walk i, parent(i), parent(parent(i)), ... */
      if (anc_mask) anc_mask[4 * i + a / 32] |= 1u << (a % 32);
      ++d;
    }
    if (depth) depth[i] = d;
  }
  return 0;
}

/* ---- cache addressing ------------------------------------------------------------------- */

typedef struct {
  int n_kv_heads, head_dim, page_size, max_pages, num_pages;
  int64_t kv_capacity;
  const int32_t* page_table;
} kv_layout;

/* Element offset of (sequence b, logical position j, kv head g, dim 0); -1 when out of range. */
static int64_t kv_row_offset(const kv_layout* L, int b, int64_t j, int g) {
  int64_t row;
  if (L->page_size == 0) {
    if (j < 0 || j >= L->kv_capacity) return -1;
    row = (int64_t)b * L->kv_capacity + j;
  } else {
    int64_t lp = j / L->page_size;
    if (j < 0 || lp >= L->max_pages) return -1;
    int32_t page = L->page_table[(int64_t)b * L->max_pages + lp];
    if (page < 0 || page >= L->num_pages) return -1;
    row = (int64_t)page * L->page_size + j % L->page_size;
  }
  return (row * L->n_kv_heads + g) * (int64_t)L->head_dim;
}

/* ---- O1: tree attention by its definition (Sec. 3.1; App. A.2; Alg. 1 "verify") ------------- */

/*
 * One query row: sequence b, node i, head h.  Lists the visible positions (whole prefix, then
 * the ancestors of i including i, at prefix_len + ancestor index), takes every score in fp64,
 * and forms the softmax-weighted sum in two plain passes.  Returns 0, or 1 when a position
 * falls outside the cache.
 */
static int attention_row(const kv_layout* L, const uint16_t* k, const uint16_t* v, int b, int P,
                         const int32_t* parent, int i, int h, int G, const uint16_t* qrow,
                         double scale, double* out, double* lse) {
  const int D = L->head_dim, g = h / G;
  int on_path[SBO_MAX_NODES];
  int n_path = 0;
  for (int a = i; a != -1; a = parent[a]) on_path[n_path++] = a;
  const int64_t n_vis = (int64_t)P + n_path;
  double* s = (double*)malloc(sizeof(double) * (size_t)n_vis);
  int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)n_vis);
  for (int64_t j = 0; j < P; ++j) pos[j] = j;
  for (int t = 0; t < n_path; ++t) pos[P + t] = (int64_t)P + on_path[n_path - 1 - t];
  int bad = 0;
  double m = -INFINITY;
  for (int64_t t = 0; t < n_vis; ++t) {
    int64_t off = kv_row_offset(L, b, pos[t], g);
    if (off < 0) { bad = 1; break; }
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += bf16_to_f64(qrow[d]) * bf16_to_f64(k[off + d]);
    s[t] = scale * acc;
    if (s[t] > m) m = s[t];
  }
  if (!bad) {
    double l = 0.0;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int64_t t = 0; t < n_vis; ++t) {
      double p = exp(s[t] - m);
      l += p;
      int64_t off = kv_row_offset(L, b, pos[t], g);
      for (int d = 0; d < D; ++d) out[d] += p * bf16_to_f64(v[off + d]);
    }
    for (int d = 0; d < D; ++d) out[d] /= l;
    *lse = m + log(l);
  }
  free(s);
  free(pos);
  return bad;
}

/*
 * Whole batch, or a selection of rows.
 *   k, v, q : bf16 bit patterns.  q [total_q][Hq][D]; sequence b's first query row is
 *   q_offsets[b] (NULL: node_offsets[b]); its first query node is q_node_begin[b] (NULL: 0).
 *   scale <= 0 means 1/sqrt(D).
 *   sel == NULL : every query row; out [total_q][Hq][D], lse [total_q][Hq].
 *   sel != NULL : n_sel triples (b, node, head); out [n_sel][D], lse [n_sel].
 *   status [batch]: 0 ok, 4 invalid tree, 5 position outside the cache (outputs of that
 *   sequence zero).  Returns the number of sequences with a non-zero status.
 */
int sbo_tree_attention(int batch, int n_q_heads, int n_kv_heads, int head_dim, const uint16_t* k,
                       const uint16_t* v, int page_size, int max_pages, int num_pages,
                       int64_t kv_capacity, const int32_t* page_table, const int32_t* prefix_len,
                       const int32_t* node_offsets, const int32_t* parent,
                       const int32_t* q_node_begin, const int32_t* q_offsets, const uint16_t* q,
                       double scale, int64_t n_sel, const int32_t* sel, double* out, double* lse,
                       int32_t* status) {
  kv_layout L = {n_kv_heads, head_dim, page_size, max_pages, num_pages, kv_capacity, page_table};
  const int D = head_dim, Hq = n_q_heads, G = n_q_heads / n_kv_heads;
  if (scale <= 0.0) scale = 1.0 / sqrt((double)D);
  for (int b = 0; b < batch; ++b) {
    int n = node_offsets[b + 1] - node_offsets[b];
    status[b] = tree_is_valid(parent + node_offsets[b], n) ? 0 : 4;
  }
  /* flat list of rows to compute */
  int64_t n_rows = 0;
  int32_t* rows; /* (b, node, head, out_row) */
  if (sel) {
    n_rows = n_sel;
    rows = (int32_t*)malloc(sizeof(int32_t) * 4 * (size_t)(n_rows > 0 ? n_rows : 1));
    for (int64_t r = 0; r < n_rows; ++r) {
      rows[4 * r + 0] = sel[3 * r + 0];
      rows[4 * r + 1] = sel[3 * r + 1];
      rows[4 * r + 2] = sel[3 * r + 2];
      rows[4 * r + 3] = (int32_t)r;
    }
  } else {
    for (int b = 0; b < batch; ++b) {
      int n = node_offsets[b + 1] - node_offsets[b];
      int q0 = q_node_begin ? q_node_begin[b] : 0;
      if (n > q0) n_rows += (int64_t)(n - q0) * Hq;
    }
    rows = (int32_t*)malloc(sizeof(int32_t) * 4 * (size_t)(n_rows > 0 ? n_rows : 1));
    int64_t r = 0;
    for (int b = 0; b < batch; ++b) {
      int n = node_offsets[b + 1] - node_offsets[b];
      int q0 = q_node_begin ? q_node_begin[b] : 0;
      int qoff = q_offsets ? q_offsets[b] : node_offsets[b];
      for (int i = q0; i < n; ++i)
        for (int h = 0; h < Hq; ++h) {
          rows[4 * r + 0] = b;
          rows[4 * r + 1] = i;
          rows[4 * r + 2] = h;
          rows[4 * r + 3] = (qoff + (i - q0)) * Hq + h;
          ++r;
        }
    }
  }
  int32_t* bad_seq = (int32_t*)calloc((size_t)batch, sizeof(int32_t));
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < n_rows; ++r) {
    int b = rows[4 * r + 0], i = rows[4 * r + 1], h = rows[4 * r + 2];
    int64_t orow = rows[4 * r + 3];
    double* o = out + orow * D;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    lse[orow] = 0.0;
    if (status[b] != 0) continue;
    int q0 = q_node_begin ? q_node_begin[b] : 0;
    int qoff = q_offsets ? q_offsets[b] : node_offsets[b];
    const uint16_t* qrow = q + ((int64_t)(qoff + (i - q0)) * Hq + h) * D;
    if (attention_row(&L, k, v, b, prefix_len[b], parent + node_offsets[b], i, h, G, qrow, scale,
                      o, &lse[orow])) {
#pragma omp atomic write
      bad_seq[b] = 1;
    }
  }
  int n_bad = 0;
  for (int b = 0; b < batch; ++b)
    if (bad_seq[b] && status[b] == 0) status[b] = 5;
  /* zero the outputs of sequences flagged after the fact */
  for (int64_t r = 0; r < n_rows; ++r) {
    int b = rows[4 * r + 0];
    if (status[b] != 0) {
      int64_t orow = rows[4 * r + 3];
      for (int d = 0; d < D; ++d) out[orow * D + d] = 0.0;
      lse[orow] = 0.0;
    }
  }
  for (int b = 0; b < batch; ++b) n_bad += status[b] != 0;
  free(bad_seq);
  free(rows);
  return n_bad;
}

/* ---- a4: per-row argmax, ties to the smallest id ------------------------------------------ */

static double logit_at(const void* logits, int dtype, int64_t idx) {
  if (dtype == 0) return score_of(bf16_to_f64(((const uint16_t*)logits)[idx]));
  return score_of((double)((const float*)logits)[idx]);
}

void sbo_row_argmax(const void* logits, int dtype, int64_t row_stride, int vocab, int64_t n_rows,
                    int32_t* amax) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < n_rows; ++r) {
    int best = 0;
    double bv = logit_at(logits, dtype, r * row_stride);
    for (int v = 1; v < vocab; ++v) {
      double x = logit_at(logits, dtype, r * row_stride + v);
      if (x > bv) { bv = x; best = v; } /* strict: the first (smallest) id keeps a tie */
    }
    amax[r] = best;
  }
}

/* ---- O2: greedy acceptance by enumerating every root-to-node path (App. A.5; Alg. 1) -------- */

/*
 * One sequence.  For every node, writes down the path root..node and checks each edge of it:
 * the child's token must be the target's greedy choice at the parent.  Keeps the deepest fully
 * matching path (ties: the smaller end node).  Returns 0 or 4 (invalid tree: node 0 must be the
 * only node with parent -1).
 */
static int accept_one(int n, const int32_t* parent, const int32_t* tok, const int32_t* amax,
                      int max_depth, int32_t* accept_len, int32_t* path_nodes,
                      int32_t* out_tokens, int32_t* bonus) {
  for (int t = 0; t <= max_depth; ++t) { path_nodes[t] = -1; out_tokens[t] = -1; }
  *accept_len = 0;
  *bonus = -1;
  if (n < 1 || !tree_is_valid(parent, n) || parent[0] != -1) return 4;
  for (int i = 1; i < n; ++i)
    if (parent[i] == -1) return 4;
  int best_len = -1, best_path[SBO_MAX_NODES];
  for (int i = 0; i < n; ++i) {
    int rev[SBO_MAX_NODES], len = 0;
    for (int a = i; a != -1; a = parent[a]) rev[len++] = a;
    int path[SBO_MAX_NODES];
    for (int t = 0; t < len; ++t) path[t] = rev[len - 1 - t]; /* root first */
    int ok = 1;
    for (int t = 1; t < len; ++t)
      if (tok[path[t]] != amax[path[t - 1]]) { ok = 0; break; }
    int drafted = len - 1;
    if (ok && drafted <= max_depth && drafted > best_len) { /* '>' keeps the smaller end node */
      best_len = drafted;
      memcpy(best_path, path, sizeof(int) * (size_t)len);
    }
  }
  *accept_len = best_len;
  for (int t = 0; t <= best_len; ++t) path_nodes[t] = best_path[t];
  for (int t = 1; t <= best_len; ++t) out_tokens[t - 1] = tok[best_path[t]];
  *bonus = amax[best_path[best_len]];
  out_tokens[best_len] = *bonus;
  return 0;
}

/*
 * Batch: argmax of every node's logits row, then accept_one per sequence.
 * amax [total], accept_len [B], path_nodes [B][max_depth+1], out_tokens [B][max_depth+1],
 * bonus [B], status [B].
 */
void sbo_verify_accept(const void* logits, int dtype, int64_t row_stride, int vocab, int batch,
                       const int32_t* node_offsets, const int32_t* parent, const int32_t* tok,
                       int max_depth, int32_t* amax, int32_t* accept_len, int32_t* path_nodes,
                       int32_t* out_tokens, int32_t* bonus, int32_t* status) {
  sbo_row_argmax(logits, dtype, row_stride, vocab, node_offsets[batch], amax);
  for (int b = 0; b < batch; ++b) {
    int o = node_offsets[b], n = node_offsets[b + 1] - o;
    status[b] = accept_one(n, parent + o, tok + o, amax + o, max_depth, &accept_len[b],
                           path_nodes + (int64_t)b * (max_depth + 1),
                           out_tokens + (int64_t)b * (max_depth + 1), &bonus[b]);
  }
}

/* Acceptance alone, from given per-node greedy choices (for exhaustive small-tree tests). */
int sbo_accept_from_amax(int n, const int32_t* parent, const int32_t* tok, const int32_t* amax,
                         int max_depth, int32_t* accept_len, int32_t* path_nodes,
                         int32_t* out_tokens, int32_t* bonus) {
  return accept_one(n, parent, tok, amax, max_depth, accept_len, path_nodes, out_tokens, bonus);
}

/* ---- the accepted path in the drafter's row numbering (App. A.2) ----------------------------- */

/*
 * A draft forward produces one cache row per block position; the tokens attached at a position share
 * it.  node_row[i] is the row (in the numbering of all rows of the iteration, first row of sequence
 * b = row_begin[b]) of the position whose distribution proposed tree node i, -1 for the root.  For the
 * accepted path p_0 = 0, ..., p_a: rows[0] = 0 (the last committed position, one slot before the
 * iteration's rows) and rows[j] = 1 + node_row[p_j] - row_begin[b]; entries past a are -1.
 * status 0 ok / 4 when a is outside [0, max_depth], a path node is outside the tree or has no row,
 * or the rows do not increase (rows then 0, -1, -1, ...).
 */
void sbo_path_rows(int batch, const int32_t* node_offsets, const int32_t* node_row, const int32_t* row_begin,
                   const int32_t* path_nodes, const int32_t* accept_len, int max_depth, int32_t* rows,
                   int32_t* status) {
  for (int b = 0; b < batch; ++b) {
    const int o = node_offsets[b], n = node_offsets[b + 1] - o, a = accept_len[b];
    const int r0 = row_begin ? row_begin[b] : 0;
    const int32_t* path = path_nodes + (int64_t)b * (max_depth + 1);
    int32_t* out = rows + (int64_t)b * (max_depth + 1);
    int bad = n < 1 || a < 0 || a > max_depth;
    for (int j = 0; j <= max_depth; ++j) out[j] = -1;
    out[0] = 0;
    for (int j = 1; !bad && j <= a; ++j) {
      const int p = path[j];
      if (p < 0 || p >= n || node_row[o + p] < r0 || node_row[o + p] < 0) { bad = 1; break; }
      out[j] = 1 + node_row[o + p] - r0;
      if (out[j] <= out[j - 1]) bad = 1;
    }
    if (bad) {
      for (int j = 1; j <= max_depth; ++j) out[j] = -1;
    }
    status[b] = bad ? 4 : 0;
  }
}

/* ---- O3: cache compaction as an out-of-place gather ---------------------------------------- */

/*
 * cache_old / cache_new: bf16 bit patterns, n_layers caches laid out layer_stride_elems apart,
 * each in the layout described by (page_size, ...).  cache_new must start as a copy of cache_old;
 * this routine then writes new[P+j] = old[P+path[j]] for j = 0..accept_len, every layer, every kv
 * head.  Call once for K and once for V.  status 0 ok / 4 bad path / 5 outside the cache.
 */
void sbo_kv_compact(int batch, int n_kv_heads, int head_dim, const uint16_t* cache_old,
                    uint16_t* cache_new, int n_layers, int64_t layer_stride_elems, int page_size,
                    int max_pages, int num_pages, int64_t kv_capacity, const int32_t* page_table,
                    const int32_t* prefix_len, const int32_t* node_offsets,
                    const int32_t* path_nodes, const int32_t* accept_len, int max_depth,
                    int32_t* new_len, int32_t* status) {
  kv_layout L = {n_kv_heads, head_dim, page_size, max_pages, num_pages, kv_capacity, page_table};
  for (int b = 0; b < batch; ++b) {
    const int n = node_offsets[b + 1] - node_offsets[b], P = prefix_len[b], a = accept_len[b];
    const int32_t* path = path_nodes + (int64_t)b * (max_depth + 1);
    status[b] = 0;
    new_len[b] = P;
    if (a < 0 || a > max_depth || path[0] != 0) { status[b] = 4; continue; }
    for (int j = 1; j <= a; ++j)
      if (path[j] <= path[j - 1] || path[j] >= n) status[b] = 4;
    if (status[b]) continue;
    for (int j = 0; j <= a; ++j)
      if (kv_row_offset(&L, b, (int64_t)P + path[j], 0) < 0) status[b] = 5;
    if (status[b]) continue;
    for (int l = 0; l < n_layers; ++l)
      for (int j = 0; j <= a; ++j)
        for (int g = 0; g < n_kv_heads; ++g) {
          int64_t src = kv_row_offset(&L, b, (int64_t)P + path[j], g) + l * layer_stride_elems;
          int64_t dst = kv_row_offset(&L, b, (int64_t)P + j, g) + l * layer_stride_elems;
          memcpy(cache_new + dst, cache_old + src, sizeof(uint16_t) * (size_t)head_dim);
        }
    new_len[b] = P + a + 1;
  }
}

/* ---- a7: per-row top-k by a full sort ---------------------------------------------------- */

typedef struct { double val; int32_t id; } scored;

static int by_score_desc_id_asc(const void* pa, const void* pb) {
  const scored *a = (const scored*)pa, *b = (const scored*)pb;
  if (a->val > b->val) return -1;
  if (a->val < b->val) return 1;
  return (a->id > b->id) - (a->id < b->id);
}

/* topk_tok [n_rows][16], topk_val [n_rows][16]; ranks beyond vocab get -1 / -inf. */
void sbo_row_topk(const float* scores, int64_t row_stride, int n_rows, int vocab,
                  int32_t* topk_tok, float* topk_val) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    scored* e = (scored*)malloc(sizeof(scored) * (size_t)vocab);
    for (int v = 0; v < vocab; ++v) {
      e[v].val = score_of((double)scores[(int64_t)r * row_stride + v]);
      e[v].id = v;
    }
    qsort(e, (size_t)vocab, sizeof(scored), by_score_desc_id_asc);
    for (int j = 0; j < SBO_KMAX; ++j) {
      topk_tok[r * SBO_KMAX + j] = j < vocab ? e[j].id : -1;
      topk_val[r * SBO_KMAX + j] = j < vocab ? (float)e[j].val : -INFINITY;
    }
    free(e);
  }
}

/* ---- O4: bucket-driven branching (Sec. 3.2; App. A.5; Alg. 1 "attach") ------------------------ */

/*
 * Steps, in the order the paper states them: top candidates per (start, position) row;
 * branching width from the bucket through the map b(.); attach the top-b tokens under the
 * chain node of the previous position of the same block (position 0: under the block's start
 * node); stop when the node budget is reached.  Returns 0, or 1 for a bad argument (bucket > 3,
 * start parent that does not exist, width > 16).
 */
int sbo_tree_expand(const float* scores, int64_t row_stride, int n_rows, int vocab, int block_k,
                    const uint8_t* bucket, const int32_t* bmap, const int32_t* start_parent,
                    int node_budget, int32_t* n_nodes, int32_t* tok, int32_t* parent,
                    int32_t* depth, int32_t* node_row, int32_t* node_rank, int32_t* topk_tok,
                    float* topk_val) {
  sbo_row_topk(scores, row_stride, n_rows, vocab, topk_tok, topk_val);
  int n = *n_nodes;
  if (n < 0 || n > node_budget || block_k < 1 || n_rows % block_k != 0) return 1;
  for (int m = 0; m < 4; ++m)
    if (bmap[m] < 0 || bmap[m] > SBO_KMAX) return 1;
  const int n_existing = n;
  for (int r = 0; r < n_rows; ++r)
    if (bucket[r] > 3) return 1;
  for (int i = 0; i < n_rows / block_k; ++i)
    if (start_parent[i] < -1 || start_parent[i] >= n_existing) return 1;
  int chain = -1;       /* node created for (previous row of this block, rank 0) */
  int chain_alive = 0;  /* does that node exist */
  for (int r = 0; r < n_rows; ++r) {
    const int i = r / block_k, kpos = r % block_k;
    int b = bmap[bucket[r]];
    if (b > vocab) b = vocab;
    int attach, alive;
    if (kpos == 0) {
      attach = start_parent[i];
      alive = 1;
    } else {
      attach = chain;
      alive = chain_alive;
    }
    chain_alive = 0;
    if (!alive) continue;
    for (int j = 0; j < b; ++j) {
      if (n >= node_budget) break;
      tok[n] = topk_tok[r * SBO_KMAX + j];
      parent[n] = attach;
      depth[n] = attach == -1 ? 0 : depth[attach] + 1;
      node_row[n] = r;
      node_rank[n] = j;
      if (j == 0) { chain = n; chain_alive = 1; }
      ++n;
    }
  }
  *n_nodes = n;
  return 0;
}

/* ---- psi(p): the rank head's 15-dimensional summary of a draft distribution (App. B) ----------- */

/*
 * For every row of drafter scores (logits), with p = softmax(row) (NaN scores count as -inf):
 *   features[0..9]  natural-log probabilities of the ten most likely tokens, most likely first
 *                   (value descending, id ascending; -inf where the vocabulary has fewer than ten);
 *   features[10..12] logit gaps between the top token and the tokens of rank 2, 3 and 5
 *                   (+inf where that rank does not exist);
 *   features[13]    probability of the top token;
 *   features[14]    entropy -sum p ln p in nats (terms with p = 0 contribute nothing).
 * Plain definition: exact maximum, fp64 log-sum-exp over the whole row, full sort.
 */
void sbo_rank_features(const float* scores, int64_t row_stride, int n_rows, int vocab, double* features) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    scored* e = (scored*)malloc(sizeof(scored) * (size_t)vocab);
    double m = -INFINITY;
    for (int v = 0; v < vocab; ++v) {
      e[v].val = score_of((double)scores[(int64_t)r * row_stride + v]);
      e[v].id = v;
      if (e[v].val > m) m = e[v].val;
    }
    double* f = features + (int64_t)r * 15;
    if (m == -INFINITY) { /* no finite score: the distribution is undefined; report a flat one */
      m = 0.0;
      for (int v = 0; v < vocab; ++v) e[v].val = 0.0;
    }
    double z = 0.0;
    for (int v = 0; v < vocab; ++v) z += exp(e[v].val - m);
    const double log_z = m + log(z);
    double entropy = 0.0;
    for (int v = 0; v < vocab; ++v) {
      const double lp = e[v].val - log_z;
      if (lp > -INFINITY) entropy -= exp(lp) * lp;
    }
    qsort(e, (size_t)vocab, sizeof(scored), by_score_desc_id_asc);
    for (int j = 0; j < 10; ++j) f[j] = j < vocab ? e[j].val - log_z : -INFINITY;
    f[10] = vocab > 1 ? e[0].val - e[1].val : INFINITY;
    f[11] = vocab > 2 ? e[0].val - e[2].val : INFINITY;
    f[12] = vocab > 4 ? e[0].val - e[4].val : INFINITY;
    f[13] = exp(e[0].val - log_z);
    f[14] = entropy;
    free(e);
  }
}

/* ---- layer-wise shift between the drafter's decoder layers (Sec. 3.1, the equation for h-tilde) -- */

/*
 * Rows r = i * block_k + k are the K positions of block i.  Before the next layer, position k's
 * state is concatenated with position k-1's state of the same block (the first position with its
 * own) and projected back to d_out features:
 *   out[r][f] = sum_j w[f][j] * h[r][j] + sum_j w[f][d + j] * h[prev(r)][j],
 *   prev(r) = r - 1 if r % block_k != 0 else r.
 * h bf16 [n_rows][d], w bf16 [d_out][2 d] (the projection acting on the concatenation), out f64.
 * block_k = 0: plain projection out = h w^T with w [d_out][d].
 */
void sbo_shift_project(const uint16_t* h, const uint16_t* w, int n_rows, int d, int d_out, int block_k,
                       double* out) {
  const int kin = block_k > 0 ? 2 * d : d;
#pragma omp parallel for schedule(static)
  for (int r = 0; r < n_rows; ++r) {
    const int prev = (block_k > 0 && r % block_k != 0) ? r - 1 : r;
    for (int f = 0; f < d_out; ++f) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j) acc += bf16_to_f64(w[(int64_t)f * kin + j]) * bf16_to_f64(h[(int64_t)r * d + j]);
      if (block_k > 0)
        for (int j = 0; j < d; ++j)
          acc += bf16_to_f64(w[(int64_t)f * kin + d + j]) * bf16_to_f64(h[(int64_t)prev * d + j]);
      out[(int64_t)r * d_out + f] = acc;
    }
  }
}

/* ---- the drafter's per-position input (Sec. 3.1, the equation for h^(0)) -------------------------- */

/*
 * h0[s * K + k] = W_fuse [ norm(c_s), norm(e_s), norm(q_k) ]:  c_s the context feature of start s,
 * e_s the embedding of its last committed token (both shared by the K positions of the block: the
 * prefix broadcast), q_k the learnable query of draft depth k.  The paper says only "normalized";
 * read as the root-mean-square norm of the target's architecture with a learnable gain,
 *   norm(x)[j] = g[j] * x[j] / sqrt(mean_j x[j]^2 + eps)        (g = NULL: all ones).
 * c, e bf16 [n_starts][d], q bf16 [block_k][d], gains f32 [d], w bf16 [d_out][3 d], out f64
 * [n_starts * block_k][d_out].
 */
static void rms_norm_f64(const uint16_t* x, const float* g, int d, double eps, double* y) {
  double ss = 0.0;
  for (int j = 0; j < d; ++j) { const double v = bf16_to_f64(x[j]); ss += v * v; }
  const double inv = 1.0 / sqrt(ss / d + eps);
  for (int j = 0; j < d; ++j) y[j] = (g ? (double)g[j] : 1.0) * bf16_to_f64(x[j]) * inv;
}

void sbo_fuse_project(const uint16_t* c, const uint16_t* e, const uint16_t* q, const float* gain_c,
                      const float* gain_e, const float* gain_q, double eps, const uint16_t* w, int n_starts,
                      int block_k, int d, int d_out, double* out) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < n_starts * block_k; ++r) {
    const int s = r / block_k, k = r % block_k;
    double* x = (double*)malloc(sizeof(double) * 3 * d);  /* the concatenation of the equation */
    rms_norm_f64(c + (int64_t)s * d, gain_c, d, eps, x);
    rms_norm_f64(e + (int64_t)s * d, gain_e, d, eps, x + d);
    rms_norm_f64(q + (int64_t)k * d, gain_q, d, eps, x + 2 * d);
    for (int f = 0; f < d_out; ++f) {
      double acc = 0.0;
      for (int j = 0; j < 3 * d; ++j) acc += bf16_to_f64(w[(int64_t)f * 3 * d + j]) * x[j];
      out[(int64_t)r * d_out + f] = acc;
    }
    free(x);
  }
}

/* ---- stochastic verification of a draft tree (Sec. 4.1 "temperature 0 and 1.0"; Sec. 4.2) ------- */

/*
 * The paper verifies at temperature 1 by rejection sampling against the target without giving
 * the procedure; this is the multi-candidate rejection sampling of tree-based speculative decoding
 * (the systems it compares with), taken in the order below.  All random numbers are inputs.
 *
 *   node a = root (0), depth 0, p = softmax(logits[a] / T).
 *   repeat:
 *     children of a = the nodes c with parent[c] == a, in increasing index (= emission order).
 *     no children, or depth == max_depth: stop.
 *     q = softmax(scores[child_row[a]] / T)   (the draft distribution that proposed them).
 *     for each child c in order, x = tok[c]:
 *         accept c iff  u_accept[c] < p(x) / q(x)   (q(x) = 0: accepted iff p(x) > 0);
 *         accepted: a = c, depth += 1, p = softmax(logits[c] / T), next round;
 *         rejected: p <- max(p - q, 0) renormalised (left as it is if nothing remains),
 *                   q(x) <- 0 and q renormalised (x was drawn without replacement).
 *     every child rejected: stop.
 *   bonus = the smallest v with  sum_{w <= v} p(w) > u_bonus * sum_w p(w)  (the last v with
 *   p(v) > 0 if rounding leaves none), p being the (possibly residual) distribution at the stop.
 * Outputs as sbo_verify_accept: accept_len = depth, path_nodes, out_tokens = accepted tokens then
 * bonus.  status 4: invalid tree; 5: child_row of an inner node on the walk outside [0, n_rows).
 * NaN logits/scores count as -inf; a row without a finite value is flat.
 */
static void softmax_row_f64(const void* row, int dtype, int64_t base, int vocab, double inv_t, double* out) {
  double m = -INFINITY;
  for (int v = 0; v < vocab; ++v) {
    const double x = score_of(logit_at(row, dtype, base + v));
    if (x > m) m = x;
  }
  double z = 0.0;
  for (int v = 0; v < vocab; ++v) {
    const double x = score_of(logit_at(row, dtype, base + v));
    out[v] = m == -INFINITY ? 1.0 : exp((x - m) * inv_t);
    z += out[v];
  }
  for (int v = 0; v < vocab; ++v) out[v] /= z;
}

void sbo_verify_sample(const void* logits, int dtype, int64_t row_stride, int vocab, const float* scores,
                       int64_t score_stride, int n_rows, int batch, const int32_t* node_offsets,
                       const int32_t* parent, const int32_t* tok, const int32_t* child_row, double temperature,
                       const float* u_accept, const float* u_bonus, int max_depth, int32_t* accept_len,
                       int32_t* path_nodes, int32_t* out_tokens, int32_t* bonus, int32_t* status) {
  const double inv_t = 1.0 / temperature;
  double* p = (double*)malloc(sizeof(double) * (size_t)vocab);
  double* q = (double*)malloc(sizeof(double) * (size_t)vocab);
  for (int b = 0; b < batch; ++b) {
    const int o = node_offsets[b], n = node_offsets[b + 1] - o;
    const int32_t *par = parent + o, *tk = tok + o;
    int32_t* path = path_nodes + (int64_t)b * (max_depth + 1);
    int32_t* otok = out_tokens + (int64_t)b * (max_depth + 1);
    for (int t = 0; t <= max_depth; ++t) { path[t] = -1; otok[t] = -1; }
    accept_len[b] = 0;
    bonus[b] = -1;
    status[b] = 0;
    int valid = n >= 1 && tree_is_valid(par, n) && par[0] == -1;
    for (int i = 1; valid && i < n; ++i)
      if (par[i] == -1) valid = 0;
    if (!valid) { status[b] = 4; continue; }
    int a = 0, depth = 0;
    path[0] = 0;
    softmax_row_f64(logits, dtype, (int64_t)(o + a) * row_stride, vocab, inv_t, p);
    for (;;) {
      int first_child = -1;
      for (int c = a + 1; c < n; ++c)
        if (par[c] == a) { first_child = c; break; }
      if (first_child < 0 || depth == max_depth) break;
      const int row = child_row[o + a];
      if (row < 0 || row >= n_rows) { status[b] = 5; break; }
      softmax_row_f64(scores, 1, (int64_t)row * score_stride, vocab, inv_t, q);
      int accepted = -1;
      for (int c = first_child; c < n; ++c) {
        if (par[c] != a) continue;
        const int x = tk[c];
        const double px = (x >= 0 && x < vocab) ? p[x] : 0.0;
        const double qx = (x >= 0 && x < vocab) ? q[x] : 0.0;
        const int take = qx > 0.0 ? ((double)u_accept[o + c] < px / qx) : (px > 0.0);
        if (take) { accepted = c; break; }
        /* rejected: residual target, and the token leaves the draft distribution */
        double z = 0.0;
        for (int v = 0; v < vocab; ++v) z += p[v] > q[v] ? p[v] - q[v] : 0.0;
        if (z > 0.0)
          for (int v = 0; v < vocab; ++v) p[v] = (p[v] > q[v] ? p[v] - q[v] : 0.0) / z;
        if (x >= 0 && x < vocab) {
          q[x] = 0.0;
          double zq = 0.0;
          for (int v = 0; v < vocab; ++v) zq += q[v];
          if (zq > 0.0)
            for (int v = 0; v < vocab; ++v) q[v] /= zq;
        }
      }
      if (accepted < 0) break;
      a = accepted;
      ++depth;
      path[depth] = a;
      otok[depth - 1] = tk[a];
      softmax_row_f64(logits, dtype, (int64_t)(o + a) * row_stride, vocab, inv_t, p);
    }
    if (status[b]) {
      for (int t = 0; t <= max_depth; ++t) { path[t] = -1; otok[t] = -1; }
      continue;
    }
    double total = 0.0;
    for (int v = 0; v < vocab; ++v) total += p[v];
    const double target = (double)u_bonus[b] * total;
    double cum = 0.0;
    int pick = -1, last_pos = -1;
    for (int v = 0; v < vocab; ++v) {
      if (p[v] > 0.0) last_pos = v;
      cum += p[v];
      if (cum > target) { pick = v; break; }
    }
    if (pick < 0) pick = last_pos;
    accept_len[b] = depth;
    bonus[b] = pick;
    otok[depth] = pick;
  }
  free(p);
  free(q);
}

/* ---- verifier-derived update signal (Sec. 3.4, the equation for s; Alg. 2 line 2) ------------- */

/*
 * s = sum over rejected positions of (1 - r), r = the drafter's probability of the token the
 * target chose at that position.  One verify iteration rejects at most one position per sequence:
 * the one right after the last accepted node `best` = path_nodes[b][accept_len[b]], where the
 * target chose bonus[b].  child_row[node] names the row of `scores` (drafter logits) that
 * predicted the token following `node`, or -1 when nothing was drafted there (then nothing was
 * rejected: r_prob = -1 and the sum is left alone).
 *   r = softmax(scores[row])[bonus] by the plain definition in fp64 (NaN scores count as -inf; a
 *   row without a finite score is flat; a token outside [0, vocab) has probability 0);
 *   r_prob[b] = r;  signal[b] += 1 - r   (signal is in/out: the caller zeroes it per query).
 * status[b] = 5 (and r_prob = -1, signal untouched) when accept_len, the path node or the row
 * index is out of range.
 */
void sbo_verifier_signal(const float* scores, int64_t row_stride, int n_rows, int vocab, int batch,
                         const int32_t* node_offsets, const int32_t* child_row, const int32_t* path_nodes,
                         const int32_t* accept_len, const int32_t* bonus, int max_depth, double* r_prob,
                         double* signal, int32_t* status) {
  for (int b = 0; b < batch; ++b) {
    const int o = node_offsets[b], n = node_offsets[b + 1] - o;
    const int a = accept_len[b];
    status[b] = 0;
    r_prob[b] = -1.0;
    if (a < 0 || a > max_depth) { status[b] = 5; continue; }
    const int best = path_nodes[(int64_t)b * (max_depth + 1) + a];
    if (best < 0 || best >= n) { status[b] = 5; continue; }
    const int row = child_row[o + best];
    if (row < 0) continue; /* nothing drafted after the last accepted node */
    if (row >= n_rows) { status[b] = 5; continue; }
    const float* x = scores + (int64_t)row * row_stride;
    const int t = bonus[b];
    double m = -INFINITY;
    for (int v = 0; v < vocab; ++v) {
      const double xv = score_of((double)x[v]);
      if (xv > m) m = xv;
    }
    double r;
    if (t < 0 || t >= vocab) {
      r = 0.0;
    } else if (m == -INFINITY) {
      r = 1.0 / (double)vocab;
    } else {
      double z = 0.0;
      for (int v = 0; v < vocab; ++v) z += exp(score_of((double)x[v]) - m);
      r = exp(score_of((double)x[t]) - m) / z;
    }
    r_prob[b] = r;
    signal[b] += 1.0 - r;
  }
}

/* Threads the OpenMP loops above use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int sbo_num_threads(void) { return omp_get_max_threads(); }
#else
int sbo_num_threads(void) { return 1; }
#endif
