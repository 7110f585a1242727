"""Seeded synthetic inputs for the SpecBlock hot path (numpy only).

This module is shared by the tests of the CPU oracle and of the CUDA library and by the
benchmark.  It holds no arithmetic of the method itself: it draws random tensors, random tree
shapes, page tables and logits with a planted accepted path, in the shapes and value
distributions of the paper's workloads (8B-class heads, K=4 blocks, trees of at most 60 nodes,
vocabulary 128256, Table-3 bucket frequencies).  It imports neither the oracle nor the CUDA
binding.  bf16 tensors are returned as uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

# Rank-bucket frequencies b0..b3 of the rank head (Table 3) -- used only to draw buckets.
BUCKET_FREQ = (0.752, 0.150, 0.041, 0.057)
# Chain acceptance alpha_1..alpha_8 for the Llama-3.1-8B drafter (Fig. 5a) -- used only to draw
# planted acceptance lengths.
CHAIN_ACCEPT = (0.835, 0.722, 0.674, 0.638, 0.661, 0.626, 0.588, 0.544)


def rng_for(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


# ---- bf16 storage -------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit pattern (uint16).  Finite inputs only."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng, shape, std=1.0) -> np.ndarray:
    """N(0, std^2) rounded to bf16, drawn in slabs to bound host memory."""
    n = int(np.prod(shape))
    out = np.empty(n, np.uint16)
    step = 1 << 24
    for s in range(0, n, step):
        e = min(n, s + step)
        x = rng.standard_normal(e - s, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[s:e] = f32_to_bf16_bits(x)
    return out.reshape(shape)


# ---- tree shapes ----------------------------------------------------------------------------

def tree_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), np.int32)
    for i, p in enumerate(parent):
        d[i] = 0 if p < 0 else d[p] + 1
    return d


def random_tree(rng, n: int, max_depth: int) -> np.ndarray:
    """Node 0 is the root (parent -1); node i>0 hangs under a uniformly drawn earlier node
    whose depth is below max_depth."""
    parent = np.full(n, -1, np.int32)
    depth = np.zeros(n, np.int32)
    for i in range(1, n):
        cand = np.flatnonzero(depth[:i] < max_depth)
        p = int(cand[rng.integers(len(cand))])
        parent[i] = p
        depth[i] = depth[p] + 1
    return parent


def chain_tree(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def _block_tree_once(rng, n_nodes, K, M, geom_p, bmax):
    """Shape of a SpecBlock draft tree: a root, then M levels of K-position blocks.  Inside a
    block, position k carries b = min(bmax, Geometric(geom_p)) sibling candidates under the
    first candidate ("chain" node) of position k-1 (position 0 under the block's start node).
    Next-level blocks start from every non-chain sibling and from the chain's end."""
    parent = [-1]
    starts = [0]
    for _level in range(M):
        next_starts = []
        for s in starts:
            attach = s
            for _k in range(K):
                b = int(min(bmax, rng.geometric(geom_p)))
                first = len(parent)
                for _j in range(b):
                    parent.append(attach)
                next_starts.extend(range(first + 1, first + b))
                attach = first
            next_starts.append(attach)
        starts = next_starts
    return np.asarray(parent[:n_nodes], np.int32), len(parent)


def block_tree(rng, n_nodes=60, K=4, M=2, geom_p=0.5, bmax=4) -> np.ndarray:
    """Redraw until the M-level tree reaches n_nodes, then cut at n_nodes in emission order."""
    for _ in range(10000):
        parent, made = _block_tree_once(rng, n_nodes, K, M, geom_p, bmax)
        if made >= n_nodes:
            return parent
    raise RuntimeError("block_tree: could not reach %d nodes" % n_nodes)


def drafter_block_tree(K=4):
    """Config-3 shape: a cached level-1 block (K-chain under the prefix), two cached level-2
    blocks started from two different level-1 nodes, and 8 new K-blocks, one per cached
    level-2 node.  Returns (parent, q_node_begin)."""
    parent = []
    for k in range(K):                      # level 1: nodes 0..K-1
        parent.append(k - 1)
    for start in (1, K - 1):                # level 2: two blocks, from level-1 nodes 1 and K-1
        attach = start
        for _k in range(K):
            parent.append(attach)
            attach = len(parent) - 1
    n_cached = len(parent)
    for start in range(K, n_cached):        # 8 new blocks, one per level-2 node
        attach = start
        for _k in range(K):
            parent.append(attach)
            attach = len(parent) - 1
    return np.asarray(parent, np.int32), n_cached


# ---- attention inputs -------------------------------------------------------------------------

@dataclass
class AttnCase:
    """One layer's tree-attention problem.  bf16 arrays are uint16 bit patterns."""
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int            # 0 = contiguous
    kv_capacity: int          # contiguous: positions per sequence
    num_pages: int
    max_pages: int
    k: np.ndarray             # contiguous [B,cap,Hkv,D] / paged [pages,ps,Hkv,D]
    v: np.ndarray
    page_table: Optional[np.ndarray]   # [B,max_pages]
    prefix_len: np.ndarray    # [B]
    node_offsets: np.ndarray  # [B+1]
    parent: np.ndarray        # [total_nodes]
    q_node_begin: Optional[np.ndarray]  # [B] or None
    q_offsets: Optional[np.ndarray]     # [B+1] or None
    q: np.ndarray             # [total_q,Hq,D]
    scale: float = 0.0
    extra: dict = field(default_factory=dict)

    @property
    def batch(self):
        return len(self.prefix_len)

    @property
    def total_q(self):
        return self.q.shape[0]

    @property
    def max_nodes(self):
        return int(np.max(np.diff(self.node_offsets)))

    @property
    def max_kv_len(self):
        return int(np.max(self.prefix_len + np.diff(self.node_offsets)))

    def oracle_kwargs(self):
        return dict(n_q_heads=self.n_q_heads, n_kv_heads=self.n_kv_heads, head_dim=self.head_dim,
                    k=self.k, v=self.v, page_size=self.page_size, max_pages=self.max_pages,
                    num_pages=self.num_pages, kv_capacity=self.kv_capacity,
                    page_table=self.page_table, prefix_len=self.prefix_len,
                    node_offsets=self.node_offsets, parent=self.parent, q=self.q,
                    q_node_begin=self.q_node_begin, q_offsets=self.q_offsets, scale=self.scale)

    def kv_bytes(self):
        """Algorithmic K+V bytes one layer call must read."""
        lens = self.prefix_len.astype(np.int64) + np.diff(self.node_offsets)
        return int(lens.sum()) * self.n_kv_heads * self.head_dim * 2 * 2

    def algorithmic_bytes(self):
        """K and V once, Q in, O out, LSE out."""
        qo = 2 * self.total_q * self.n_q_heads * self.head_dim * 2
        return self.kv_bytes() + qo + self.total_q * self.n_q_heads * 4

    def flops(self):
        lens = self.prefix_len.astype(np.int64) + np.diff(self.node_offsets)
        nq = np.diff(self.node_offsets).astype(np.int64)
        if self.q_node_begin is not None:
            nq = nq - self.q_node_begin
        return int((nq * lens).sum()) * self.n_q_heads * self.head_dim * 4


def make_attn_case(rng, *, parents, prefix_lens, n_q_heads, n_kv_heads, head_dim, page_size=0,
                   q_node_begin=None, q_std=1.0, kv_std=1.0, slack_pages=3, scale=0.0,
                   capacity_pad=0) -> AttnCase:
    """Random Q/K/V ~ N(0, std^2) in bf16 for the given trees and prefix lengths.  Paged caches
    get a pool with `slack_pages` unused pages and a page table that is a random permutation of
    the pool (unused table entries hold -1)."""
    B = len(parents)
    n_nodes = np.asarray([len(p) for p in parents], np.int32)
    node_offsets = np.concatenate([[0], np.cumsum(n_nodes)]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32) if B else np.zeros(0, np.int32)
    prefix_len = np.asarray(prefix_lens, np.int32)
    lens = prefix_len + n_nodes
    if q_node_begin is not None:
        q_node_begin = np.asarray(q_node_begin, np.int32)
        nq = n_nodes - q_node_begin
        q_offsets = np.concatenate([[0], np.cumsum(nq)]).astype(np.int32)
    else:
        nq = n_nodes
        q_offsets = None
    total_q = int(nq.sum())
    q = normal_bf16(rng, (total_q, n_q_heads, head_dim), q_std)
    if page_size == 0:
        cap = int(lens.max()) + capacity_pad
        k = normal_bf16(rng, (B, cap, n_kv_heads, head_dim), kv_std)
        v = normal_bf16(rng, (B, cap, n_kv_heads, head_dim), kv_std)
        return AttnCase(n_q_heads, n_kv_heads, head_dim, 0, cap, 0, 0, k, v, None, prefix_len,
                        node_offsets, parent, q_node_begin, q_offsets, q, scale)
    pages_per_seq = (lens + page_size - 1) // page_size
    max_pages = int(pages_per_seq.max()) + 1
    num_pages = int(pages_per_seq.sum()) + slack_pages
    perm = rng.permutation(num_pages).astype(np.int32)
    page_table = np.full((B, max_pages), -1, np.int32)
    at = 0
    for b in range(B):
        page_table[b, :pages_per_seq[b]] = perm[at:at + pages_per_seq[b]]
        at += pages_per_seq[b]
    k = normal_bf16(rng, (num_pages, page_size, n_kv_heads, head_dim), kv_std)
    v = normal_bf16(rng, (num_pages, page_size, n_kv_heads, head_dim), kv_std)
    return AttnCase(n_q_heads, n_kv_heads, head_dim, page_size, 0, num_pages, max_pages, k, v,
                    page_table, prefix_len, node_offsets, parent, q_node_begin, q_offsets, q,
                    scale)


def kv_slot(case: AttnCase, b: int, pos: int):
    """Index tuple of logical position `pos` of sequence b in case.k / case.v (first 2 axes)."""
    if case.page_size == 0:
        return (b, pos)
    return (int(case.page_table[b, pos // case.page_size]), pos % case.page_size)


# ---- verification inputs ---------------------------------------------------------------------

@dataclass
class VerifyCase:
    logits: np.ndarray        # [total_nodes, V] float32, or uint16 bf16 bits
    tok: np.ndarray           # [total_nodes]
    node_offsets: np.ndarray
    parent: np.ndarray
    max_depth: int
    planted_len: np.ndarray   # [B] drafted tokens planted as accepted
    planted_path: list        # per sequence: node ids root..end of the planted path
    planted_bonus: np.ndarray # [B]


def _children_lists(parent):
    ch = [[] for _ in parent]
    for i, p in enumerate(parent):
        if p >= 0:
            ch[p].append(i)
    return ch


def make_verify_case(rng, *, parents, vocab, dtype="f32", std=2.0, accept_lens=None,
                     max_depth=None) -> VerifyCase:
    """Target logits ~ N(0, std^2) per tree node and drafted tokens with one planted path.

    For each sequence a root-to-node path of the wanted number of drafted tokens (clipped to
    what the tree has) is drawn at random; along it logits[parent][tok[child]] is raised to
    rowmax + 4 so the child's token is the unique row maximum; at the path's end the same is
    done for a bonus token that none of its children carries.  Every other child token is
    drawn among ids that do not attain its parent's row maximum, so no other edge can match.
    Sibling tokens under one parent are distinct.  All other rows keep their natural maxima
    (in bf16 these are frequently tied)."""
    B = len(parents)
    n_nodes = np.asarray([len(p) for p in parents], np.int32)
    node_offsets = np.concatenate([[0], np.cumsum(n_nodes)]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    total = int(n_nodes.sum())
    x = rng.standard_normal((total, vocab), dtype=np.float32) * np.float32(std)
    if dtype == "bf16":
        x = bf16_bits_to_f32(f32_to_bf16_bits(x))
    tok = np.zeros(total, np.int32)
    planted_len = np.zeros(B, np.int32)
    planted_bonus = np.zeros(B, np.int32)
    planted_path = []
    tree_max_depth = 0
    for b in range(B):
        o = int(node_offsets[b])
        par = parents[b]
        depth = tree_depths(par)
        tree_max_depth = max(tree_max_depth, int(depth.max()))
        ch = _children_lists(par)
        want = int(accept_lens[b]) if accept_lens is not None else int(rng.integers(0, depth.max() + 1))
        want = min(want, int(depth.max()))
        ends = np.flatnonzero(depth == want)
        end = int(ends[rng.integers(len(ends))])
        path = [end]
        while par[path[-1]] >= 0:
            path.append(int(par[path[-1]]))
        path = path[::-1]
        on_path_child = {path[t]: path[t + 1] for t in range(len(path) - 1)}
        tok[o] = int(rng.integers(vocab))      # root: the last committed token
        for i in range(len(par)):
            row = x[o + i]
            rowmax = row.max()
            kids = ch[i]
            # ids that do not attain the row maximum, distinct per parent
            chosen = []
            while len(chosen) < len(kids) + 1:
                t = int(rng.integers(vocab))
                if row[t] < rowmax and t not in chosen:
                    chosen.append(t)
            for c, t in zip(kids, chosen):
                tok[o + c] = t
            if i in on_path_child:
                row[tok[o + on_path_child[i]]] = rowmax + np.float32(4.0)
            elif i == end:
                row[chosen[-1]] = rowmax + np.float32(4.0)
                planted_bonus[b] = chosen[-1]
        planted_len[b] = want
        planted_path.append(path)
    if dtype == "bf16":
        logits = f32_to_bf16_bits(x)
    else:
        logits = x
    md = tree_max_depth if max_depth is None else max_depth
    return VerifyCase(logits, tok, node_offsets, parent, md, planted_len, planted_path,
                      planted_bonus)


def draw_accept_lens(rng, batch, max_len):
    """Accepted-length draw: position k is accepted with probability alpha_k given k-1 was."""
    out = np.zeros(batch, np.int32)
    for b in range(batch):
        a = 0
        while a < max_len and rng.random() < CHAIN_ACCEPT[min(a, len(CHAIN_ACCEPT) - 1)]:
            a += 1
        out[b] = a
    return out


# ---- expansion inputs ---------------------------------------------------------------------------

@dataclass
class ExpandCase:
    scores: np.ndarray        # [R, V] float32
    block_k: int
    bucket: np.ndarray        # [R] uint8
    bmap: np.ndarray          # [4] int32
    start_parent: np.ndarray  # [R/K] int32
    node_budget: int
    tree: Optional[dict]      # existing nodes (tok,parent,depth,node_row,node_rank) or None


def make_expand_case(rng, *, n_starts, block_k, vocab, bmap, node_budget, existing_parent=None,
                     start_parent=None, std=2.0, tie_rows=0) -> ExpandCase:
    """Drafter scores ~ N(0, std^2) fp32, buckets drawn with the Table-3 frequencies.
    `tie_rows` rows get their values quantised coarsely so that equal scores are common."""
    R = n_starts * block_k
    scores = rng.standard_normal((R, vocab), dtype=np.float32) * np.float32(std)
    for r in range(min(tie_rows, R)):
        scores[r] = np.round(scores[r] * 2.0) / 2.0
    bucket = rng.choice(4, size=R, p=np.asarray(BUCKET_FREQ) / sum(BUCKET_FREQ)).astype(np.uint8)
    tree = None
    n0 = 0
    if existing_parent is not None:
        n0 = len(existing_parent)
        tree = dict(tok=rng.integers(0, vocab, n0).astype(np.int32),
                    parent=np.asarray(existing_parent, np.int32),
                    depth=tree_depths(existing_parent),
                    node_row=np.full(n0, -1, np.int32), node_rank=np.full(n0, -1, np.int32))
    if start_parent is None:
        start_parent = (np.full(n_starts, -1, np.int32) if n0 == 0
                        else rng.integers(0, n0, n_starts).astype(np.int32))
    return ExpandCase(scores, block_k, bucket, np.asarray(bmap, np.int32),
                      np.asarray(start_parent, np.int32), node_budget, tree)


# ---- the five benchmark configurations ---------------------------------------------------------------

SEEDS = {1: 1001, 2: 2002, 3: 3003, 4: 4004, 5: 5005}


def config1_tiny(seed=SEEDS[1]):
    """1 sequence, 4 query heads on 1 KV head, D=64, prefix 128, 15-node random tree (depth<=4),
    fp32 logits over vocab 1000 with one planted path."""
    rng = rng_for(seed)
    par = random_tree(rng, 15, 4)
    attn = make_attn_case(rng, parents=[par], prefix_lens=[128], n_q_heads=4, n_kv_heads=1,
                          head_dim=64)
    ver = make_verify_case(rng, parents=[par], vocab=1000, dtype="f32", std=2.0)
    return attn, ver


def config2_tree(seed=SEEDS[2]):
    return block_tree(rng_for(seed), 60, 4, 2)


def config2_verify_layer(seed=SEEDS[2], layer=0, prefix=2048, par=None):
    """One layer of the 8B-shaped verify step: 32/8 heads, D=128, contiguous prefix 2048,
    60-node K=4/M=2 block tree."""
    par = config2_tree(seed) if par is None else par
    rng = rng_for(seed * 1000 + 17 + layer)
    return make_attn_case(rng, parents=[par], prefix_lens=[prefix], n_q_heads=32, n_kv_heads=8,
                          head_dim=128)


def config2_logits(seed=SEEDS[2], accept_len=3, vocab=128256, par=None):
    par = config2_tree(seed) if par is None else par
    rng = rng_for(seed * 1000 + 5)
    return make_verify_case(rng, parents=[par], vocab=vocab, dtype="bf16", std=2.0,
                            accept_lens=[accept_len], max_depth=8)


def config3_drafter(seed=SEEDS[3], prefix=4096, vocab=128256, variant=0):
    """Drafter block expansion: 12 cached + 32 query nodes over prefix 4096; fp32 scores
    [32, vocab] with Table-3 buckets and the map [1,2,3,4]."""
    rng = rng_for(seed + 7919 * variant)
    par, n_cached = drafter_block_tree(4)
    attn = make_attn_case(rng, parents=[par], prefix_lens=[prefix], n_q_heads=32, n_kv_heads=8,
                          head_dim=128, q_node_begin=[n_cached])
    exp = make_expand_case(rng, n_starts=8, block_k=4, vocab=vocab, bmap=[1, 2, 3, 4],
                           node_budget=128, existing_parent=par[:n_cached],
                           start_parent=np.arange(4, n_cached, dtype=np.int32), tie_rows=4)
    return attn, exp


def config4_batched(seed=SEEDS[4], batch=16, p_lo=512, p_hi=8192, n_lo=32, n_hi=96,
                    vocab=128256, with_logits=True):
    """Batched serving verify: paged KV (page 64, shuffled table), ragged prefixes and trees."""
    rng = rng_for(seed)
    prefix = rng.integers(p_lo, p_hi + 1, batch)
    sizes = rng.integers(n_lo, n_hi + 1, batch)
    parents = [random_tree(rng, int(n), 10) for n in sizes]
    attn = make_attn_case(rng, parents=parents, prefix_lens=prefix, n_q_heads=32, n_kv_heads=8,
                          head_dim=128, page_size=64)
    ver = None
    if with_logits:
        lens = draw_accept_lens(rng, batch, 10)
        ver = make_verify_case(rng, parents=parents, vocab=vocab, dtype="bf16", std=2.0,
                               accept_lens=lens, max_depth=10)
    return attn, ver


def config5_long(seed=SEEDS[5], batch=4, prefix=32768, n_nodes=128, vocab=128256,
                 with_logits=True):
    """Long-context verify: 64/8 heads, D=128, paged (64), 128-node trees of depth <= 12."""
    rng = rng_for(seed)
    parents = [random_tree(rng, n_nodes, 12) for _ in range(batch)]
    attn = make_attn_case(rng, parents=parents, prefix_lens=[prefix] * batch, n_q_heads=64,
                          n_kv_heads=8, head_dim=128, page_size=64)
    ver = None
    if with_logits:
        lens = draw_accept_lens(rng, batch, 12)
        ver = make_verify_case(rng, parents=parents, vocab=vocab, dtype="f32", std=2.0,
                               accept_lens=lens, max_depth=12)
    return attn, ver
