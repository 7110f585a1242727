"""One whole verifier iteration of SpecBlock (Algorithm 1) as a chain of library calls on one stream.

`SpecBlockIteration` grows the draft tree ON THE DEVICE with M block expansions, verifies it with
tree attention over every target layer, commits the longest accepted path and compacts the target's
KV cache -- no host round trip anywhere: the tree arrays that `sb_tree_expand` appends to are the
very arrays `sb_tree_ancestors`, `sb_tree_attention`, `sb_verify_accept` and `sb_kv_compact` read,
and the device scalar holding the node count is the second entry of the `node_offsets` array the
verify calls take.  The whole chain can be captured in one CUDA graph.

Per drafter block m (Algorithm 1, the loop over m):
    [W_cond]      block 1 only: the target's concatenated multi-layer features -> c   (sb_shift_project, plain)
    W_fuse        per-position inputs from c, the embedding and the position queries  (sb_fuse_project)
    L_d layers    tree attention over the drafter's cache, then the layer-wise shift  (sb_tree_attention,
                  sb_shift_project)
    psi(p)        the rank head's distribution summary of every row   } one pass over  (sb_tree_expand_features)
    attach        top-b tokens of every row under the block's starts  } the scores
then  verify:     ancestor masks, tree attention of every target layer, greedy acceptance, the verifier-derived
                  signal of the iteration, compaction.

The pieces that need trained weights are not in the library (the decoder layers' own projections
and MLPs, the lm_head, the rank head, the choice of next-block starts): their outputs are inputs
here (`scores`, `bucket`, `start_parent`, the Q/K/V of each attention call, the hidden states
entering each shift), so every call runs on given data and can be checked on its own.  What flows
from call to call on the device is the tree and everything derived from it.

This module only sequences calls of paper_2605_07243_b200.binding; all arithmetic is in the library.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import binding as sb
from . import device_inputs as dev


@dataclass
class DraftBlock:
    """Inputs of one drafter block forward over S starts (R = S * K rows, row = start * K + position)."""
    scores: np.ndarray                      # fp32 [R, V]: the draft distributions' logits
    bucket: np.ndarray                      # uint8 [R]: the rank head's bucket per row
    start_parent: np.ndarray                # int32 [S]: the tree node each start continues from
    cond: Optional[np.ndarray] = None       # bf16 bits: block 1 [1, 3 d_t] target features; later [S, d] cached states
    embed: Optional[np.ndarray] = None      # bf16 bits [S, d]: embeddings of the starts' tokens
    attn: Optional[List] = None             # one workloads.AttnCase per drafter layer (the rows as query nodes)
    hidden: Optional[List[np.ndarray]] = None   # bf16 bits [R, d] per drafter layer: the state entering the shift


@dataclass
class DrafterWeights:
    """bf16 bit patterns; gains fp32 or None."""
    w_cond: np.ndarray                      # [d, 3 d_t]
    w_fuse: np.ndarray                      # [d, 3 d]
    queries: np.ndarray                     # [K, d] learnable position queries
    w_shift: List[np.ndarray]               # per layer [d, 2 d]
    gains: tuple = (None, None, None)
    eps: float = 1e-5


def _bf16(x, device):
    """bf16 bit patterns (numpy uint16) or a bf16 torch tensor -> bf16 tensor on the device."""
    if isinstance(x, torch.Tensor):
        assert x.dtype == torch.bfloat16
        return x.to(device).contiguous()
    return dev.bf16_tensor(x, device)


class SpecBlockIteration:
    def __init__(self, *, block_k: int, bmap, node_budget: int, root_tok: int, blocks: List[DraftBlock],
                 target_layers: List, logits: np.ndarray, max_depth: int, weights: Optional[DrafterWeights] = None,
                 device="cuda", num_splits=0, temperature: float = 0.0, u_accept=None, u_bonus=None,
                 drafter_cache: Optional[List] = None):
        """target_layers: one workloads.AttnCase per target layer over ONE sequence whose tree has
        `node_budget` nodes (their K/V rows and Q rows are used; the tree itself is built here);
        logits: [node_budget, V] fp32 or bf16 bits (the target's scores per tree node).
        temperature > 0: the tree is verified by rejection sampling (sb_verify_sample) with the given uniforms
        (u_accept fp32 [node_budget], u_bonus fp32 [1]) instead of greedy acceptance.
        drafter_cache: one workloads.AttnCase per drafter layer (contiguous, one sequence) whose K/V hold,
        behind a prefix that ends with the last committed position, one row per block position of this
        iteration in the order of the blocks' score rows (a "tree" of 1 + total rows nodes, prefix_len = the
        drafter's committed length - 1).  A committed position keeps the keys and values of its own draft
        forward (App. A.2): the accepted path is translated to rows (sb_path_rows, through node_row) and
        committed by a second sb_kv_compact."""
        self.device, self.block_k, self.budget, self.max_depth = device, block_k, node_budget, max_depth
        self.bmap = [int(x) for x in bmap]
        self.num_splits = num_splits
        i32 = dict(dtype=torch.int32, device=device)
        # ---- the tree, grown on the device --------------------------------------------------------------
        self.node_offsets = torch.zeros(2, **i32)            # [0, n_nodes]
        self.tree = {k: torch.empty(node_budget, **i32) for k in ("tok", "parent", "depth", "node_row", "node_rank")}
        self.tree["n_nodes"] = self.node_offsets[1:]          # the same word: expand's counter IS node_offsets[1]
        root = dict(tok=root_tok, parent=-1, depth=0, node_row=-1, node_rank=-1)
        self._tree0 = {k: torch.full((node_budget,), -1, **i32) for k in root}
        for k, v in root.items():
            self._tree0[k][0] = v
        self._offsets0 = torch.tensor([0, 1], **i32)
        # ---- drafter blocks --------------------------------------------------------------------------------
        self.weights = None
        if weights is not None:
            w = weights
            self.weights = dict(w_cond=_bf16(w.w_cond, device), w_fuse=_bf16(w.w_fuse, device),
                                queries=_bf16(w.queries, device), w_shift=[_bf16(x, device) for x in w.w_shift],
                                gains=[None if g is None else torch.as_tensor(np.asarray(g, np.float32)).to(device)
                                       for g in w.gains], eps=float(w.eps))
            d = w.w_fuse.shape[0]
            self.q_term = torch.empty((block_k, d), dtype=torch.float32, device=device)
            self.q_term_valid = False
        # the blocks' scores lie one after the other in ONE matrix: a node's draft distribution is then a row of it
        self.scores_all = torch.from_numpy(np.ascontiguousarray(np.concatenate([b.scores for b in blocks]), np.float32)).to(device)
        self.child_row = torch.empty(node_budget, **i32)      # per node: the row that proposed its children (-1: none)
        self._child_row0 = torch.full((node_budget,), -1, **i32)
        self.signal = torch.zeros(1, dtype=torch.float32, device=device)   # verifier-derived signal, summed over iterations
        self.r_prob = torch.empty(1, dtype=torch.float32, device=device)
        self.signal_status = torch.empty(1, **i32)
        self.blocks = []
        row_base = 0
        for m, b in enumerate(blocks):
            R, V = b.scores.shape
            S = R // block_k
            e = dict(scores=self.scores_all[row_base:row_base + R], row_base=row_base,
                     bucket=torch.from_numpy(np.ascontiguousarray(b.bucket, np.uint8)).to(device),
                     start_parent=dev.i32_tensor(b.start_parent, device), R=R, S=S,
                     topk_tok=torch.empty((R, sb.SB_KMAX), **i32),
                     topk_val=torch.empty((R, sb.SB_KMAX), dtype=torch.float32, device=device),
                     status=torch.empty(1, **i32),
                     ws=torch.empty(max(256, sb.sb_tree_expand_workspace_bytes(R, V)), dtype=torch.uint8, device=device),
                     features=torch.empty((R, 15), dtype=torch.float32, device=device),
                     features_ws=torch.empty(max(256, sb.sb_rank_features_workspace_bytes(R, V)), dtype=torch.uint8,
                                             device=device))
            if self.weights is not None and b.cond is not None:
                d = self.weights["w_fuse"].shape[0]
                e["embed"] = _bf16(b.embed, device)
                e["cond_in"] = _bf16(b.cond, device)
                bf = dict(dtype=torch.bfloat16, device=device)
                e["h0"] = torch.empty((R, d), **bf)
                e["dense_status"] = torch.zeros(1, **i32)
                if m == 0:     # the first block's condition comes from the target's features through W_cond
                    e["c"] = torch.empty((S, d), **bf)
                    e["cond_ws"] = torch.zeros(sb.sb_shift_project_workspace_bytes(S, b.cond.shape[1], d, 0),
                                               dtype=torch.uint8, device=device)
                else:          # later blocks continue from the drafter's own cached states
                    e["c"] = e["cond_in"]
                e["fuse_ws"] = torch.zeros(sb.sb_fuse_project_workspace_bytes(S, block_k, d, d, False),
                                           dtype=torch.uint8, device=device)
            if b.attn is not None:
                e["attn"] = []
                for case in b.attn:
                    tb, q, kw = dev.attention_args(case, device)
                    e["attn"].append(dict(tb=tb, q=q, kw=kw, out=torch.empty_like(q),
                                          lse=torch.empty((q.shape[0], tb.n_q_heads), dtype=torch.float32, device=device),
                                          status=torch.empty(tb.prefix_len.numel(), **i32),
                                          ws=torch.empty(max(256, sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], 0)),
                                                         dtype=torch.uint8, device=device)))
            if self.weights is not None and b.hidden is not None:
                d = self.weights["w_fuse"].shape[0]
                e["hidden"] = [_bf16(h, device) for h in b.hidden]
                e["shifted"] = [torch.empty((R, d), dtype=torch.bfloat16, device=device) for _ in b.hidden]
                e["shift_ws"] = torch.zeros(sb.sb_shift_project_workspace_bytes(R, d, d, block_k), dtype=torch.uint8,
                                            device=device)
                e["shift_status"] = torch.zeros(1, **i32)
            self.blocks.append(e)
            row_base += R
        # ---- the target's verify forward ------------------------------------------------------------------
        c0 = target_layers[0]
        assert c0.batch == 1 and int(c0.node_offsets[-1]) == node_budget and c0.q_node_begin is None
        self.n_layers = len(target_layers)
        self.layer_stride = int(c0.k.size)
        self.k_all = dev.bf16_tensor(np.stack([c.k for c in target_layers]), device)
        self.v_all = dev.bf16_tensor(np.stack([c.v for c in target_layers]), device)
        self.q_all = dev.bf16_tensor(np.stack([c.q for c in target_layers]), device)
        self.out_all = torch.empty_like(self.q_all)
        self.lse_all = torch.empty((self.n_layers, node_budget, c0.n_q_heads), dtype=torch.float32, device=device)
        self.tb = sb.TreeBatch(
            n_q_heads=c0.n_q_heads, n_kv_heads=c0.n_kv_heads, head_dim=c0.head_dim, k_cache=self.k_all[0],
            v_cache=self.v_all[0], prefix_len=dev.i32_tensor(c0.prefix_len, device), node_offsets=self.node_offsets,
            parent=self.tree["parent"], total_nodes=node_budget, max_nodes=node_budget, max_kv_len=c0.max_kv_len,
            page_size=c0.page_size, kv_capacity=c0.kv_capacity,
            page_table=None if c0.page_table is None else dev.i32_tensor(c0.page_table, device),
            num_pages=c0.num_pages, max_pages=c0.max_pages)
        self.scale = float(c0.scale)
        self.attn_ws = torch.empty(max(256, sb.sb_tree_attention_workspace_bytes(self.tb, node_budget, num_splits)),
                                   dtype=torch.uint8, device=device)
        self.attn_status = torch.empty(1, **i32)
        self.anc = torch.empty((node_budget, 4), **i32)
        self.depth = torch.empty(node_budget, **i32)
        self.anc_status = torch.empty(1, **i32)
        self.logits = dev.bf16_tensor(logits, device) if logits.dtype == np.uint16 else torch.from_numpy(logits).to(device)
        md = max_depth
        self.accept = dict(amax=torch.empty(node_budget, **i32), accept_len=torch.empty(1, **i32),
                           path_nodes=torch.empty((1, md + 1), **i32), out_tokens=torch.empty((1, md + 1), **i32),
                           bonus=torch.empty(1, **i32), status=torch.empty(1, **i32))
        self.accept_ws = torch.empty(max(256, sb.sb_verify_accept_workspace_bytes(node_budget, self.logits.shape[1])),
                                     dtype=torch.uint8, device=device)
        self.new_len = torch.empty(1, **i32)
        self.compact_status = torch.empty(1, **i32)
        # ---- the drafter's cache of the same tree (optional) -------------------------------------------------
        self.drafter_tb = None
        if drafter_cache:
            d0 = drafter_cache[0]
            n_rows_all = int(self.scores_all.shape[0])
            assert d0.batch == 1 and d0.page_size == 0 and int(d0.node_offsets[-1]) == 1 + n_rows_all
            self.drafter_k = dev.bf16_tensor(np.stack([c.k for c in drafter_cache]), device)
            self.drafter_v = dev.bf16_tensor(np.stack([c.v for c in drafter_cache]), device)
            self.drafter_layers, self.drafter_stride = len(drafter_cache), int(d0.k.size)
            self.drafter_tb = sb.TreeBatch(
                n_q_heads=d0.n_q_heads, n_kv_heads=d0.n_kv_heads, head_dim=d0.head_dim, k_cache=self.drafter_k[0],
                v_cache=self.drafter_v[0], prefix_len=dev.i32_tensor(d0.prefix_len, device),
                node_offsets=dev.i32_tensor(d0.node_offsets, device), parent=dev.i32_tensor(d0.parent, device),
                total_nodes=1 + n_rows_all, max_nodes=1 + n_rows_all, max_kv_len=d0.max_kv_len, page_size=0,
                kv_capacity=d0.kv_capacity)
            self.path_rows = torch.empty((1, max_depth + 1), **i32)
            self.path_rows_status = torch.empty(1, **i32)
            self.drafter_new_len = torch.empty(1, **i32)
            self.drafter_compact_status = torch.empty(1, **i32)
        self.temperature = float(temperature)
        if self.temperature > 0.0:
            self.u_accept = torch.as_tensor(np.asarray(u_accept, np.float32)).to(device)
            self.u_bonus = torch.as_tensor(np.asarray(u_bonus, np.float32)).to(device)
            self.sample_ws = torch.empty(max(256, sb.sb_verify_sample_workspace_bytes(
                1, self.logits.shape[1], node_budget, self.scores_all.shape[0])), dtype=torch.uint8, device=device)

    # ---- the chain ---------------------------------------------------------------------------------------

    def reset_tree(self):
        """The empty draft tree rooted at the last committed token (device-to-device copies)."""
        for k, t0 in self._tree0.items():
            self.tree[k].copy_(t0)
        self.node_offsets.copy_(self._offsets0)
        self.child_row.copy_(self._child_row0)

    def run_block(self, m: int):
        e, w = self.blocks[m], self.weights
        if "h0" in e:
            if m == 0:
                sb.sb_shift_project(e["cond_in"], w["w_cond"], 0, out=e["c"], workspace=e["cond_ws"],
                                    status=e["dense_status"])
            g = w["gains"]
            sb.sb_fuse_project(e["c"], e["embed"], w["queries"], w["w_fuse"], gain_c=g[0], gain_e=g[1], gain_q=g[2],
                               eps=w["eps"], q_term=self.q_term, q_term_valid=self.q_term_valid, out=e["h0"],
                               workspace=e["fuse_ws"], status=e["dense_status"])
            self.q_term_valid = True     # the query term of these weights is on the device from now on
        n_layers = max(len(e.get("attn", [])), len(e.get("hidden", [])))
        for l in range(n_layers):
            if l < len(e.get("attn", [])):
                a = e["attn"][l]
                # the block's index arrays and its drafter cache are inputs that no kernel of the chain writes:
                # whatever was enqueued just before, lengths and prefix keys may be fetched under its tail
                sb.sb_tree_attention(a["tb"], a["q"], a["out"], a["lse"], workspace=a["ws"], status=a["status"],
                                     index_arrays_settled=True, prefix_rows_settled=True, **a["kw"])
            if l < len(e.get("hidden", [])):
                sb.sb_shift_project(e["hidden"][l], w["w_shift"][l], self.block_k, out=e["shifted"][l],
                                    workspace=e["shift_ws"], status=e["shift_status"])
        # psi(p) and the expansion read the same scores: one pass over them serves both
        sb.sb_tree_expand(e["scores"], self.block_k, e["bucket"], self.bmap, e["start_parent"], self.budget, self.tree,
                          workspace=e["features_ws"], topk_tok=e["topk_tok"], topk_val=e["topk_val"], status=e["status"],
                          features=e["features"], child_row=self.child_row, row_base=e["row_base"])

    def run_verify(self):
        sb.sb_tree_ancestors(self.node_offsets, self.tree["parent"], self.budget, self.anc, self.depth, self.anc_status)
        for l in range(self.n_layers):
            sb.sb_tree_attention(self.tb, self.q_all[l], self.out_all[l], self.lse_all[l], scale=self.scale,
                                 num_splits=self.num_splits, workspace=self.attn_ws, status=self.attn_status,
                                 k_cache=self.k_all[l], v_cache=self.v_all[l], index_arrays_settled=l > 0,
                                 prefix_rows_settled=l > 0)
        if self.temperature > 0.0:   # rejection sampling against the target: the drafter rows come through child_row
            sb.sb_verify_sample(self.logits, self.scores_all, self.node_offsets, self.tree["parent"], self.tree["tok"],
                                self.child_row, self.temperature, self.u_accept, self.u_bonus, self.max_depth,
                                workspace=self.sample_ws, out=self.accept)
        else:
            sb.sb_verify_accept(self.logits, self.node_offsets, self.tree["parent"], self.tree["tok"], self.max_depth,
                                workspace=self.accept_ws, out=self.accept)
        # the verifier-derived signal of this iteration (Algorithm 2, line 2): the drafter's probability of the
        # bonus token in the row that proposed the children of the last accepted node -- found through child_row,
        # which the expansions filled in on the device
        sb.sb_verifier_signal(self.scores_all, self.node_offsets, self.child_row, self.accept["path_nodes"],
                              self.accept["accept_len"], self.accept["bonus"], self.max_depth, self.signal,
                              r_prob=self.r_prob, status=self.signal_status)
        sb.sb_kv_compact(self.tb, self.n_layers, self.layer_stride, self.accept["path_nodes"],
                         self.accept["accept_len"], self.max_depth, self.new_len, self.compact_status)
        if self.drafter_tb is not None:   # the drafter commits the block rows that proposed the accepted nodes
            sb.sb_path_rows(self.node_offsets, self.tree["node_row"], self.accept["path_nodes"], self.accept["accept_len"],
                            self.max_depth, self.path_rows, self.path_rows_status)
            sb.sb_kv_compact(self.drafter_tb, self.drafter_layers, self.drafter_stride, self.path_rows,
                             self.accept["accept_len"], self.max_depth, self.drafter_new_len,
                             self.drafter_compact_status)

    def run(self):
        """The whole iteration (enqueue only): returns nothing, results stay on the device."""
        self.reset_tree()
        for m in range(len(self.blocks)):
            self.run_block(m)
        self.run_verify()

    def launches(self) -> int:
        before = sb.sb_kernel_launch_count()
        self.run()
        return sb.sb_kernel_launch_count() - before


def build_8b_iteration(target_layers, logits, max_depth, *, d=4096, vocab=128256, drafter_layers=2, seed=7007,
                       device="cuda", num_splits=0) -> SpecBlockIteration:
    """An iteration at the shapes of an 8B target and its drafter, for timing: K = 4, M = 2, node budget
    len(tree of target_layers), block 1 from the root (4 rows, every row two siblings, so that nodes 1..8
    exist whatever the scores are), block 2 from those 8 nodes (32 rows, buckets at the Table-3
    frequencies, map [1, 2, 3, 4]); the drafter's attention per block over a 4096-token cache; all
    weights ~ N(0, 0.02^2) in bf16, d = 4096, the target's feature width equal to d."""
    from . import workloads as W
    rng = W.rng_for(seed)
    gen = torch.Generator(device=device).manual_seed(seed)
    K, budget = 4, int(target_layers[0].node_offsets[-1])
    rb = lambda *shape, std=1.0: (torch.randn(*shape, generator=gen, device=device) * std).to(torch.bfloat16)
    freq = np.asarray(W.BUCKET_FREQ) / sum(W.BUCKET_FREQ)

    def block(n_starts, start_parent, bucket, attn, first):
        R = n_starts * K
        scores = rng.standard_normal((R, vocab), dtype=np.float32) * np.float32(2.0)
        return DraftBlock(scores, bucket, np.asarray(start_parent, np.int32),
                          cond=rb(1, 3 * d, std=2.0) if first else rb(n_starts, d), embed=rb(n_starts, d, std=0.05),
                          attn=attn, hidden=[rb(R, d) for _ in range(drafter_layers)])

    attn1 = [W.make_attn_case(rng, parents=[W.chain_tree(K)], prefix_lens=[4096], n_q_heads=32, n_kv_heads=8,
                              head_dim=128, q_node_begin=[0]) for _ in range(drafter_layers)]
    attn2 = [W.config3_drafter(variant=l, vocab=8)[0] for l in range(drafter_layers)]
    b1 = block(1, [0], np.ones(K, np.uint8), attn1, True)
    b2 = block(8, np.arange(1, 9), rng.choice(4, size=8 * K, p=freq).astype(np.uint8), attn2, False)
    weights = DrafterWeights(w_cond=rb(d, 3 * d, std=0.02), w_fuse=rb(d, 3 * d, std=0.02), queries=rb(K, d),
                             w_shift=[rb(d, 2 * d, std=0.02) for _ in range(drafter_layers)])
    # the drafter's own cache: 4096 committed positions, then one row per block position (4 + 32)
    cache = [W.make_attn_case(rng, parents=[W.chain_tree(1 + 9 * K)], prefix_lens=[4095], n_q_heads=32, n_kv_heads=8,
                              head_dim=128) for _ in range(drafter_layers)]
    return SpecBlockIteration(block_k=K, bmap=[1, 2, 3, 4], node_budget=budget, root_tok=1, blocks=[b1, b2],
                              target_layers=target_layers, logits=logits, max_depth=max_depth, weights=weights,
                              device=device, num_splits=num_splits, drafter_cache=cache)
