"""One SpecBlock draft-and-verify iteration's device steps, chained on a stream (Alg. 1).

`VerifyStep` owns the device buffers of one iteration of an L-layer target model and issues, in
order: ancestor masks / position ids, the drafter's top-k expansion, tree attention for every
layer, greedy acceptance, and KV compaction of every layer.  It only sequences calls of the
C-ABI library (paper_2605_07243_b200.binding); every step runs in the library's kernels.

Two ways to run it:
  run_device()     all inputs already resident in device memory;
  run_from_host()  inputs in pinned host memory: copies them in, runs, copies the results out.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding as sb
from . import device_inputs as dev


class VerifyStep:
    def __init__(self, layers: List, verify_case, expand_case=None, device="cuda", num_splits=0,
                 keep_host=False):
        """layers: one workloads.AttnCase per target layer (same tree and layout, different Q/K/V);
        verify_case: workloads.VerifyCase over the same tree; expand_case: optional
        workloads.ExpandCase (the drafter's batched block forward of this iteration)."""
        self.device = device
        self.n_layers = len(layers)
        c0 = layers[0]
        self.case0 = c0
        self.num_splits = num_splits
        self.max_depth = verify_case.max_depth
        self.planted_len = verify_case.planted_len
        L = self.n_layers
        # K/V of all layers in one allocation each: layer l starts layer_stride elements after l-1
        self.layer_stride = int(c0.k.size)
        self.host = {}
        k_all = np.stack([c.k for c in layers])
        v_all = np.stack([c.v for c in layers])
        q_all = np.stack([c.q for c in layers])
        self.k_all = dev.bf16_tensor(k_all, device)
        self.v_all = dev.bf16_tensor(v_all, device)
        self.q_all = dev.bf16_tensor(q_all, device)
        self.out_all = torch.empty_like(self.q_all)
        self.lse_all = torch.empty((L, c0.total_q, c0.n_q_heads), dtype=torch.float32, device=device)
        self.tb = dev.tree_batch(c0, device, k=self.k_all[0], v=self.v_all[0])
        self.kw = {}
        if c0.q_node_begin is not None:
            self.kw = dict(q_node_begin=dev.i32_tensor(c0.q_node_begin, device),
                           q_offsets=dev.i32_tensor(c0.q_offsets, device))
        self.scale = float(c0.scale)
        ws = sb.sb_tree_attention_workspace_bytes(self.tb, c0.total_q, num_splits)
        self.attn_ws = torch.empty(max(ws, 256), dtype=torch.uint8, device=device)
        B = c0.batch
        i32 = dict(dtype=torch.int32, device=device)
        self.attn_status = torch.empty(B, **i32)
        self.anc = torch.empty((self.tb.total_nodes, 4), **i32)
        self.depth = torch.empty(self.tb.total_nodes, **i32)
        self.anc_status = torch.empty(B, **i32)
        # verification inputs
        if verify_case.logits.dtype == np.uint16:
            self.logits = dev.bf16_tensor(verify_case.logits, device)
        else:
            self.logits = torch.from_numpy(verify_case.logits).to(device)
        self.tok = dev.i32_tensor(verify_case.tok, device)
        total = self.tb.total_nodes
        md = self.max_depth
        self.accept = dict(amax=torch.empty(total, **i32), accept_len=torch.empty(B, **i32),
                           path_nodes=torch.empty((B, md + 1), **i32),
                           out_tokens=torch.empty((B, md + 1), **i32), bonus=torch.empty(B, **i32),
                           status=torch.empty(B, **i32))
        vws = sb.sb_verify_accept_workspace_bytes(total, self.logits.shape[1])
        self.accept_ws = torch.empty(max(vws, 256), dtype=torch.uint8, device=device)
        self.new_len = torch.empty(B, **i32)
        self.compact_status = torch.empty(B, **i32)
        # expansion inputs
        self.expand = None
        if expand_case is not None:
            e = expand_case
            budget = e.node_budget
            n0 = 0 if e.tree is None else len(e.tree["tok"])
            tree0 = {k: torch.full((budget,), -1, **i32) for k in ("tok", "parent", "depth", "node_row", "node_rank")}
            if e.tree is not None:
                for k in tree0:
                    tree0[k][:n0] = dev.i32_tensor(e.tree[k], device)
            R, V = e.scores.shape
            ews = sb.sb_tree_expand_workspace_bytes(R, V)
            self.expand = dict(
                scores=torch.from_numpy(e.scores).to(device), bucket=torch.from_numpy(e.bucket).to(device),
                bmap=[int(x) for x in e.bmap], start_parent=dev.i32_tensor(e.start_parent, device),
                budget=budget, block_k=e.block_k, n0=n0, tree0=tree0,
                tree={k: t.clone() for k, t in tree0.items()},
                n_nodes=torch.tensor([n0], **i32), n_nodes0=torch.tensor([n0], **i32),
                topk_tok=torch.empty((R, sb.SB_KMAX), **i32),
                topk_val=torch.empty((R, sb.SB_KMAX), dtype=torch.float32, device=device),
                status=torch.empty(1, **i32), ws=torch.empty(max(ews, 256), dtype=torch.uint8, device=device))
        if keep_host:
            self._make_host_copies(k_all, v_all, q_all, verify_case, expand_case)

    # ---- pieces ----------------------------------------------------------------------------

    def run_ancestors(self):
        sb.sb_tree_ancestors(self.tb.node_offsets, self.tb.parent, self.tb.max_nodes, self.anc, self.depth,
                             self.anc_status)

    def run_expand(self):
        e = self.expand
        if e is None:
            return
        e["n_nodes"].copy_(e["n_nodes0"])      # the tree arrays restart from the existing nodes
        tree = dict(e["tree"], n_nodes=e["n_nodes"])
        sb.sb_tree_expand(e["scores"], e["block_k"], e["bucket"], e["bmap"], e["start_parent"], e["budget"],
                          tree, workspace=e["ws"], topk_tok=e["topk_tok"], topk_val=e["topk_val"],
                          status=e["status"])

    COLD_SETS = 17   # copies of the 15-16 MB score / logit matrices walked by the *_cold runs: > 2 x L2 in total

    def run_expand_cold(self):
        """sb_tree_expand once per copy of the score matrix (COLD_SETS copies, more than twice the L2 size
        together), each call on its own tree arrays: every call streams its scores from HBM, as it does in
        a real iteration where the scores were just produced by another kernel's pass over other data."""
        e = self.expand
        if e is None:
            return
        if "cold" not in e:
            e["cold"] = [dict(scores=e["scores"].clone(), tree={k: t.clone() for k, t in e["tree0"].items()})
                         for _ in range(self.COLD_SETS)]
            e["cold_n_nodes"] = torch.full((self.COLD_SETS,), e["n0"], dtype=torch.int32, device=self.device)
            e["cold_n_nodes0"] = e["cold_n_nodes"].clone()
        e["cold_n_nodes"].copy_(e["cold_n_nodes0"])      # one reset for the whole walk
        for i, c in enumerate(e["cold"]):
            tree = dict(c["tree"], n_nodes=e["cold_n_nodes"][i:i + 1])
            sb.sb_tree_expand(c["scores"], e["block_k"], e["bucket"], e["bmap"], e["start_parent"], e["budget"],
                              tree, workspace=e["ws"], topk_tok=e["topk_tok"], topk_val=e["topk_val"],
                              status=e["status"])

    def run_accept_cold(self):
        """sb_verify_accept once per copy of the logits (COLD_SETS copies, more than twice the L2 size)."""
        if not hasattr(self, "logits_cold"):
            self.logits_cold = [self.logits.clone() for _ in range(self.COLD_SETS)]
        for lg in self.logits_cold:
            sb.sb_verify_accept(lg, self.tb.node_offsets, self.tb.parent, self.tok, self.max_depth,
                                workspace=self.accept_ws, out=self.accept)

    def run_rank_features(self):
        """psi(p) of every drafter row (not part of run_device(): a 'next' row, timed on its own)."""
        e = self.expand
        if e is None:
            return None
        if "features" not in e:
            R, V = e["scores"].shape
            e["features"] = torch.empty((R, 15), dtype=torch.float32, device=self.device)
            e["features_ws"] = torch.empty(max(256, sb.sb_rank_features_workspace_bytes(R, V)), dtype=torch.uint8,
                                           device=self.device)
        return sb.sb_rank_features(e["scores"], features=e["features"], workspace=e["features_ws"])

    def run_expand_features(self):
        """The expansion and psi(p) of the same scores from ONE pass over them (sb_tree_expand_features); not part
        of run_device(), timed on its own beside run_expand() and run_rank_features()."""
        e = self.expand
        if e is None:
            return None
        self.run_rank_features() if "features" not in e else None
        e["n_nodes"].copy_(e["n_nodes0"])
        tree = dict(e["tree"], n_nodes=e["n_nodes"])
        sb.sb_tree_expand(e["scores"], e["block_k"], e["bucket"], e["bmap"], e["start_parent"], e["budget"], tree,
                          workspace=e["features_ws"], topk_tok=e["topk_tok"], topk_val=e["topk_val"], status=e["status"],
                          features=e["features"])

    def run_signal(self):
        """One iteration's term of the verifier-derived update signal, chained after run_accept() (not
        part of run_device(): a 'next' row, timed on its own).  The benchmark's tree and drafter rows
        are separate synthetic pieces, so node i is mapped to drafter row i mod R."""
        e = self.expand
        if e is None:
            return None
        if "signal" not in e:
            R = e["scores"].shape[0]
            n = int(self.tb.total_nodes)
            e["child_row"] = (torch.arange(n, dtype=torch.int32, device=self.device) % R).contiguous()
            e["signal"] = torch.zeros(self.tb.prefix_len.numel(), dtype=torch.float32, device=self.device)
            e["r_prob"] = torch.empty(self.tb.prefix_len.numel(), dtype=torch.float32, device=self.device)
            e["signal_status"] = torch.empty(self.tb.prefix_len.numel(), dtype=torch.int32, device=self.device)
        return sb.sb_verifier_signal(e["scores"], self.tb.node_offsets, e["child_row"], self.accept["path_nodes"],
                                     self.accept["accept_len"], self.accept["bonus"], self.max_depth, e["signal"],
                                     r_prob=e["r_prob"], status=e["signal_status"])

    def run_sample(self, temperature=1.0):
        """Stochastic (temperature > 0) verification of the same tree and logits (not part of run_device():
        a 'next' row, timed on its own); drafter rows are mapped as in run_signal(), the uniforms are fixed."""
        e = self.expand
        if e is None:
            return None
        if "sample_out" not in e:
            self.run_signal()
            n, B = int(self.tb.total_nodes), self.tb.prefix_len.numel()
            gen = torch.Generator(device="cpu").manual_seed(1234)
            e["u_accept"] = torch.rand(n, generator=gen).to(self.device)
            e["u_bonus"] = torch.rand(B, generator=gen).to(self.device)
            V = self.logits.shape[1]
            e["sample_ws"] = torch.empty(max(256, sb.sb_verify_sample_workspace_bytes(B, V, n, e["scores"].shape[0])),
                                         dtype=torch.uint8,
                                         device=self.device)
            i32 = dict(dtype=torch.int32, device=self.device)
            e["sample_out"] = dict(accept_len=torch.empty(B, **i32),
                                   path_nodes=torch.empty((B, self.max_depth + 1), **i32),
                                   out_tokens=torch.empty((B, self.max_depth + 1), **i32),
                                   bonus=torch.empty(B, **i32), status=torch.empty(B, **i32))
        return sb.sb_verify_sample(self.logits, e["scores"], self.tb.node_offsets, self.tb.parent, self.tok,
                                   e["child_row"], temperature, e["u_accept"], e["u_bonus"], self.max_depth,
                                   workspace=e["sample_ws"], out=e["sample_out"])

    SHIFT_SETS = 4   # weight matrices rotated per run_shift_all(): 4 x 64 MB > L2

    def run_shift_all(self, d=4096, block_k=4):
        """The drafter's layer-wise shift projection on the expansion's rows (not part of run_device():
        a 'next' row, timed on its own), once per weight matrix of a rotating set so that the weights
        come from HBM every time."""
        e = self.expand
        if e is None:
            return None
        if "shift_w" not in e:
            R = e["scores"].shape[0]
            gen = torch.Generator(device="cpu").manual_seed(4321)
            e["shift_h"] = torch.randn(R, d, generator=gen).to(torch.bfloat16).to(self.device)
            e["shift_w"] = [(torch.randn(d, 2 * d, generator=gen) * 0.02).to(torch.bfloat16).to(self.device)
                            for _ in range(self.SHIFT_SETS)]
            e["shift_out"] = torch.empty(R, d, dtype=torch.bfloat16, device=self.device)
            e["shift_ws"] = torch.zeros(sb.sb_shift_project_workspace_bytes(R, d, d, block_k), dtype=torch.uint8,
                                        device=self.device)
            e["shift_status"] = torch.zeros(1, dtype=torch.int32, device=self.device)
        for w in e["shift_w"]:
            sb.sb_shift_project(e["shift_h"], w, block_k, out=e["shift_out"], workspace=e["shift_ws"],
                                status=e["shift_status"])
        return e["shift_out"]

    FUSE_SETS = 3    # W_fuse matrices rotated per run_fuse_all(): 3 x 96 MB (64 MB of each streamed) > L2

    def run_fuse_all(self, d=4096, n_starts=8, block_k=4):
        """The drafter's fused per-position input (W_fuse over the normalised context, embedding and
        position query) for a block forward of n_starts starts, with the query term cached as in steady
        state; timed on its own like run_shift_all(), once per weight matrix of a rotating set."""
        e = self.expand
        if e is None:
            return None
        if "fuse_w" not in e:
            gen = torch.Generator(device="cpu").manual_seed(8765)
            bf = lambda *shape, std=1.0: (torch.randn(*shape, generator=gen) * std).to(torch.bfloat16).to(self.device)
            e["fuse_c"], e["fuse_e"], e["fuse_q"] = bf(n_starts, d, std=3.0), bf(n_starts, d, std=0.05), bf(block_k, d)
            e["fuse_w"] = [bf(d, 3 * d, std=0.02) for _ in range(self.FUSE_SETS)]
            e["fuse_gain"] = [(torch.rand(d, generator=gen) + 0.5).to(self.device) for _ in range(3)]
            e["fuse_out"] = torch.empty(n_starts * block_k, d, dtype=torch.bfloat16, device=self.device)
            e["fuse_ws"] = torch.zeros(sb.sb_fuse_project_workspace_bytes(n_starts, block_k, d, d, False),
                                       dtype=torch.uint8, device=self.device)
            e["fuse_status"] = torch.zeros(1, dtype=torch.int32, device=self.device)
            e["fuse_q_term"] = []
            for w in e["fuse_w"]:        # the first call with a weight matrix leaves its query term behind
                qt = torch.empty(block_k, d, dtype=torch.float32, device=self.device)
                self._fuse_call(w, qt, False)
                e["fuse_q_term"].append(qt)
        for w, qt in zip(e["fuse_w"], e["fuse_q_term"]):
            self._fuse_call(w, qt, True)
        return e["fuse_out"]

    def _fuse_call(self, w, q_term, valid):
        e = self.expand
        g = e["fuse_gain"]
        sb.sb_fuse_project(e["fuse_c"], e["fuse_e"], e["fuse_q"], w, gain_c=g[0], gain_e=g[1], gain_q=g[2], eps=1e-5,
                           q_term=q_term, q_term_valid=valid, out=e["fuse_out"], workspace=e["fuse_ws"],
                           status=e["fuse_status"])

    def run_attention(self, layers=None):
        first = True
        for l in range(self.n_layers) if layers is None else layers:
            # from the second layer on the kernel just before is the previous layer's attention, which
            # writes neither the index arrays nor the cache: lengths and prefix keys may be read under its tail
            sb.sb_tree_attention(self.tb, self.q_all[l], self.out_all[l], self.lse_all[l], scale=self.scale,
                                 num_splits=self.num_splits, workspace=self.attn_ws, status=self.attn_status,
                                 k_cache=self.k_all[l], v_cache=self.v_all[l], index_arrays_settled=not first,
                                 prefix_rows_settled=not first,
                                 **self.kw)
            first = False

    def run_accept(self):
        sb.sb_verify_accept(self.logits, self.tb.node_offsets, self.tb.parent, self.tok, self.max_depth,
                            workspace=self.accept_ws, out=self.accept)

    def run_compact(self):
        sb.sb_kv_compact(self.tb, self.n_layers, self.layer_stride, self.accept["path_nodes"],
                         self.accept["accept_len"], self.max_depth, self.new_len, self.compact_status)

    # ---- whole step --------------------------------------------------------------------------

    def run_device(self):
        """The whole iteration with inputs resident in device memory (enqueue only)."""
        self.run_ancestors()
        self.run_expand()
        self.run_attention()
        self.run_accept()
        self.run_compact()

    def launches_per_step(self) -> int:
        before = sb.sb_kernel_launch_count()
        self.run_device()
        return sb.sb_kernel_launch_count() - before

    def _make_host_copies(self, k_all, v_all, q_all, verify_case, expand_case):
        def pin(t):
            return t.cpu().pin_memory()
        h = self.host
        h["k"], h["v"], h["q"] = pin(self.k_all), pin(self.v_all), pin(self.q_all)
        h["parent"], h["node_offsets"] = pin(self.tb.parent), pin(self.tb.node_offsets)
        h["prefix_len"], h["logits"], h["tok"] = pin(self.tb.prefix_len), pin(self.logits), pin(self.tok)
        if self.tb.page_table is not None:
            h["page_table"] = pin(self.tb.page_table)
        if self.expand is not None:
            h["scores"], h["bucket"] = pin(self.expand["scores"]), pin(self.expand["bucket"])
            h["start_parent"] = pin(self.expand["start_parent"])
        h["out"] = torch.empty(self.out_all.shape, dtype=self.out_all.dtype).pin_memory()
        h["lse"] = torch.empty(self.lse_all.shape, dtype=torch.float32).pin_memory()
        h["res"] = {k: torch.empty(t.shape, dtype=t.dtype).pin_memory() for k, t in self.accept.items()}
        h["new_len"] = torch.empty(self.new_len.shape, dtype=torch.int32).pin_memory()

    def host_bytes(self):
        """(host->device, device->host) bytes of one run_from_host()."""
        h = self.host
        h2d = sum(h[k].numel() * h[k].element_size() for k in
                  ("k", "v", "q", "parent", "node_offsets", "prefix_len", "logits", "tok", "page_table",
                   "scores", "bucket", "start_parent") if k in h)
        d2h = sum(t.numel() * t.element_size() for t in [h["out"], h["lse"], h["new_len"]] +
                  list(h["res"].values()))
        return h2d, d2h

    def run_from_host(self):
        """Inputs in pinned host memory -> device, the whole iteration, results -> pinned host
        memory.  Enqueue only; synchronise the current stream before reading the host results.

        The copies are pipelined with the kernels: a copy stream brings layer l's K, V and Q while
        layer l-1 is being attended to, a second one returns each layer's output while later layers
        are still arriving (the link is full duplex).  Both streams fork from the current stream
        at entry and join it at the end, so to the caller the call is ordered like any other work
        of that stream."""
        h = self.host
        main = torch.cuda.current_stream()
        L = self.n_layers
        if not hasattr(self, "_h2d"):
            self._h2d, self._d2h = torch.cuda.Stream(), torch.cuda.Stream()
            self._ev = {k: torch.cuda.Event() for k in ("fork", "small", "logits", "d2h_end")}
            self._ev_in = [torch.cuda.Event() for _ in range(L)]
            self._ev_done = [torch.cuda.Event() for _ in range(L)]
        ev = self._ev
        ev["fork"].record(main)
        self._h2d.wait_event(ev["fork"])
        self._d2h.wait_event(ev["fork"])
        with torch.cuda.stream(self._h2d):
            self.tb.parent.copy_(h["parent"], non_blocking=True)
            self.tb.node_offsets.copy_(h["node_offsets"], non_blocking=True)
            self.tb.prefix_len.copy_(h["prefix_len"], non_blocking=True)
            self.tok.copy_(h["tok"], non_blocking=True)
            if "page_table" in h:
                self.tb.page_table.copy_(h["page_table"], non_blocking=True)
            if self.expand is not None:
                self.expand["scores"].copy_(h["scores"], non_blocking=True)
                self.expand["bucket"].copy_(h["bucket"], non_blocking=True)
                self.expand["start_parent"].copy_(h["start_parent"], non_blocking=True)
            ev["small"].record()
            for l in range(L):
                self.q_all[l].copy_(h["q"][l], non_blocking=True)
                self.k_all[l].copy_(h["k"][l], non_blocking=True)
                self.v_all[l].copy_(h["v"][l], non_blocking=True)
                self._ev_in[l].record()
            self.logits.copy_(h["logits"], non_blocking=True)
            ev["logits"].record()
        main.wait_event(ev["small"])
        self.run_ancestors()
        self.run_expand()
        for l in range(L):
            main.wait_event(self._ev_in[l])
            self.run_attention(layers=[l])
            self._ev_done[l].record(main)
            with torch.cuda.stream(self._d2h):
                self._d2h.wait_event(self._ev_done[l])
                h["out"][l].copy_(self.out_all[l], non_blocking=True)
                h["lse"][l].copy_(self.lse_all[l], non_blocking=True)
        with torch.cuda.stream(self._d2h):
            ev["d2h_end"].record()
        main.wait_event(ev["logits"])
        self.run_accept()
        self.run_compact()
        for k, t in self.accept.items():
            h["res"][k].copy_(t, non_blocking=True)
        h["new_len"].copy_(self.new_len, non_blocking=True)
        main.wait_event(ev["d2h_end"])

    # ---- accounting -------------------------------------------------------------------------

    def algorithmic_bytes(self):
        """Bytes each part of the step must move at minimum (every input read once, every output
        written once)."""
        c0 = self.case0
        attn_layer = c0.algorithmic_bytes()
        logits = self.logits.numel() * self.logits.element_size()
        total = self.tb.total_nodes
        accept = logits + total * 4 * 3
        row = c0.n_kv_heads * c0.head_dim * 2
        parts = dict(attention_per_layer=attn_layer, attention=attn_layer * self.n_layers, accept=accept,
                     ancestors=total * 4 * 6)
        if self.expand is not None:
            s = self.expand["scores"]
            parts["expand"] = s.numel() * 4 + s.shape[0] * sb.SB_KMAX * 8
        # accepted path rows (the root stays in place) read + written, K and V, every layer
        moved = int(np.sum(self.planted_len)) if self.planted_len is not None else 0
        parts["compact"] = moved * row * 2 * 2 * self.n_layers
        parts["total"] = sum(v for k, v in parts.items() if k != "attention_per_layer")
        return parts
