"""One whole SpecBlock iteration (Algorithm 1) through iteration.SpecBlockIteration: the draft tree is
grown on the device by two block expansions and consumed there by the verify forward, acceptance and
compaction.  Everything is compared with the oracle running the same chain on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import workloads as W
from paper_2605_07243_b200.iteration import DraftBlock, DrafterWeights, SpecBlockIteration

pytestmark = pytest.mark.gpu

K, BUDGET, VOCAB, P = 4, 40, 3001, 300
BMAP = [2, 3, 4, 1]
ROOT_TOK = 77


def _oracle_tree(blocks):
    tree = dict(tok=np.array([ROOT_TOK], np.int32), parent=np.array([-1], np.int32), depth=np.array([0], np.int32),
                node_row=np.array([-1], np.int32), node_rank=np.array([-1], np.int32))
    res = None
    for b in blocks:
        res = oracle.tree_expand(b.scores, K, b.bucket, BMAP, b.start_parent, BUDGET, tree=tree)
        assert res["status"] == 0
        n = res["n_nodes"]
        tree = {k: res[k][:n].copy() for k in tree}
    return res, tree


def _build(seed, n_target_layers=2, with_drafter=True):
    rng = W.rng_for(seed)
    d, d_t = 256, 128
    bf = lambda shape, std=1.0: W.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))
    freq = np.asarray(W.BUCKET_FREQ) / sum(W.BUCKET_FREQ)

    def block(n_starts, start_parent, first):
        R = n_starts * K
        scores = rng.standard_normal((R, VOCAB), dtype=np.float32) * np.float32(2.0)
        bucket = rng.choice(4, size=R, p=freq).astype(np.uint8)
        b = DraftBlock(scores, bucket, np.asarray(start_parent, np.int32))
        if with_drafter:
            b.cond = bf((1, 3 * d_t), 2.0) if first else bf((n_starts, d))
            b.embed = bf((n_starts, d), 0.05)
            # the block's rows as the query nodes of the drafter's row tree: chains of K under each start
            cached = 0 if first else K
            parents = np.concatenate([np.arange(-1, cached - 1)] +
                                     [np.concatenate([[int(rng.integers(0, cached)) if cached else -1],
                                                      cached + s * K + np.arange(0, K - 1)]) for s in range(n_starts)])
            b.attn = [W.make_attn_case(rng, parents=[parents.astype(np.int32)], prefix_lens=[200], n_q_heads=4,
                                       n_kv_heads=2, head_dim=64, q_node_begin=[cached]) for _ in range(2)]
            b.hidden = [bf((R, d)) for _ in range(2)]
        return b

    b1 = block(1, [0], True)
    # next-block starts: the end of the first block's chain and two more of its nodes (the rank head's choice
    # is an input of the iteration; any existing nodes will do)
    res1, tree1 = _oracle_tree([b1])
    n1 = res1["n_nodes"]
    chain_end = int(np.flatnonzero((tree1["node_rank"] == 0))[-1])
    others = [int(x) for x in rng.permutation(np.arange(1, n1)) if int(x) != chain_end][:2]
    b2 = block(3, [chain_end] + others, False)
    res2, tree2 = _oracle_tree([b1, b2])
    n = res2["n_nodes"]
    # target logits: a planted accepted path of the tree the oracle built
    logits = rng.standard_normal((BUDGET, VOCAB), dtype=np.float32) * np.float32(2.0)
    depth = tree2["depth"]
    end = int(np.flatnonzero(depth == min(3, depth.max()))[0])
    path = [end]
    while tree2["parent"][path[-1]] >= 0:
        path.append(int(tree2["parent"][path[-1]]))
    path = path[::-1]
    for a, c in zip(path[:-1], path[1:]):
        logits[a, tree2["tok"][c]] = logits[a].max() + np.float32(4.0)
    kids = set(int(t) for t in tree2["tok"][np.flatnonzero(tree2["parent"] == end)])
    bonus = next(t for t in range(VOCAB) if t not in kids)
    logits[end, bonus] = logits[end].max() + np.float32(4.0)
    target = [W.make_attn_case(rng, parents=[W.chain_tree(BUDGET)], prefix_lens=[P], n_q_heads=8, n_kv_heads=2,
                               head_dim=128) for _ in range(n_target_layers)]
    weights, drafter_cache = None, None
    if with_drafter:
        # the drafter's own cache: 78 committed positions (the last one is slot 0 of the row numbering), then one
        # K/V row per block position of the iteration (4 rows of block 1, 12 of block 2)
        drafter_cache = [W.make_attn_case(rng, parents=[W.chain_tree(1 + 4 * K)], prefix_lens=[77], n_q_heads=4,
                                          n_kv_heads=2, head_dim=64) for _ in range(2)]
        weights = DrafterWeights(w_cond=bf((d, 3 * d_t), 0.05), w_fuse=bf((d, 3 * d), 0.05), queries=bf((K, d)),
                                 w_shift=[bf((d, 2 * d), 0.05) for _ in range(2)],
                                 gains=tuple(rng.uniform(0.5, 1.5, d).astype(np.float32) for _ in range(3)))
    it = SpecBlockIteration(block_k=K, bmap=BMAP, node_budget=BUDGET, root_tok=ROOT_TOK, blocks=[b1, b2],
                            target_layers=target, logits=logits, max_depth=2 * K, weights=weights,
                            drafter_cache=drafter_cache)
    it.drafter_cases = drafter_cache    # kept for the check below
    return it, [b1, b2], tree2, n, logits, target, weights, (len(path) - 1, bonus)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _close(got, ref, scale=1.0):
    return (np.abs(got - ref) <= 1e-2 * scale + 1e-2 * np.abs(ref)).all()


def _check_against_oracle(it, blocks, tree2, n, logits, target, weights, planted):
    # ---- the tree grown on the device ------------------------------------------------------------------
    assert it.node_offsets.cpu().tolist() == [0, n]
    for k in ("tok", "parent", "depth", "node_rank"):
        np.testing.assert_array_equal(it.tree[k].cpu().numpy()[:n], tree2[k], err_msg=k)
    for e in it.blocks:
        assert int(e["status"].cpu()[0]) == 0
    # ---- the verify forward on that tree ----------------------------------------------------------------
    assert int(it.attn_status.cpu()[0]) == 0 and int(it.anc_status.cpu()[0]) == 0
    masks, depth, _ = oracle.tree_ancestors(tree2["parent"])
    np.testing.assert_array_equal(it.anc.cpu().numpy().view(np.uint32)[:n], masks)
    np.testing.assert_array_equal(it.depth.cpu().numpy()[:n], depth)
    offs = np.array([0, n], np.int32)
    for l, case in enumerate(target):
        kw = case.oracle_kwargs()
        kw.update(node_offsets=offs, parent=tree2["parent"], q=case.q[:n])
        ref_out, ref_lse, st = oracle.tree_attention(**kw)
        assert st[0] == 0
        got = it.out_all[l].float().cpu().numpy().astype(np.float64)[:n]
        assert _close(got, ref_out), f"target layer {l}"
        assert (np.abs(it.lse_all[l].cpu().numpy()[:n] - ref_lse) <= 1e-5 * np.maximum(1, np.abs(ref_lse))).all()
    ref = oracle.verify_accept(logits[:n], offs, tree2["parent"], tree2["tok"], 2 * K)
    assert int(ref["accept_len"][0]) == planted[0] and int(ref["bonus"][0]) == planted[1]
    for key in ("accept_len", "path_nodes", "out_tokens", "bonus", "status"):
        np.testing.assert_array_equal(it.accept[key].cpu().numpy(), ref[key], err_msg=key)
    np.testing.assert_array_equal(it.accept["amax"].cpu().numpy()[:n], ref["amax"])
    # the row that proposed each node's children, recorded by the expansions, and the verifier-derived signal
    child_row = np.full(n, -1, np.int32)
    global_row = np.full(n, -1, np.int32)       # per node: the iteration-wide row that proposed it
    row_base = np.cumsum([0] + [b.scores.shape[0] for b in blocks])
    first_new = 1
    for m, b in enumerate(blocks):                      # nodes are appended block by block, in row order
        res_m, _ = _oracle_tree(blocks[:m + 1])
        for c in range(first_new, res_m["n_nodes"]):
            child_row[tree2["parent"][c]] = row_base[m] + tree2["node_row"][c]
            global_row[c] = row_base[m] + tree2["node_row"][c]
        first_new = res_m["n_nodes"]
    np.testing.assert_array_equal(it.child_row.cpu().numpy()[:n], child_row)
    # the device numbers the rows through the blocks of the iteration (row_base of each expansion)
    np.testing.assert_array_equal(it.tree["node_row"].cpu().numpy()[:n], global_row)
    scores_all = np.concatenate([b.scores for b in blocks])
    sig = oracle.verifier_signal(scores_all, offs, child_row, ref["path_nodes"], ref["accept_len"], ref["bonus"], 2 * K)
    assert int(it.signal_status.cpu()[0]) == int(sig["status"][0]) == 0
    assert abs(float(it.r_prob.cpu()[0]) - sig["r_prob"][0]) <= 2e-5 * max(sig["r_prob"][0], 1e-3)
    caches = [(target, it.k_all, it.v_all, it.new_len, it.compact_status, "target", offs, ref["path_nodes"])]
    if it.drafter_cases:   # the drafter commits the block rows that proposed the accepted nodes
        rows = oracle.path_rows(offs, global_row, ref["path_nodes"], ref["accept_len"], 2 * K)
        assert int(rows["status"][0]) == 0 and int(it.path_rows_status.cpu()[0]) == 0
        np.testing.assert_array_equal(it.path_rows.cpu().numpy(), rows["path_rows"])
        caches.append((it.drafter_cases, it.drafter_k, it.drafter_v, it.drafter_new_len, it.drafter_compact_status,
                       "drafter", it.drafter_cases[0].node_offsets, rows["path_rows"]))
    for cases, k_all, v_all, got_len, got_status, who, c_offs, c_path in caches:
        c0 = cases[0]
        assert int(got_status.cpu()[0]) == 0
        for name, got_all in (("k", k_all), ("v", v_all)):
            cache = np.stack([getattr(c, name) for c in cases]).reshape(-1)
            ref_c, ref_len, _ = oracle.kv_compact(
                n_kv_heads=c0.n_kv_heads, head_dim=c0.head_dim, cache=cache, n_layers=len(cases),
                layer_stride_elems=int(c0.k.size), kv_capacity=c0.kv_capacity, prefix_len=c0.prefix_len,
                node_offsets=c_offs, path_nodes=c_path, accept_len=ref["accept_len"], max_depth=2 * K)
            new_len = int(ref_len[0])
            assert new_len == int(c0.prefix_len[0]) + planted[0] + 1
            row = c0.n_kv_heads * c0.head_dim
            np.testing.assert_array_equal(got_len.cpu().numpy(), ref_len)
            np.testing.assert_array_equal(_bits(got_all).reshape(len(cases), -1)[:, :new_len * row],
                                          ref_c.reshape(len(cases), -1)[:, :new_len * row], err_msg=f"{who} {name}")
    # ---- the drafter's side of every block --------------------------------------------------------------
    for m, (b, e) in enumerate(zip(blocks, it.blocks)):
        ref_f = oracle.rank_features(b.scores)
        got_f = e["features"].cpu().numpy().astype(np.float64)
        fin = np.isfinite(ref_f)
        assert (np.abs(got_f[fin] - ref_f[fin]) <= 2e-5 * np.maximum(1, np.abs(ref_f[fin]))).all()
        if weights is None:
            continue
        assert int(e["dense_status"].cpu()[0]) == 0 and int(e["shift_status"].cpu()[0]) == 0
        if m == 0:
            ref_c = oracle.shift_project(b.cond, weights.w_cond, 0)
            got_c = e["c"].float().cpu().numpy().astype(np.float64)
            assert _close(got_c, ref_c)
            c_bits = _bits(e["c"])       # the fused input is checked on the condition the device produced ...
            c_bits_ref = W.f32_to_bf16_bits(ref_c.astype(np.float32))
            # ... which must be the oracle's condition rounded to bf16, up to the last bit of a few entries
            assert (np.abs(c_bits.astype(np.int64) - c_bits_ref.astype(np.int64)) <= 1).mean() > 0.99
            cond = c_bits_ref
        else:
            cond = b.cond
        ref_h0 = oracle.fuse_project(cond, b.embed, weights.queries, weights.w_fuse, *weights.gains, eps=weights.eps)
        got_h0 = e["h0"].float().cpu().numpy().astype(np.float64)
        scale = max(1.0, float(np.sqrt(np.mean(ref_h0 ** 2))))
        assert _close(got_h0, ref_h0, 2 * scale if m == 0 else scale), f"fused input of block {m}"
        for l, (case, a) in enumerate(zip(b.attn, e["attn"])):
            ref_out, ref_lse, _ = oracle.tree_attention(**case.oracle_kwargs())
            assert _close(a["out"].float().cpu().numpy().astype(np.float64), ref_out), f"drafter attention {m}/{l}"
            assert int(a["status"].cpu()[0]) == 0
        for l, h in enumerate(b.hidden):
            ref_s = oracle.shift_project(h, weights.w_shift[l], K)
            assert _close(e["shifted"][l].float().cpu().numpy().astype(np.float64), ref_s), f"shift {m}/{l}"


def test_iteration_matches_the_oracle_chain():
    built = _build(9001)
    built[0].run()
    torch.cuda.synchronize()
    _check_against_oracle(*built)


def test_iteration_replayed_from_one_cuda_graph():
    """The chain has no host round trip, so one graph holds it; a replay on fresh inputs gives the same
    results as the eager run of an identical second instance."""
    it, *rest = _build(9002, with_drafter=True)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        # warm-up outside the capture on a twin, so that the captured instance's caches are untouched
        twin, *_ = _build(9002, with_drafter=True)
        twin.run()
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            it.run()
        g.replay()
        s.synchronize()
    _check_against_oracle(it, *rest)
    for key in ("accept_len", "path_nodes", "out_tokens", "bonus"):
        assert torch.equal(it.accept[key], twin.accept[key]), key
    n = rest[2]                                   # rows past the tree's node count are never written
    assert torch.equal(it.out_all[:, :n].view(torch.int16), twin.out_all[:, :n].view(torch.int16))
    assert it.launches() > 0


def test_iteration_without_the_drafter_side_and_budget_cut():
    """Only the tree path (expansion -> verify -> accept -> compact), with a node budget the second block overruns."""
    global BUDGET
    old = BUDGET
    BUDGET = 14
    try:
        built = _build(9003, n_target_layers=1, with_drafter=False)
        assert built[3] == 14                      # the tree is full: the last rows were cut
        built[0].run()
        torch.cuda.synchronize()
        _check_against_oracle(*built)
    finally:
        BUDGET = old


def test_iteration_with_stochastic_verification():
    """Temperature 1: the tree grown on the device is verified by rejection sampling, the drafter's rows found
    through the child_row array the expansions filled in; walk and signal against the oracle on the same tree."""
    from test_gpu_tree_ops import _robust_uniforms
    it, blocks, tree2, n, logits, target, weights, planted = _build(9004, n_target_layers=1, with_drafter=False)
    rng = W.rng_for(9005)
    offs = np.array([0, n], np.int32)
    child_row = np.full(n, -1, np.int32)
    row_base = np.cumsum([0] + [b.scores.shape[0] for b in blocks])
    first_new = 1
    for m in range(len(blocks)):
        res_m, _ = _oracle_tree(blocks[:m + 1])
        for c in range(first_new, res_m["n_nodes"]):
            child_row[tree2["parent"][c]] = row_base[m] + tree2["node_row"][c]
        first_new = res_m["n_nodes"]
    scores_all = np.concatenate([b.scores for b in blocks])
    args = (logits[:n], scores_all, offs, tree2["parent"], tree2["tok"], child_row)
    u_a, u_b, ref = _robust_uniforms(rng, args, 1.0, 2 * K, n, 1)
    u_full = np.zeros(BUDGET, np.float32)
    u_full[:n] = u_a
    it2 = SpecBlockIteration(block_k=K, bmap=BMAP, node_budget=BUDGET, root_tok=ROOT_TOK, blocks=blocks,
                             target_layers=target, logits=logits, max_depth=2 * K, temperature=1.0, u_accept=u_full,
                             u_bonus=u_b)
    it2.run()
    torch.cuda.synchronize()
    for key in ("status", "accept_len", "path_nodes"):
        np.testing.assert_array_equal(it2.accept[key].cpu().numpy(), ref[key], err_msg=key)
    a = int(ref["accept_len"][0])
    np.testing.assert_array_equal(it2.accept["out_tokens"].cpu().numpy()[0, :a], ref["out_tokens"][0, :a])
    lo = oracle.verify_sample(*args, 1.0, u_a, (u_b * np.float32(1 - 1e-3)).astype(np.float32), 2 * K)["bonus"][0]
    hi = oracle.verify_sample(*args, 1.0, u_a, (u_b * np.float32(1 + 1e-3)).astype(np.float32), 2 * K)["bonus"][0]
    got_bonus = int(it2.accept["bonus"].cpu()[0])
    assert lo <= got_bonus <= hi
    # the signal follows the sampled path and bonus (compared when the device drew the oracle's own bonus token,
    # which it does unless u_bonus falls within 1e-3 of a cell boundary)
    sig = oracle.verifier_signal(scores_all, offs, child_row, ref["path_nodes"], ref["accept_len"], ref["bonus"], 2 * K)
    assert int(it2.signal_status.cpu()[0]) == int(sig["status"][0])
    if got_bonus == int(ref["bonus"][0]) and sig["r_prob"][0] >= 0:
        assert abs(float(it2.r_prob.cpu()[0]) - sig["r_prob"][0]) <= 2e-5 * max(sig["r_prob"][0], 1e-3)
