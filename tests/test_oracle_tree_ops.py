"""Pins of the CPU oracle's integer steps (argmax, acceptance, compaction, top-k, branching) to
library routines, independent algorithms on exhaustive small inputs, planted constructions and
the paper's printed examples."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2605_07243_b200 import workloads as W


# ---- argmax / top-k against numpy -------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("vocab", [7, 1000, 32000])
def test_row_argmax_matches_numpy_first_maximum(dtype, vocab):
    rng = W.rng_for(21)
    x = rng.standard_normal((9, vocab), dtype=np.float32) * 2
    x[3] = np.round(x[3])                      # many exact ties
    x[4, :] = -np.inf
    x[5, 2] = np.nan
    x[5, 5] = np.inf
    if dtype == "bf16":
        bits = W.f32_to_bf16_bits(np.nan_to_num(x, nan=0.0, posinf=3e38, neginf=-3e38))
        ref = np.argmax(W.bf16_bits_to_f32(bits), axis=1)       # numpy: first maximal index
        got = oracle.row_argmax(bits)
    else:
        ref = np.argmax(np.where(np.isnan(x), -np.inf, x), axis=1)
        got = oracle.row_argmax(x)
    np.testing.assert_array_equal(got, ref)


def test_row_argmax_all_nan_row_and_signed_zero():
    x = np.full((2, 5), np.nan, np.float32)
    x[1] = [-0.0, 0.0, -1.0, 0.0, -0.0]        # +0 == -0: the first one wins
    np.testing.assert_array_equal(oracle.row_argmax(x), [0, 0])


@pytest.mark.parametrize("vocab", [5, 16, 1000, 32000])
def test_row_topk_matches_numpy_stable_sort(vocab):
    rng = W.rng_for(22)
    x = rng.standard_normal((6, vocab), dtype=np.float32) * 2
    x[1] = np.round(x[1] * 2) / 2              # ties
    x[2, ::3] = np.nan
    tok, val = oracle.row_topk(x)
    clean = np.where(np.isnan(x), -np.inf, x)
    order = np.argsort(-clean, axis=1, kind="stable")           # value desc, id asc
    k = min(16, vocab)
    np.testing.assert_array_equal(tok[:, :k], order[:, :k])
    np.testing.assert_array_equal(val[:, :k], np.take_along_axis(clean, order[:, :k], 1))
    assert (tok[:, k:] == -1).all() and np.isneginf(val[:, k:]).all()
    np.testing.assert_array_equal(tok[:, 0], oracle.row_argmax(x))   # k = 1 is the argmax


# ---- acceptance ------------------------------------------------------------------------------------

def _accept_by_recurrence(parent, tok, amax, max_depth):
    """Independent algorithm: acc[i] = acc[parent] and tok[i] == amax[parent], in index order."""
    n = len(parent)
    acc = [False] * n
    depth = [0] * n
    acc[0] = True
    best = 0
    for i in range(1, n):
        p = parent[i]
        depth[i] = depth[p] + 1
        acc[i] = acc[p] and tok[i] == amax[p] and depth[i] <= max_depth
        if acc[i] and depth[i] > depth[best]:
            best = i
    path = [best]
    while parent[path[-1]] >= 0:
        path.append(parent[path[-1]])
    path = path[::-1]
    return depth[best], path, [tok[i] for i in path[1:]] + [amax[best]]


def _all_trees(n):
    """Every parent array with parent[0] = -1 and parent[i] in [0, i)."""
    for rest in itertools.product(*[range(i) for i in range(1, n)]):
        yield [-1] + list(rest)


def test_accept_exhaustive_small_trees():
    """All trees with up to 5 nodes x all token/choice assignments over a 2-letter alphabet
    (plus 6-node trees on a sample): path enumeration equals the recurrence."""
    rng = W.rng_for(23)
    checked = 0
    for n in range(1, 7):
        for parent in _all_trees(n):
            assigns = itertools.product(range(2), repeat=2 * n - 1)
            if n == 6:
                assigns = [tuple(rng.integers(0, 3, 2 * n - 1)) for _ in range(4)]
            for a in assigns:
                tok = [7] + list(a[: n - 1])
                amax = list(a[n - 1:])
                r = oracle.accept_from_amax(parent, tok, amax, max_depth=8)
                ln, path, toks = _accept_by_recurrence(parent, tok, amax, 8)
                assert r["status"] == 0 and r["accept_len"] == ln
                assert list(r["path_nodes"][: ln + 1]) == path
                assert list(r["out_tokens"][: ln + 1]) == toks
                assert (r["path_nodes"][ln + 1:] == -1).all()
                checked += 1
    assert checked > 5000


def test_accept_exhaustive_three_letter_alphabet():
    """All trees with up to 4 nodes x every token / choice assignment over a THREE-letter alphabet (a third
    letter lets a sibling match while another one mismatches under the same parent): path enumeration equals
    the recurrence, also with the depth cut at 1 and 2."""
    checked = 0
    for n in range(1, 5):
        for parent in _all_trees(n):
            for a in itertools.product(range(3), repeat=2 * n - 1):
                tok = [7] + list(a[: n - 1])
                amax = list(a[n - 1:])
                for md in (1, 2, 8):
                    r = oracle.accept_from_amax(parent, tok, amax, max_depth=md)
                    ln, path, toks = _accept_by_recurrence(parent, tok, amax, md)
                    assert r["status"] == 0 and r["accept_len"] == ln
                    assert list(r["path_nodes"][: ln + 1]) == path
                    assert list(r["out_tokens"][: ln + 1]) == toks
                    checked += 1
    assert checked > 40000


def test_accept_random_trees_with_duplicates_and_depth_cut():
    rng = W.rng_for(24)
    for _ in range(300):
        n = int(rng.integers(1, 16))
        parent = W.random_tree(rng, n, 6)
        tok = rng.integers(0, 3, n)            # tiny alphabet: duplicate siblings, many matches
        amax = rng.integers(0, 3, n)
        md = int(rng.integers(1, 7))
        r = oracle.accept_from_amax(parent, tok, amax, md)
        ln, path, toks = _accept_by_recurrence(list(parent), list(tok), list(amax), md)
        assert r["accept_len"] == ln and list(r["path_nodes"][: ln + 1]) == path
        assert list(r["out_tokens"][: ln + 1]) == toks and r["bonus"] == toks[-1]


def test_accept_chain_is_longest_matching_prefix():
    """A chain tree is textbook greedy speculative verification of one draft sequence."""
    rng = W.rng_for(25)
    for _ in range(50):
        n = int(rng.integers(2, 12))
        tok = rng.integers(0, 2, n)
        amax = rng.integers(0, 2, n)
        matched = 0
        while matched < n - 1 and tok[matched + 1] == amax[matched]:
            matched += 1
        r = oracle.accept_from_amax(W.chain_tree(n), tok, amax, 16)
        assert r["accept_len"] == matched and r["bonus"] == amax[matched]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_accept_planted_path_is_recovered(dtype):
    rng = W.rng_for(26)
    parents = [W.random_tree(rng, int(n), 6) for n in (15, 1, 40, 9)]
    case = W.make_verify_case(rng, parents=parents, vocab=777, dtype=dtype)
    r = oracle.verify_accept(case.logits, case.node_offsets, case.parent, case.tok,
                             case.max_depth)
    assert not r["status"].any()
    np.testing.assert_array_equal(r["accept_len"], case.planted_len)
    np.testing.assert_array_equal(r["bonus"], case.planted_bonus)
    for b, path in enumerate(case.planted_path):
        assert list(r["path_nodes"][b, : len(path)]) == path


def test_accept_case_study_tree(golden_dir):
    """Case study, tree (b): the K=4 chain is accepted and a bonus follows -> five tokens."""
    nodes, expect = [], {}
    for line in open(os.path.join(golden_dir, "case_study_tree.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("expect_"):
            key, *vals = line.split()
            expect[key] = [int(t) for t in vals]
        else:
            nodes.append([int(t) for t in line.split()])
    nodes = np.asarray(nodes)
    r = oracle.accept_from_amax(nodes[:, 1], nodes[:, 2], nodes[:, 3], 8)
    a = expect["expect_accept_len"][0]
    assert r["accept_len"] == a and a + 1 == 5
    assert list(r["out_tokens"][: a + 1]) == expect["expect_tokens"]


def test_accept_rejects_second_root_and_bad_parent():
    assert oracle.accept_from_amax([-1, -1], [1, 2], [2, 2], 4)["status"] == 4
    assert oracle.accept_from_amax([-1, 1], [1, 2], [2, 2], 4)["status"] == 4


# ---- compaction ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("page_size", [0, 16])
def test_kv_compact_equals_numpy_gather(page_size):
    rng = W.rng_for(27)
    parents = [W.random_tree(rng, 20, 6), W.random_tree(rng, 9, 4)]
    L = 3
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[19, 33], n_q_heads=4,
                            n_kv_heads=2, head_dim=16, page_size=page_size)
    layers = np.stack([rng.integers(0, 65536, case.k.shape).astype(np.uint16) for _ in range(L)])
    paths = np.full((2, 7), -1, np.int32)
    paths[0, :4] = [0, 2, 5, 11]
    paths[1, :1] = [0]
    alen = np.asarray([3, 0], np.int32)
    new, new_len, st = oracle.kv_compact(
        n_kv_heads=2, head_dim=16, cache=layers.reshape(-1), n_layers=L,
        layer_stride_elems=layers[0].size, page_size=page_size, max_pages=case.max_pages,
        num_pages=case.num_pages, kv_capacity=case.kv_capacity, page_table=case.page_table,
        prefix_len=case.prefix_len, node_offsets=case.node_offsets, path_nodes=paths,
        accept_len=alen, max_depth=6)
    assert not st.any()
    np.testing.assert_array_equal(new_len, case.prefix_len + alen + 1)
    new = new.reshape(layers.shape)
    ref = layers.copy()
    for b in range(2):
        P = int(case.prefix_len[b])
        src = [W.kv_slot(case, b, P + int(p)) for p in paths[b, : alen[b] + 1]]
        dst = [W.kv_slot(case, b, P + j) for j in range(alen[b] + 1)]
        si, sj = zip(*src)
        di, dj = zip(*dst)
        ref[:, list(di), list(dj)] = layers[:, list(si), list(sj)]     # numpy fancy-index gather
    np.testing.assert_array_equal(new, ref)


def test_compaction_then_chain_attention_equals_tree_attention_of_last_path_node():
    """After compaction the accepted path is an ordinary prefix: a new token attending to the
    compacted cache sees exactly what the path's last node saw (plus itself)."""
    rng = W.rng_for(28)
    par = W.random_tree(rng, 12, 5)
    case = W.make_attn_case(rng, parents=[par], prefix_lens=[23], n_q_heads=2, n_kv_heads=1,
                            head_dim=32, capacity_pad=4)
    end = 11
    path = [end]
    while par[path[-1]] >= 0:
        path.append(int(par[path[-1]]))
    path = path[::-1]
    a = len(path) - 1
    paths = np.full((1, 8), -1, np.int32)
    paths[0, : a + 1] = path
    out_tree, lse_tree, _ = oracle.tree_attention(**case.oracle_kwargs())
    new = {}
    for name in ("k", "v"):
        arr = getattr(case, name)
        new[name], new_len, st = oracle.kv_compact(
            n_kv_heads=1, head_dim=32, cache=arr.reshape(-1), n_layers=1, layer_stride_elems=0,
            kv_capacity=case.kv_capacity, prefix_len=case.prefix_len,
            node_offsets=case.node_offsets, path_nodes=paths, accept_len=[a], max_depth=7)
        new[name] = new[name].reshape(arr.shape)
    # the path's last node, re-asked as a single node whose own K/V sit at the new prefix end
    P2 = int(new_len[0]) - 1
    kw = case.oracle_kwargs()
    kw.update(k=new["k"], v=new["v"], prefix_len=[P2], node_offsets=[0, 1], parent=[-1],
              q=case.q[end:end + 1])
    out2, lse2, st2 = oracle.tree_attention(**kw)
    np.testing.assert_allclose(out2[0], out_tree[end], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse2[0], lse_tree[end], rtol=1e-13)


def test_kv_compact_flags_bad_paths():
    rng = W.rng_for(29)
    case = W.make_attn_case(rng, parents=[W.chain_tree(5)], prefix_lens=[4], n_q_heads=1,
                            n_kv_heads=1, head_dim=16)
    for bad in ([1, 2, -1], [0, 3, 2], [0, 2, 7]):
        _n, new_len, st = oracle.kv_compact(
            n_kv_heads=1, head_dim=16, cache=case.k.reshape(-1), n_layers=1, layer_stride_elems=0,
            kv_capacity=case.kv_capacity, prefix_len=case.prefix_len,
            node_offsets=case.node_offsets, path_nodes=np.asarray([bad], np.int32),
            accept_len=[2], max_depth=2)
        assert st[0] == 4 and new_len[0] == 4


# ---- branching ---------------------------------------------------------------------------------------------

def _read_expand_examples(golden_dir):
    ex, cur = {}, None
    for line in open(os.path.join(golden_dir, "expand_examples.txt")):
        t = line.split()
        if not t or t[0] == "#" or t[0].startswith("#"):
            continue
        if t[0] == "example":
            cur = dict(nodes=[])
            ex[t[1]] = cur
        elif t[0] == "node":
            cur["nodes"].append([int(x) for x in t[1:]])
        elif t[0] == "existing":
            cur["existing"] = t[1]
        elif t[0] != "end":
            cur[t[0]] = [int(x) for x in t[1:]]
    return ex


def _scores_with_known_ranking(rng, n_rows, vocab):
    """Row r ranks the ids of a random permutation: its j-th entry gets the j-th largest score."""
    ranking = np.stack([rng.permutation(vocab) for _ in range(n_rows)])
    scores = np.zeros((n_rows, vocab), np.float32)
    for r in range(n_rows):
        scores[r, ranking[r]] = 100.0 - np.arange(vocab, dtype=np.float32)
    return scores, ranking


def test_path_rows_hand_worked_two_block_tree():
    """K = 4.  Block 1 (rows 0..3) starts at the root: row 0 proposes nodes 1, 2 (siblings), row 1 node 3 under node 1,
    row 2 node 4, row 3 node 5 (the chain 1-3-4-5).  Block 2 (rows 4..7) starts at sibling 2: row 4 proposes nodes
    6, 7 under 2, row 5 node 8 under 6.  A committed position keeps the row of its own draft forward (App. A.2),
    and slot 0 of the row numbering is the last committed position."""
    offs = [0, 9]
    node_row = [-1, 0, 0, 1, 2, 3, 4, 4, 5]
    cases = [([0, 1, 3, 4, 5], 4, [0, 1, 2, 3, 4]),          # the whole first chain: rows 0..3 -> slots 1..4
             ([0, 2, 7, -1, -1], 2, [0, 1, 5, -1, -1]),     # sibling 2 shares row 0 with node 1; node 7 shares row 4
             ([0, 2, 6, 8, -1], 3, [0, 1, 5, 6, -1]),
             ([0, -1, -1, -1, -1], 0, [0, -1, -1, -1, -1])]  # nothing drafted was accepted
    for path, a, want in cases:
        r = oracle.path_rows(offs, node_row, [path], [a], 4)
        assert r["status"].tolist() == [0]
        assert r["path_rows"][0].tolist() == want
    # the rows must increase along a path, a path node must exist and must have a row, a must fit
    for path, a in (([0, 3, 1, -1, -1], 2), ([0, 9, -1, -1, -1], 1), ([0, 0, -1, -1, -1], 1), ([0, 1, 3, 4, 5], 5)):
        r = oracle.path_rows(offs, node_row, [path], [a], 4)
        assert r["status"].tolist() == [4] and r["path_rows"][0].tolist() == [0, -1, -1, -1, -1]


def test_path_rows_equals_numpy_fancy_indexing_on_random_batches():
    rng = W.rng_for(5150)
    for _ in range(50):
        B, md = int(rng.integers(1, 5)), int(rng.integers(1, 9))
        n = rng.integers(md + 1, 40, size=B)
        offs = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
        row_begin = np.cumsum(np.concatenate([[0], n[:-1] + 3])).astype(np.int32)   # any first row per sequence
        node_row = np.full(offs[-1], -1, np.int32)
        paths, acc, want = [], [], []
        for b in range(B):
            # rows never decrease with the node id; siblings share a row
            rows_b = np.sort(rng.integers(0, n[b] + 3, size=n[b] - 1))
            node_row[offs[b] + 1:offs[b + 1]] = row_begin[b] + rows_b
            distinct = np.unique(rows_b)
            a = int(rng.integers(0, min(md, len(distinct)) + 1))
            # one node from each of `a` different rows, in row order: the rows increase along the path
            picked = np.sort(rng.choice(distinct, size=a, replace=False))
            nodes = np.array([1 + int(rng.choice(np.flatnonzero(rows_b == r))) for r in picked], np.int64)
            path = np.full(md + 1, -1, np.int32)
            path[0] = 0
            path[1:a + 1] = nodes
            w = np.full(md + 1, -1, np.int32)
            w[0] = 0
            w[1:a + 1] = 1 + node_row[offs[b] + nodes] - row_begin[b]
            paths.append(path), acc.append(a), want.append(w)
        r = oracle.path_rows(offs, node_row, np.stack(paths), acc, md, row_begin=row_begin)
        assert not r["status"].any()
        np.testing.assert_array_equal(r["path_rows"], np.stack(want))


def test_expand_hand_derived_examples(golden_dir):
    """The two printed branching maps on hand-worked blocks, incl. a width-0 bucket that ends a
    block, a second block level, and the node budget cutting a row."""
    ex = _read_expand_examples(golden_dir)
    rng = W.rng_for(30)
    results = {}
    for name in ("A", "B", "C"):
        e = ex[name]
        n_rows = len(e["bucket"])
        scores, ranking = _scores_with_known_ranking(rng, n_rows, 50)
        tree = None if e["existing"] == "0" else results[e["existing"]]
        n0 = 0 if tree is None else len(tree["tok"])
        r = oracle.tree_expand(scores, e["block_k"][0], e["bucket"], e["bmap"], e["start_parent"],
                               e["budget"][0], tree=tree)
        assert r["status"] == 0
        want = np.asarray(e["nodes"])
        assert r["n_nodes"] == n0 + len(want)
        new = slice(n0, r["n_nodes"])
        np.testing.assert_array_equal(r["parent"][new], want[:, 0])
        np.testing.assert_array_equal(r["depth"][new], want[:, 1])
        np.testing.assert_array_equal(r["node_row"][new], want[:, 2])
        np.testing.assert_array_equal(r["node_rank"][new], want[:, 3])
        np.testing.assert_array_equal(r["tok"][new], ranking[want[:, 2], want[:, 3]])
        results[name] = {k: r[k][: r["n_nodes"]] for k in
                         ("tok", "parent", "depth", "node_row", "node_rank")}


def test_expand_width_one_gives_pure_chains_and_invariants():
    rng = W.rng_for(31)
    case = W.make_expand_case(rng, n_starts=3, block_k=4, vocab=500, bmap=[1, 1, 1, 1],
                              node_budget=64)
    r = oracle.tree_expand(case.scores, 4, case.bucket, case.bmap, case.start_parent, 64)
    assert r["n_nodes"] == 12
    for i in range(3):
        np.testing.assert_array_equal(r["parent"][4 * i: 4 * i + 4],
                                      [-1, 4 * i, 4 * i + 1, 4 * i + 2])
        np.testing.assert_array_equal(r["depth"][4 * i: 4 * i + 4], [0, 1, 2, 3])
    np.testing.assert_array_equal(r["tok"][:12], np.argmax(case.scores, axis=1))
    # random maps: budget respected, parents precede children, depth bounded by M*K
    for trial in range(20):
        bmap = rng.integers(0, 11, 4)
        existing = W.random_tree(rng, 6, 3)
        c = W.make_expand_case(rng, n_starts=5, block_k=4, vocab=300, bmap=bmap, node_budget=60,
                               existing_parent=existing)
        r = oracle.tree_expand(c.scores, 4, c.bucket, c.bmap, c.start_parent, 60, tree=c.tree)
        n = r["n_nodes"]
        assert 6 <= n <= 60
        assert (r["parent"][6:n] < np.arange(6, n)).all()
        assert r["depth"][:n].max() <= 3 + 4
        assert (r["depth"][6:n] == r["depth"][r["parent"][6:n]] + 1).all()


def test_expand_rejects_bad_arguments():
    rng = W.rng_for(32)
    c = W.make_expand_case(rng, n_starts=1, block_k=4, vocab=50, bmap=[2, 4, 10, 0],
                           node_budget=20)
    assert oracle.tree_expand(c.scores, 4, [0, 1, 4, 0], c.bmap, [-1], 20)["status"] == 1
    assert oracle.tree_expand(c.scores, 4, c.bucket, [2, 4, 17, 0], [-1], 20)["status"] == 1
    assert oracle.tree_expand(c.scores, 4, c.bucket, c.bmap, [0], 20)["status"] == 1


# ---- rank-head distribution summary psi(p) (App. B) --------------------------------------------------------

def test_rank_features_match_scipy_and_closed_forms():
    from scipy.special import log_softmax
    from scipy.stats import entropy as scipy_entropy
    rng = W.rng_for(33)
    x = (rng.standard_normal((5, 3000), dtype=np.float32) * 3).astype(np.float32)
    x[1] = np.round(x[1])                       # ties among the leaders
    x[2, ::7] = np.nan                          # NaN counts as -inf
    x[3, 5:] = -np.inf                          # only five finite scores
    f = oracle.rank_features(x)
    clean = np.where(np.isnan(x), -np.inf, x).astype(np.float64)
    lsm = log_softmax(clean, axis=1)            # library routine
    order = np.argsort(-clean, axis=1, kind="stable")
    top = np.take_along_axis(clean, order[:, :10], 1)
    np.testing.assert_allclose(f[:, :10], np.take_along_axis(lsm, order[:, :10], 1), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f[:, 10], top[:, 0] - top[:, 1], atol=1e-12)
    np.testing.assert_allclose(f[:, 11], top[:, 0] - top[:, 2], atol=1e-12)
    np.testing.assert_allclose(f[:, 12], top[:, 0] - top[:, 4], atol=1e-12)
    np.testing.assert_allclose(f[:, 13], np.exp(lsm.max(axis=1)), rtol=1e-12)
    np.testing.assert_allclose(f[:, 14], [scipy_entropy(np.exp(r)) for r in lsm], rtol=1e-10)
    assert np.isneginf(f[3, 5:10]).all()          # row 3 has only five finite scores
    # closed forms: a uniform row has entropy ln V, zero gaps and log-probs -ln V ...
    V = 1000
    u = oracle.rank_features(np.full((1, V), 2.5, np.float32))[0]
    np.testing.assert_allclose(u[:10], -np.log(V), rtol=1e-12)
    np.testing.assert_allclose(u[10:13], 0.0, atol=1e-12)
    np.testing.assert_allclose(u[13:], [1.0 / V, np.log(V)], rtol=1e-12)
    # ... and one token 50 above the rest owns the distribution: entropy ~ 0, top probability ~ 1
    d = np.zeros((1, V), np.float32)
    d[0, 123] = 50.0
    o = oracle.rank_features(d)[0]
    assert abs(o[0]) < 1e-18 and abs(o[13] - 1.0) < 1e-15 and o[14] < 1e-15
    np.testing.assert_allclose(o[10:13], 50.0)
    # fewer than ten / five tokens
    s = oracle.rank_features(np.asarray([[1.0, 3.0, 2.0]], np.float32))[0]
    assert np.isneginf(s[3:10]).all() and s[10] == 1.0 and s[11] == 2.0 and np.isposinf(s[12])


# ---- verifier-derived update signal s = sum (1 - r) (Sec. 3.4; Alg. 2 line 2) ---------------------------------

def _signal_inputs(best_nodes, bonus, child_row, n_nodes, max_depth=4):
    """One sequence per entry; the accepted path is only needed at its last node."""
    B = len(best_nodes)
    node_offsets = np.arange(B + 1, dtype=np.int32) * n_nodes
    path = np.full((B, max_depth + 1), -1, np.int32)
    accept_len = np.zeros(B, np.int32)
    for b, node in enumerate(best_nodes):
        accept_len[b] = b % (max_depth + 1)
        path[b, accept_len[b]] = node
    return dict(node_offsets=node_offsets, child_row=np.tile(np.asarray(child_row, np.int32), B), path_nodes=path,
                accept_len=accept_len, bonus=np.asarray(bonus, np.int32), max_depth=max_depth)


def test_verifier_signal_matches_scipy_softmax_and_closed_forms():
    from scipy.special import softmax
    rng = W.rng_for(34)
    V, R = 777, 6
    x = (rng.standard_normal((R, V), dtype=np.float32) * 3).astype(np.float32)
    x[2, ::5] = np.nan                           # NaN counts as -inf
    x[3, 10:] = -np.inf
    child_row = [4, 2, -1, 0, 3, 5, 1]           # node -> drafter row that predicted its successor
    best = [0, 1, 3, 4, 5, 6, 2]
    bonus = [5, 10, 700, 3, V - 1, 0, 9]
    got = oracle.verifier_signal(x, **_signal_inputs(best, bonus, child_row, 7))
    p = softmax(np.where(np.isnan(x), -np.inf, x).astype(np.float64), axis=1)   # library routine
    want_r = np.asarray([p[child_row[n], t] if child_row[n] >= 0 else -1.0 for n, t in zip(best, bonus)])
    np.testing.assert_allclose(got["r_prob"], want_r, rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(got["signal"], np.where(want_r >= 0, 1.0 - want_r, 0.0), rtol=1e-12)
    assert (got["status"] == 0).all()
    assert got["r_prob"][6] == -1.0 and got["signal"][6] == 0.0    # nothing drafted after node 2: nothing rejected
    assert got["r_prob"][1] == 0.0                                  # token 10 sits on a NaN score of row 2

    # closed forms: a flat row gives r = 1/V; one token raised by c gives e^c / (e^c + V - 1)
    flat = np.full((1, V), -1.25, np.float32)
    g = oracle.verifier_signal(flat, **_signal_inputs([0], [123], [0], 1))
    np.testing.assert_allclose(g["signal"], 1.0 - 1.0 / V, rtol=1e-15)
    c = 6.5
    raised = np.zeros((1, V), np.float32)
    raised[0, 40] = c
    g = oracle.verifier_signal(raised, **_signal_inputs([0, 0], [40, 41], [0], 1))
    np.testing.assert_allclose(g["r_prob"], [np.exp(c) / (np.exp(c) + V - 1), 1.0 / (np.exp(c) + V - 1)], rtol=1e-13)
    # a row with no finite score is read as flat; a token outside the vocabulary has probability 0
    dead = np.full((1, V), -np.inf, np.float32)
    assert oracle.verifier_signal(dead, **_signal_inputs([0], [7], [0], 1))["r_prob"][0] == 1.0 / V
    out = oracle.verifier_signal(flat, **_signal_inputs([0, 0], [V, -1], [0], 1))
    assert (out["r_prob"] == 0.0).all() and (out["signal"] == 1.0).all()


def test_verifier_signal_invariants_accumulation_and_bounds():
    rng = W.rng_for(35)
    V = 50
    x = (rng.standard_normal((3, V), dtype=np.float32) * 2).astype(np.float32)
    # the probabilities of all tokens of one row sum to one
    r = oracle.verifier_signal(x, **_signal_inputs([0] * V, list(range(V)), [1], 1))["r_prob"]
    np.testing.assert_allclose(r.sum(), 1.0, rtol=1e-14)
    # adding a constant to a row changes nothing (values chosen exactly representable)
    y = np.round(x * 8) / 8
    a = oracle.verifier_signal(y, **_signal_inputs([0, 0], [3, 4], [2], 1))
    b = oracle.verifier_signal(y + np.float32(16.0), **_signal_inputs([0, 0], [3, 4], [2], 1))
    np.testing.assert_allclose(a["r_prob"], b["r_prob"], rtol=1e-13)
    # the query-level signal is the sum over iterations: feed the running value back in
    args = _signal_inputs([0, 0], [3, 4], [2], 1)
    s1 = oracle.verifier_signal(x, **args)
    s2 = oracle.verifier_signal(x, signal=s1["signal"], **_signal_inputs([0, 0], [5, 6], [0], 1))
    np.testing.assert_allclose(s2["signal"], (1 - s1["r_prob"]) + (1 - s2["r_prob"]), rtol=1e-14)
    assert (0 <= s1["signal"]).all() and (s1["signal"] <= 1).all()
    # out-of-range accept_len / path node / row are reported per sequence and change nothing
    bad = _signal_inputs([0, 0, 0], [1, 1, 1], [7], 1)      # row 7 of a 3-row matrix
    bad["accept_len"][1] = 9
    g = oracle.verifier_signal(x, signal=[0.5, 0.5, 0.5], **bad)
    assert (g["status"] == 5).all() and (g["signal"] == 0.5).all() and (g["r_prob"] == -1).all()
    bad = _signal_inputs([4], [1], [0], 1)                  # path node 4 of a 1-node tree
    assert oracle.verifier_signal(x, **bad)["status"][0] == 5


# ---- stochastic verification (temperature > 0): multi-candidate rejection sampling on the tree -----------------

def _one_level_case(rng, V, cand):
    """Root with len(cand) leaf children carrying the tokens `cand`; one drafter row."""
    n = 1 + len(cand)
    logits = (rng.standard_normal((n, V)) * 1.5).astype(np.float32)
    scores = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
    parent = np.asarray([-1] + [0] * len(cand), np.int32)
    tok = np.asarray([0] + list(cand), np.int32)
    child_row = np.asarray([0] + [-1] * len(cand), np.int32)
    return logits, scores, parent, tok, child_row


def _run_sample(case, u_accept, u_bonus, T=1.0, max_depth=4):
    logits, scores, parent, tok, child_row = case
    r = oracle.verify_sample(logits, scores, [0, len(parent)], parent, tok, child_row, T, u_accept, [u_bonus], max_depth)
    assert r["status"][0] == 0
    return int(r["accept_len"][0]), int(r["out_tokens"][0, 0]), int(r["bonus"][0])


def _threshold(f):
    """sup{u in [0,1]: f(u)} for a predicate that is true on [0, theta) (float32 resolution)."""
    if not f(0.0):
        return 0.0
    if f(np.nextafter(np.float32(1.0), np.float32(0.0))):
        return 1.0
    lo, hi = 0.0, 1.0
    for _ in range(30):
        mid = 0.5 * (lo + hi)
        lo, hi = (mid, hi) if f(mid) else (lo, mid)
    return 0.5 * (lo + hi)


def _bonus_distribution(run_with_u_bonus, V):
    """Measure of the u_bonus interval that yields each token (the bonus is monotone in u)."""
    edges = [0.0] + [_threshold(lambda u, v=v: run_with_u_bonus(u) <= v) for v in range(V - 1)] + [1.0]
    return np.diff(np.asarray(edges))


def test_verify_sample_one_candidate_from_q_commits_exactly_the_target_distribution():
    """Speculative sampling's identity: x ~ q accepted with probability min(1, p/q), else a draw from
    norm(max(p - q, 0)), is distributed as p.  Checked by exact integration over both uniforms."""
    from scipy.special import softmax
    rng = W.rng_for(36)
    V = 6
    first = np.zeros(V)
    base = None
    for x in range(V):
        rng_x = W.rng_for(360)                      # the same p and q for every candidate
        case = _one_level_case(rng_x, V, [x])
        if base is None:
            base = case
            p = softmax(case[0][0].astype(np.float64))
            q = softmax(case[1][0].astype(np.float64))
        theta = _threshold(lambda u: _run_sample(case, [0.0, u], 0.5)[0] == 1)
        np.testing.assert_allclose(theta, min(1.0, p[x] / q[x]), atol=2e-7)      # the acceptance rule itself
        first[x] += q[x] * theta
        if theta < 1.0:
            res = _bonus_distribution(lambda u: _run_sample(case, [0.0, 1.0], u)[2], V)
            want = np.maximum(p - q, 0.0)
            np.testing.assert_allclose(res, want / want.sum(), atol=5e-7)         # the residual distribution
            first += q[x] * (1.0 - theta) * res
    np.testing.assert_allclose(first, p, atol=2e-6)
    del rng


def test_verify_sample_two_candidates_without_replacement_is_still_exact():
    from scipy.special import softmax
    V = 5
    first = np.zeros(V)
    for x1 in range(V):
        for x2 in range(V):
            if x2 == x1:
                continue
            case = _one_level_case(W.rng_for(361), V, [x1, x2])
            p = softmax(case[0][0].astype(np.float64))
            q = softmax(case[1][0].astype(np.float64))
            q2 = q.copy()
            q2[x1] = 0.0
            q2 /= q2.sum()
            w = q[x1] * q2[x2]                        # probability of drawing (x1, x2) without replacement
            th1 = _threshold(lambda u: _run_sample(case, [0.0, u, 0.0], 0.5)[1] == x1 and
                             _run_sample(case, [0.0, u, 0.0], 0.5)[0] == 1)
            first[x1] += w * th1
            if th1 >= 1.0:
                continue
            th2 = _threshold(lambda u: _run_sample(case, [0.0, 1.0, u], 0.5)[0] == 1)
            first[x2] += w * (1.0 - th1) * th2
            if th2 >= 1.0:
                continue
            res = _bonus_distribution(lambda u: _run_sample(case, [0.0, 1.0, 1.0], u)[2], V)
            first += w * (1.0 - th1) * (1.0 - th2) * res
    p = softmax(_one_level_case(W.rng_for(361), V, [0, 1])[0][0].astype(np.float64))
    np.testing.assert_allclose(first, p, atol=5e-6)


def test_verify_sample_low_temperature_is_greedy_and_walks_the_tree():
    rng = W.rng_for(37)
    par = W.random_tree(rng, 30, 6)
    ver = W.make_verify_case(rng, parents=[par], vocab=300, dtype="f32", std=2.0, accept_lens=[4], max_depth=6)
    n = len(par)
    scores = (rng.standard_normal((n, 300)) * 2).astype(np.float32)
    child_row = np.arange(n, dtype=np.int32)
    greedy = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
    # T -> 0 against a flat draft distribution (which no temperature sharpens): the target becomes
    # one-hot at its argmax, a child is accepted iff it carries that token, whatever the uniforms
    flat = np.zeros_like(scores)
    for rep in range(5):
        u_a = rng.random(n).astype(np.float32)
        got = oracle.verify_sample(ver.logits, flat, ver.node_offsets, ver.parent, ver.tok, child_row, 0.02, u_a,
                                   [rng.random()], ver.max_depth)
        for key in ("accept_len", "path_nodes", "out_tokens", "bonus"):
            np.testing.assert_array_equal(got[key], greedy[key], err_msg=key)
    # at temperature 1 the result is a root-to-node path whose tokens are the path's, followed by the bonus
    for rep in range(20):
        got = oracle.verify_sample(ver.logits, scores, ver.node_offsets, ver.parent, ver.tok, child_row, 1.0,
                                   rng.random(n).astype(np.float32), [rng.random()], 3)
        a = int(got["accept_len"][0])
        path = got["path_nodes"][0]
        assert 0 <= a <= 3 and path[0] == 0 and (path[a + 1:] == -1).all()
        for t in range(1, a + 1):
            assert ver.parent[path[t]] == path[t - 1] and got["out_tokens"][0, t - 1] == ver.tok[path[t]]
        assert got["out_tokens"][0, a] == got["bonus"][0] and 0 <= got["bonus"][0] < 300
    # invalid trees and a missing drafter row are reported
    bad = oracle.verify_sample(ver.logits, scores, ver.node_offsets, np.full(n, -1, np.int32), ver.tok, child_row, 1.0,
                               np.zeros(n, np.float32), [0.5], 3)
    assert bad["status"][0] == 4
    no_row = oracle.verify_sample(ver.logits, scores, ver.node_offsets, ver.parent, ver.tok, np.full(n, -1, np.int32),
                                  1.0, np.zeros(n, np.float32), [0.5], 3)
    assert no_row["status"][0] == 5


# ---- layer-wise shift projection between drafter layers (Sec. 3.1) ---------------------------------------------

def test_shift_project_matches_numpy_on_the_concatenated_input():
    rng = W.rng_for(38)
    R, K, d, d_out = 12, 4, 96, 40
    h = W.f32_to_bf16_bits(rng.standard_normal((R, d), dtype=np.float32))
    w = W.f32_to_bf16_bits(rng.standard_normal((d_out, 2 * d), dtype=np.float32) * 0.1)
    hf = W.bf16_bits_to_f32(h).astype(np.float64)
    wf = W.bf16_bits_to_f32(w).astype(np.float64)
    prev = np.asarray([r - 1 if r % K else r for r in range(R)])
    want = np.concatenate([hf, hf[prev]], axis=1) @ wf.T          # library matmul on [h_k, h_{k-1}]
    np.testing.assert_allclose(oracle.shift_project(h, w, K), want, rtol=1e-12, atol=1e-12)
    # plain projection
    w1 = W.f32_to_bf16_bits(rng.standard_normal((d_out, d), dtype=np.float32))
    np.testing.assert_allclose(oracle.shift_project(h, w1, 0), hf @ W.bf16_bits_to_f32(w1).astype(np.float64).T,
                               rtol=1e-12, atol=1e-12)
    # W = [I, 0] returns the input; W = [0, I] returns the previous position's state, and the
    # first position of a block gets its own (the convention h_0 = h_1)
    eye = np.eye(d, dtype=np.float32)
    zero = np.zeros((d, d), np.float32)
    np.testing.assert_array_equal(oracle.shift_project(h, W.f32_to_bf16_bits(np.hstack([eye, zero])), K), hf)
    np.testing.assert_array_equal(oracle.shift_project(h, W.f32_to_bf16_bits(np.hstack([zero, eye])), K), hf[prev])
    assert (prev[::K] == np.arange(0, R, K)).all()


# ---- the drafter's fused per-position input (Sec. 3.1, the equation for h^(0)) ------------------------------------

def _fuse_inputs(rng, S, K, d, d_out, scale=1.0):
    c = W.f32_to_bf16_bits(rng.standard_normal((S, d), dtype=np.float32) * 3.0 * scale)
    e = W.f32_to_bf16_bits(rng.standard_normal((S, d), dtype=np.float32) * 0.05)
    q = W.f32_to_bf16_bits(rng.standard_normal((K, d), dtype=np.float32))
    w = W.f32_to_bf16_bits(rng.standard_normal((d_out, 3 * d), dtype=np.float32) * 0.1)
    return c, e, q, w


def test_fuse_project_matches_numpy_on_the_concatenated_normalised_input():
    rng = W.rng_for(51)
    S, K, d, d_out = 5, 4, 96, 40                                 # W is not square: a transposed operand cannot pass
    c, e, q, w = _fuse_inputs(rng, S, K, d, d_out)
    gains = [rng.uniform(0.5, 1.5, d).astype(np.float32) for _ in range(3)]
    eps = 1e-5
    f64 = lambda bits: W.bf16_bits_to_f32(bits).astype(np.float64)

    def norm(x, g):
        return g.astype(np.float64) * x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)

    cn, en, qn = norm(f64(c), gains[0]), norm(f64(e), gains[1]), norm(f64(q), gains[2])
    x = np.concatenate([np.repeat(cn, K, axis=0), np.repeat(en, K, axis=0), np.tile(qn, (S, 1))], axis=1)
    want = x @ f64(w).T
    got = oracle.fuse_project(c, e, q, w, *gains, eps=eps)
    assert got.shape == (S * K, d_out)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # gains left out are ones
    ones = np.ones(d, np.float32)
    np.testing.assert_allclose(oracle.fuse_project(c, e, q, w, eps=eps), oracle.fuse_project(c, e, q, w, ones, ones, ones, eps=eps),
                               rtol=0, atol=0)


def test_fuse_project_closed_forms_with_selector_weights():
    S, K, d = 2, 3, 8
    eye, zero = np.eye(d, dtype=np.float32), np.zeros((d, d), np.float32)
    # c_0 = (3, 4, 3, 4, ...): mean square 12.5; c_1 constant -2: norm = -1 everywhere (eps = 0)
    c = np.stack([np.tile([3.0, 4.0], d // 2), np.full(d, -2.0)]).astype(np.float32)
    e = np.stack([np.full(d, 0.5), np.tile([1.0, -1.0], d // 2)]).astype(np.float32)
    q = np.stack([np.full(d, 7.0), np.tile([0.0, 2.0], d // 2), np.tile([1.0, 0.0], d // 2)]).astype(np.float32)
    bits = W.f32_to_bf16_bits
    sel = lambda i: bits(np.hstack([eye if j == i else zero for j in range(3)]))
    out_c = oracle.fuse_project(bits(c), bits(e), bits(q), sel(0), eps=0.0)
    for k in range(K):                                            # the prefix broadcast: the same c for every position
        np.testing.assert_allclose(out_c[0 * K + k], np.tile([3.0, 4.0], d // 2) / np.sqrt(12.5), rtol=1e-15)
        np.testing.assert_allclose(out_c[1 * K + k], np.full(d, -1.0), rtol=1e-15)
    out_e = oracle.fuse_project(bits(c), bits(e), bits(q), sel(1), eps=0.0)
    np.testing.assert_allclose(out_e[0], np.full(d, 1.0), rtol=1e-15)
    np.testing.assert_allclose(out_e[K + 2], np.tile([1.0, -1.0], d // 2), rtol=1e-15)
    out_q = oracle.fuse_project(bits(c), bits(e), bits(q), sel(2), eps=0.0)
    for s in range(S):                                            # only q varies across the positions of a block
        np.testing.assert_allclose(out_q[s * K + 0], np.full(d, 1.0), rtol=1e-15)
        np.testing.assert_allclose(out_q[s * K + 1], np.tile([0.0, np.sqrt(2.0)], d // 2), rtol=1e-15)
        np.testing.assert_allclose(out_q[s * K + 2], np.tile([np.sqrt(2.0), 0.0], d // 2), rtol=1e-15)
    # eps enters under the root: constant input a gives a / sqrt(a^2 + eps)
    out_eps = oracle.fuse_project(bits(c), bits(e), bits(q), sel(0), eps=5.0)
    np.testing.assert_allclose(out_eps[K], np.full(d, -2.0 / 3.0), rtol=1e-15)
    # a gain multiplies after the normalisation
    g = np.arange(1, d + 1, dtype=np.float32)
    out_g = oracle.fuse_project(bits(c), bits(e), bits(q), sel(0), gain_c=g, eps=0.0)
    np.testing.assert_allclose(out_g[K], -g.astype(np.float64), rtol=1e-15)


def test_fuse_project_invariants():
    rng = W.rng_for(52)
    S, K, d, d_out = 4, 4, 64, 24
    c, e, q, w = _fuse_inputs(rng, S, K, d, d_out)
    base = oracle.fuse_project(c, e, q, w, eps=0.0)
    # with eps = 0 each input is normalised on its own: rescaling one by a power of two changes nothing
    c4 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(c) * 4.0)
    e8 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(e) * 0.125)
    np.testing.assert_allclose(oracle.fuse_project(c4, e8, q, w, eps=0.0), base, rtol=1e-12, atol=1e-12)
    # the difference between two positions of a block comes from the queries alone: the same for every start
    diffs = base.reshape(S, K, d_out) - base.reshape(S, K, d_out)[:, :1]
    np.testing.assert_allclose(diffs, np.broadcast_to(diffs[0], diffs.shape), rtol=1e-10, atol=1e-10)
    assert np.abs(diffs[0, 1:]).max() > 0.1
    # linear in W
    w2 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(w) * 2.0)
    np.testing.assert_allclose(oracle.fuse_project(c, e, q, w2, eps=0.0), 2.0 * base, rtol=1e-12, atol=1e-12)
