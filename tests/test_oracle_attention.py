"""Pins of the CPU oracle's tree attention and ancestor sets to things other than itself:
the paper's printed mask example (Fig. 4), a library attention routine on special cases, and
closed forms."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import workloads as W


def _read_fig4(golden_dir):
    rows, pos, parent = [], None, None
    for line in open(os.path.join(golden_dir, "fig4_mask.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("pos"):
            pos = [int(t) for t in line.split()[1:]]
        elif line.startswith("parent"):
            parent = [int(t) for t in line.split()[1:]]
        else:
            rows.append([int(c) for c in line])
    return np.asarray(rows), np.asarray(pos), np.asarray(parent, np.int32)


def test_fig4_ancestors_and_position_ids(golden_dir):
    """Fig. 4: the ancestor sets reproduce rows 2..9 of the printed matrix, depth gives the
    printed position ids."""
    mask, pos, parent = _read_fig4(golden_dir)
    P = 2
    anc, depth, rc = oracle.tree_ancestors(parent)
    assert rc == 0
    for i in range(len(parent)):
        row = [1] * P + [(int(anc[i, a // 32]) >> (a % 32)) & 1 for a in range(len(parent))]
        assert row == list(mask[P + i]), f"node {i}"
    assert list(P + depth) == list(pos[P:])


def test_fig4_visibility_read_out_through_attention(golden_dir):
    """Fig. 4 through the attention itself: with q = 0 every visible key has the same score, so
    with one-hot value rows out = indicator(visible)/|visible| and lse = ln|visible|."""
    mask, _pos, parent = _read_fig4(golden_dir)
    P, n, D = 2, len(parent), 16
    k = W.normal_bf16(W.rng_for(1), (1, P + n, 1, D))
    v = np.zeros((1, P + n, 1, D), np.float32)
    for j in range(P + n):
        v[0, j, 0, j] = 1.0
    q = np.zeros((n, 1, D), np.float32)
    out, lse, st = oracle.tree_attention(
        n_q_heads=1, n_kv_heads=1, head_dim=D, k=k, v=W.f32_to_bf16_bits(v), kv_capacity=P + n,
        prefix_len=[P], node_offsets=[0, n], parent=parent, q=W.f32_to_bf16_bits(q))
    assert st[0] == 0
    for i in range(n):
        vis = mask[P + i].astype(np.float64)
        np.testing.assert_allclose(out[i, 0, :P + n], vis / vis.sum(), atol=1e-15)
        np.testing.assert_allclose(lse[i, 0], np.log(vis.sum()), atol=1e-15)


def _sdpa_last_rows(q_rows, k_rows, v_rows, scale):
    """Library routine: causal attention where query t sees keys 0..len-n+t (fp64, CPU)."""
    n, L = q_rows.shape[0], k_rows.shape[0]
    mask = torch.zeros(n, L, dtype=torch.bool)
    for t in range(n):
        mask[t, : L - n + t + 1] = True
    o = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q_rows)[None, None], torch.from_numpy(k_rows)[None, None],
        torch.from_numpy(v_rows)[None, None], attn_mask=mask[None, None], scale=scale)
    return o[0, 0].numpy()


def _f64(bits):
    return W.bf16_bits_to_f32(bits).astype(np.float64)


@pytest.mark.parametrize("paged", [False, True])
def test_path_linearisation_equals_causal_attention(paged):
    """A node's tree attention equals plain causal attention's last row over the sequence
    [prefix, root-to-node path] (library SDPA), for every node, head and a GQA group of 2;
    K/V heads are distinct so a wrong head mapping fails."""
    rng = W.rng_for(11)
    pars = [W.random_tree(rng, 13, 5), W.random_tree(rng, 7, 3)]
    case = W.make_attn_case(rng, parents=pars, prefix_lens=[37, 5], n_q_heads=4, n_kv_heads=2,
                            head_dim=32, page_size=16 if paged else 0)
    out, lse, st = oracle.tree_attention(**case.oracle_kwargs())
    assert not st.any()
    scale = 1.0 / np.sqrt(32)
    for b, par in enumerate(pars):
        P = int(case.prefix_len[b])
        for i in range(len(par)):
            path = [i]
            while par[path[-1]] >= 0:
                path.append(int(par[path[-1]]))
            pos = list(range(P)) + [P + a for a in path[::-1]]
            for h in range(4):
                g = h // 2
                kk = np.stack([_f64(case.k[W.kv_slot(case, b, p)][g]) for p in pos])
                vv = np.stack([_f64(case.v[W.kv_slot(case, b, p)][g]) for p in pos])
                row = int(case.node_offsets[b]) + i
                qq = _f64(case.q[row, h])[None]
                ref = _sdpa_last_rows(qq, kk, vv, scale)[0]
                np.testing.assert_allclose(out[row, h], ref, rtol=1e-12, atol=1e-13)
                s = scale * (kk @ qq[0])
                ref_lse = torch.logsumexp(torch.from_numpy(s), 0).item()
                assert abs(lse[row, h] - ref_lse) < 1e-12


def test_chain_tree_is_ordinary_causal_decode():
    """parent[i] = i-1: the tree attention is causal attention over P+N tokens, last N rows."""
    rng = W.rng_for(12)
    n, P, D = 9, 21, 64
    case = W.make_attn_case(rng, parents=[W.chain_tree(n)], prefix_lens=[P], n_q_heads=2,
                            n_kv_heads=2, head_dim=D, scale=0.2)
    out, _lse, st = oracle.tree_attention(**case.oracle_kwargs())
    assert st[0] == 0
    for h in range(2):
        ref = _sdpa_last_rows(_f64(case.q[:, h]), _f64(case.k[0, :P + n, h]),
                              _f64(case.v[0, :P + n, h]), 0.2)
        np.testing.assert_allclose(out[:, h], ref, rtol=1e-12, atol=1e-13)


def test_closed_forms():
    rng = W.rng_for(13)
    D = 32
    # (a) P = 0, a node under the prefix sees only itself: out = v, lse = scale * q.k
    case = W.make_attn_case(rng, parents=[np.asarray([-1, -1, 0], np.int32)], prefix_lens=[0],
                            n_q_heads=1, n_kv_heads=1, head_dim=D)
    out, lse, _ = oracle.tree_attention(**case.oracle_kwargs())
    for i in (0, 1):
        np.testing.assert_allclose(out[i, 0], _f64(case.v[0, i, 0]), atol=1e-15)
        s = (_f64(case.q[i, 0]) * _f64(case.k[0, i, 0])).sum() / np.sqrt(D)
        assert abs(lse[i, 0] - s) < 1e-13
    # (b) all value rows equal: out = that row whatever the scores
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 6, 3)], prefix_lens=[9],
                            n_q_heads=2, n_kv_heads=1, head_dim=D)
    case.v[:] = case.v[0, 0, 0]
    out, _, _ = oracle.tree_attention(**case.oracle_kwargs())
    np.testing.assert_allclose(out, np.broadcast_to(_f64(case.v[0, 0, 0]), out.shape), atol=1e-14)
    # (c) permuting prefix positions (K and V together) changes nothing
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 6, 3)], prefix_lens=[17],
                            n_q_heads=2, n_kv_heads=1, head_dim=D)
    o1, l1, _ = oracle.tree_attention(**case.oracle_kwargs())
    perm = rng.permutation(17)
    case.k[0, :17] = case.k[0, perm]
    case.v[0, :17] = case.v[0, perm]
    o2, l2, _ = oracle.tree_attention(**case.oracle_kwargs())
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(l1, l2, rtol=1e-13)


def test_off_path_keys_do_not_leak_and_on_path_keys_count():
    """Mask sensitivity: an off-path tree key built to dominate must not move the output; the
    same key on the path must dominate it."""
    rng = W.rng_for(14)
    D = 32
    par = np.asarray([-1, 0, 0, 1, 2], np.int32)        # node 3 under 1, node 4 under 2
    case = W.make_attn_case(rng, parents=[par], prefix_lens=[40], n_q_heads=1, n_kv_heads=1,
                            head_dim=D)
    P = 40
    qf = W.bf16_bits_to_f32(case.q[3, 0])
    big = (8.0 * np.sqrt(D) * qf / np.linalg.norm(qf)).astype(np.float32)
    base, _, _ = oracle.tree_attention(**case.oracle_kwargs())
    case.k[0, P + 2, 0] = W.f32_to_bf16_bits(big)        # node 2 is off node 3's path
    case.v[0, P + 2, 0] = W.f32_to_bf16_bits(np.full(D, 100.0, np.float32))
    out, _, _ = oracle.tree_attention(**case.oracle_kwargs())
    np.testing.assert_allclose(out[3], base[3], atol=1e-14)       # unchanged
    qf4 = W.bf16_bits_to_f32(case.q[4, 0])                        # node 4 has node 2 on its path
    case.k[0, P + 2, 0] = W.f32_to_bf16_bits(
        (8.0 * np.sqrt(D) * qf4 / np.linalg.norm(qf4)).astype(np.float32))
    out, _, _ = oracle.tree_attention(**case.oracle_kwargs())
    np.testing.assert_allclose(out[3], base[3], atol=1e-14)
    assert np.abs(out[4, 0] - 100.0).max() < 1.0                  # the planted key dominates


def test_selection_and_q_node_begin_match_full_run():
    rng = W.rng_for(15)
    par, n_cached = W.drafter_block_tree(4)
    full = W.make_attn_case(rng, parents=[par], prefix_lens=[33], n_q_heads=4, n_kv_heads=2,
                            head_dim=32)
    o_full, l_full, _ = oracle.tree_attention(**full.oracle_kwargs())
    kw = full.oracle_kwargs()
    kw.update(q=full.q[n_cached:], q_node_begin=[n_cached], q_offsets=[0, len(par) - n_cached])
    o_q, l_q, _ = oracle.tree_attention(**kw)
    np.testing.assert_array_equal(o_q, o_full[n_cached:])
    sel = np.asarray([[0, 5, 3], [0, 43, 0]], np.int32)
    o_s, l_s, _ = oracle.tree_attention(**full.oracle_kwargs(), sel=sel)
    np.testing.assert_array_equal(o_s[0], o_full[5, 3])
    np.testing.assert_array_equal(o_s[1], o_full[43, 0])
    assert l_s[1] == l_full[43, 0]


def test_invalid_tree_and_bounds_are_flagged():
    rng = W.rng_for(16)
    case = W.make_attn_case(rng, parents=[np.asarray([-1, 0, 1], np.int32),
                                          np.asarray([-1, 0], np.int32)], prefix_lens=[4, 4],
                            n_q_heads=1, n_kv_heads=1, head_dim=16)
    case.parent[2] = 2                      # parent not earlier than the child
    out, lse, st = oracle.tree_attention(**case.oracle_kwargs())
    assert list(st) == [4, 0]
    assert not out[:3].any() and out[3:].any()
    case.parent[2] = 1
    kw = case.oracle_kwargs()
    kw["kv_capacity"] = case.kv_capacity    # unchanged layout, but claim a longer prefix
    kw["prefix_len"] = np.asarray([4, 40], np.int32)
    _o, _l, st = oracle.tree_attention(**kw)
    assert list(st) == [0, 5]
