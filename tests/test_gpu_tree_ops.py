"""GPU parity of sb_verify_accept, sb_tree_expand and sb_kv_compact against the CPU oracle, through
the C ABI.  Everything here is integer / byte work: the comparison is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import device_inputs as dev
from paper_2605_07243_b200 import workloads as W

from gpu_helpers import require_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


# ---- verify / accept ----------------------------------------------------------------------------------

def _logits_tensor(logits):
    if logits.dtype == np.uint16:
        return dev.bf16_tensor(logits)
    return torch.from_numpy(logits).cuda()


def _gpu_accept(case, vocab=None):
    r = sb.sb_verify_accept(_logits_tensor(case.logits), dev.i32_tensor(case.node_offsets),
                            dev.i32_tensor(case.parent), dev.i32_tensor(case.tok), case.max_depth,
                            vocab=vocab)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in r.items()}


def _check_accept(case, vocab=None):
    got = _gpu_accept(case, vocab)
    ref = oracle.verify_accept(case.logits, case.node_offsets, case.parent, case.tok, case.max_depth,
                               vocab=vocab)
    for key in ("status", "amax", "accept_len", "path_nodes", "out_tokens", "bonus"):
        np.testing.assert_array_equal(got[key], ref[key], err_msg=key)
    return got


def test_accept_config1_tiny():
    _, ver = W.config1_tiny()
    got = _check_accept(ver)
    np.testing.assert_array_equal(got["accept_len"], ver.planted_len)
    np.testing.assert_array_equal(got["bonus"], ver.planted_bonus)


@pytest.mark.parametrize("accept_len", range(0, 9))
def test_accept_config2_bf16_full_vocab(accept_len):
    ver = W.config2_logits(accept_len=accept_len)
    got = _check_accept(ver)
    assert got["accept_len"][0] == ver.planted_len[0]
    assert got["bonus"][0] == ver.planted_bonus[0]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("vocab", [1, 7, 1000, 4099, 32000])
def test_accept_ragged_batches_vocab_sizes(dtype, vocab):
    rng = W.rng_for(60 + vocab)
    parents = [W.random_tree(rng, int(n), 10) for n in (1, 96, 33, 128, 2)]
    if vocab < 200:
        # a tiny vocabulary cannot hold distinct sibling tokens: draw tokens directly, many ties
        total = sum(len(p) for p in parents)
        x = np.round(rng.standard_normal((total, vocab), dtype=np.float32))
        case = W.VerifyCase(W.f32_to_bf16_bits(x) if dtype == "bf16" else x,
                            rng.integers(0, vocab, total).astype(np.int32),
                            np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32),
                            np.concatenate(parents), 10, None, None, None)
    else:
        case = W.make_verify_case(rng, parents=parents, vocab=vocab, dtype=dtype, max_depth=10)
    _check_accept(case)


def test_accept_row_stride_padding_nan_inf_and_ties():
    rng = W.rng_for(61)
    parents = [W.random_tree(rng, 20, 5)]
    x = np.round(rng.standard_normal((20, 1003 + 5), dtype=np.float32) * 2)   # coarse: many ties
    x[:, 1003:] = 1e9                       # padding beyond vocab must be ignored
    x[3, :1003] = np.nan                     # all-NaN row -> id 0
    x[4, 10] = np.nan
    x[5, 77] = np.inf
    x[6, :1003] = -np.inf
    x[7, :1003] = 0.0
    x[7, 5] = -0.0
    case = W.VerifyCase(x, rng.integers(0, 1003, 20).astype(np.int32), np.asarray([0, 20], np.int32),
                        parents[0], 5, None, None, None)
    got = _check_accept(case, vocab=1003)
    assert got["amax"][3] == 0 and got["amax"][5] == 77 and got["amax"][6] == 0 and got["amax"][7] == 0


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_accept_degenerate_rows_large_vocab(dtype):
    """Rows with nothing above -inf, over a vocabulary that spans many chunks and many vectors per thread."""
    rng = W.rng_for(63)
    vocab = 128256
    parents = [W.chain_tree(8)]
    x = np.round(rng.standard_normal((8, vocab), dtype=np.float32) * 2)
    x[1, :] = -np.inf                        # -> id 0
    x[2, :] = np.nan                         # NaN reads as -inf -> id 0
    x[3, :] = -np.inf
    x[3, vocab - 1] = -7.0                   # the only finite value sits in the last chunk's tail
    x[4, :] = -np.inf
    x[4, 40000:40003] = np.nan               # still nothing above -inf -> id 0
    x[5, :] = 3.0                            # all equal -> id 0
    x[6, :] = -np.inf
    x[6, 70001] = -np.inf
    x[6, 70002] = -1e30
    logits = W.f32_to_bf16_bits(x) if dtype == "bf16" else x
    case = W.VerifyCase(logits, rng.integers(0, vocab, 8).astype(np.int32), np.asarray([0, 8], np.int32),
                        parents[0], 8, None, None, None)
    got = _check_accept(case)
    np.testing.assert_array_equal(got["amax"][1:7], [0, 0, vocab - 1, 0, 0, 70002])


def test_accept_depth_cut_duplicates_and_invalid_trees():
    rng = W.rng_for(62)
    # duplicate sibling tokens and a tiny alphabet -> many equally long accepted paths
    parents = [W.random_tree(rng, 40, 12), np.asarray([-1, -1, 0], np.int32), W.chain_tree(30),
               np.asarray([-1, 0, 3, 1], np.int32)]
    total = sum(len(p) for p in parents)
    x = np.zeros((total, 3), np.float32)
    choice = rng.integers(0, 3, total)
    x[np.arange(total), choice] = 1.0
    case = W.VerifyCase(x, rng.integers(0, 3, total).astype(np.int32),
                        np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32),
                        np.concatenate(parents), 4, None, None, None)
    case.tok[43:73] = 1                      # the chain accepts everything: cut at max_depth
    x[43:73] = [0, 1, 0]
    got = _check_accept(case)
    assert list(got["status"]) == [0, 4, 0, 4]
    assert got["accept_len"][2] == 4


def test_accept_config4_and_5_full_size():
    _, ver4 = W.config4_batched()
    got = _check_accept(ver4)
    np.testing.assert_array_equal(got["accept_len"], ver4.planted_len)
    _, ver5 = W.config5_long()
    got = _check_accept(ver5)
    np.testing.assert_array_equal(got["accept_len"], ver5.planted_len)
    np.testing.assert_array_equal(got["bonus"], ver5.planted_bonus)


# ---- expansion -------------------------------------------------------------------------------------------

def _gpu_expand(case, vocab=None):
    budget = case.node_budget
    n0 = 0 if case.tree is None else len(case.tree["tok"])
    tree = {k: torch.full((budget,), -1, dtype=torch.int32, device="cuda")
            for k in ("tok", "parent", "depth", "node_row", "node_rank")}
    if case.tree is not None:
        for k in tree:
            tree[k][:n0] = dev.i32_tensor(case.tree[k])
    tree["n_nodes"] = torch.tensor([n0], dtype=torch.int32, device="cuda")
    topk_tok, topk_val, status = sb.sb_tree_expand(
        torch.from_numpy(case.scores).cuda(), case.block_k, torch.from_numpy(case.bucket).cuda(),
        case.bmap, dev.i32_tensor(case.start_parent), budget, tree, vocab=vocab)
    torch.cuda.synchronize()
    out = {k: v.cpu().numpy() for k, v in tree.items()}
    out.update(topk_tok=topk_tok.cpu().numpy(), topk_val=topk_val.cpu().numpy(),
               status=int(status.cpu().numpy()[0]))
    out["n_nodes"] = int(out["n_nodes"][0])
    return out


def _check_expand(case, vocab=None):
    got = _gpu_expand(case, vocab)
    ref = oracle.tree_expand(case.scores, case.block_k, case.bucket, case.bmap, case.start_parent,
                             case.node_budget, tree=case.tree, vocab=vocab)
    assert got["status"] == ref["status"]
    np.testing.assert_array_equal(got["topk_tok"], ref["topk_tok"])
    np.testing.assert_array_equal(got["topk_val"], ref["topk_val"])
    if ref["status"] == 0:
        assert got["n_nodes"] == ref["n_nodes"]
        for k in ("tok", "parent", "depth", "node_row", "node_rank"):
            np.testing.assert_array_equal(got[k], ref[k], err_msg=k)
    return got


def test_expand_config3_full_vocab():
    _, exp = W.config3_drafter()
    got = _check_expand(exp)
    assert got["n_nodes"] > 12


@pytest.mark.parametrize("bmap", [[2, 4, 10, 0], [2, 4, 6, 4], [16, 16, 16, 16], [0, 0, 0, 0]])
@pytest.mark.parametrize("vocab", [5, 1000, 32000])
def test_expand_printed_maps_and_vocab_sizes(bmap, vocab):
    rng = W.rng_for(70 + vocab)
    case = W.make_expand_case(rng, n_starts=3, block_k=4, vocab=vocab, bmap=bmap, node_budget=60,
                              existing_parent=W.random_tree(rng, 5, 3), tie_rows=6)
    _check_expand(case)


def test_expand_ties_nan_inf_padding_and_budget():
    rng = W.rng_for(71)
    case = W.make_expand_case(rng, n_starts=2, block_k=4, vocab=2000 + 3, bmap=[3, 5, 10, 2],
                              node_budget=17)
    s = case.scores
    s[:, 2000:] = 1e9                        # padding columns beyond vocab
    s[0, :2000] = 1.0                        # all equal: ids 0..15 in order
    s[1, :2000] = np.nan                     # all NaN: treated as -inf, ids 0..15
    s[2, ::2] = np.inf
    s[3, :2000] = np.round(s[3, :2000])      # heavy ties
    s[4, :1990] = -np.inf                    # only 10 finite values
    got = _check_expand(case, vocab=2000)
    assert list(got["topk_tok"][0]) == list(range(16))
    assert got["n_nodes"] == 17


def test_expand_device_argument_errors():
    rng = W.rng_for(72)
    case = W.make_expand_case(rng, n_starts=1, block_k=4, vocab=100, bmap=[2, 4, 10, 0], node_budget=20)
    case.bucket[2] = 9
    assert _check_expand(case)["status"] == 1
    case.bucket[2] = 1
    case.start_parent[0] = 3                 # no such node
    assert _check_expand(case)["status"] == 1


# ---- compaction ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("page_size", [0, 64, 16])
def test_kv_compact_matches_oracle(page_size):
    rng = W.rng_for(80 + page_size)
    parents = [W.random_tree(rng, 60, 8), W.chain_tree(40), W.random_tree(rng, 9, 4), W.chain_tree(3)]
    L = 3
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[250, 64, 1, 0], n_q_heads=32, n_kv_heads=8,
                            head_dim=128, page_size=page_size)
    layer_elems = case.k.size
    k_all = rng.integers(0, 65536, (L,) + case.k.shape).astype(np.uint16)
    v_all = rng.integers(0, 65536, (L,) + case.v.shape).astype(np.uint16)
    max_depth = 32
    paths = np.full((4, max_depth + 1), -1, np.int32)
    alen = np.zeros(4, np.int32)
    # sequence 0: a real root-to-node path; 1: the full chain (identity moves only, 32 deep);
    # 2: root only; 3: an invalid path (not increasing)
    end = int(np.argmax(W.tree_depths(parents[0])))
    p0 = [end]
    while parents[0][p0[-1]] >= 0:
        p0.append(int(parents[0][p0[-1]]))
    p0 = p0[::-1]
    paths[0, :len(p0)] = p0
    alen[0] = len(p0) - 1
    paths[1, :33] = np.arange(33)
    alen[1] = 32
    paths[2, 0] = 0
    paths[3, :3] = [0, 2, 1]
    alen[3] = 2
    tb = dev.tree_batch(case, k=dev.bf16_tensor(k_all), v=dev.bf16_tensor(v_all))
    new_len, status = sb.sb_kv_compact(tb, L, layer_elems, dev.i32_tensor(paths), dev.i32_tensor(alen),
                                       max_depth)
    torch.cuda.synchronize()
    kw = dict(n_kv_heads=8, head_dim=128, n_layers=L, layer_stride_elems=layer_elems, page_size=page_size,
              max_pages=case.max_pages, num_pages=case.num_pages, kv_capacity=case.kv_capacity,
              page_table=case.page_table, prefix_len=case.prefix_len, node_offsets=case.node_offsets,
              path_nodes=paths, accept_len=alen, max_depth=max_depth)
    ref_k, ref_len, ref_st = oracle.kv_compact(cache=k_all.reshape(-1), **kw)
    ref_v, _, _ = oracle.kv_compact(cache=v_all.reshape(-1), **kw)
    np.testing.assert_array_equal(status.cpu().numpy(), ref_st)
    np.testing.assert_array_equal(new_len.cpu().numpy(), ref_len)
    assert list(ref_st) == [0, 0, 0, 4]
    got_k = tb.k_cache.view(torch.int16).cpu().numpy().view(np.uint16).reshape(k_all.shape)
    got_v = tb.v_cache.view(torch.int16).cpu().numpy().view(np.uint16).reshape(v_all.shape)
    ref_k, ref_v = ref_k.reshape(k_all.shape), ref_v.reshape(v_all.shape)
    # compare the live range [0, new_len) of every sequence, plus everything outside the trees
    for b in range(4):
        for pos in range(int(ref_len[b])):
            sl = W.kv_slot(case, b, pos)
            np.testing.assert_array_equal(got_k[(slice(None),) + sl], ref_k[(slice(None),) + sl])
            np.testing.assert_array_equal(got_v[(slice(None),) + sl], ref_v[(slice(None),) + sl])
    # the in-place result equals the out-of-place gather everywhere in this construction:
    # a slot beyond new_len is never written by either
    np.testing.assert_array_equal(got_k, ref_k)
    np.testing.assert_array_equal(got_v, ref_v)


def test_accept_then_compact_chain_on_device():
    """sb_verify_accept's device outputs feed sb_kv_compact without a host round trip."""
    par = W.config2_tree()
    ver = W.config2_logits(accept_len=5, vocab=4096, par=par)
    case = W.config2_verify_layer(prefix=200, par=par)
    r = sb.sb_verify_accept(dev.bf16_tensor(ver.logits), dev.i32_tensor(ver.node_offsets),
                            dev.i32_tensor(ver.parent), dev.i32_tensor(ver.tok), 8)
    tb = dev.tree_batch(case)
    new_len, status = sb.sb_kv_compact(tb, 1, 0, r["path_nodes"], r["accept_len"], 8)
    torch.cuda.synchronize()
    assert int(new_len[0]) == 200 + 5 + 1 and int(status[0]) == 0
    path = r["path_nodes"].cpu().numpy()[0, :6]
    assert list(path) == ver.planted_path[0]
    got_k = tb.k_cache.view(torch.int16).cpu().numpy().view(np.uint16)
    for j, node in enumerate(path):
        np.testing.assert_array_equal(got_k[0, 200 + j], case.k[0, 200 + node])


@pytest.mark.parametrize("which", [4, 5])
def test_accept_then_compact_on_the_batched_and_long_configurations(which):
    """Configurations 4 (16 ragged paged sequences, accept lengths drawn with the paper's per-position
    acceptance rates) and 5 (four 32k-token sequences) at full size: acceptance on the planted logits, then
    the in-place compaction of two layers of the real paged caches, chained on the device; paths, tokens,
    new lengths and every live cache row against the oracle."""
    attn, ver = W.config4_batched() if which == 4 else W.config5_long()
    L = 2
    layer_elems = int(attn.k.size)
    rng = W.rng_for(8800 + which)
    k_all = np.stack([attn.k, attn.v])                         # two "layers" with distinct contents
    v_all = np.stack([attn.v, attn.k])
    logits = dev.bf16_tensor(ver.logits) if ver.logits.dtype == np.uint16 else torch.from_numpy(ver.logits).cuda()
    r = sb.sb_verify_accept(logits, dev.i32_tensor(ver.node_offsets), dev.i32_tensor(ver.parent),
                            dev.i32_tensor(ver.tok), ver.max_depth)
    tb = dev.tree_batch(attn, k=dev.bf16_tensor(k_all), v=dev.bf16_tensor(v_all))
    new_len, status = sb.sb_kv_compact(tb, L, layer_elems, r["path_nodes"], r["accept_len"], ver.max_depth)
    torch.cuda.synchronize()
    ref = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
    for key in ("amax", "accept_len", "path_nodes", "out_tokens", "bonus", "status"):
        np.testing.assert_array_equal(r[key].cpu().numpy(), ref[key], err_msg=key)
    np.testing.assert_array_equal(ref["accept_len"], ver.planted_len)
    kw = dict(n_kv_heads=attn.n_kv_heads, head_dim=attn.head_dim, n_layers=L, layer_stride_elems=layer_elems,
              page_size=attn.page_size, max_pages=attn.max_pages, num_pages=attn.num_pages, kv_capacity=attn.kv_capacity,
              page_table=attn.page_table, prefix_len=attn.prefix_len, node_offsets=attn.node_offsets,
              path_nodes=ref["path_nodes"], accept_len=ref["accept_len"], max_depth=ver.max_depth)
    ref_k, ref_len, ref_st = oracle.kv_compact(cache=k_all.reshape(-1), **kw)
    ref_v, _, _ = oracle.kv_compact(cache=v_all.reshape(-1), **kw)
    np.testing.assert_array_equal(status.cpu().numpy(), ref_st)
    np.testing.assert_array_equal(new_len.cpu().numpy(), ref_len)
    np.testing.assert_array_equal(ref_len, attn.prefix_len + ver.planted_len + 1)
    got_k = tb.k_cache.view(torch.int16).cpu().numpy().view(np.uint16).reshape(k_all.shape)
    got_v = tb.v_cache.view(torch.int16).cpu().numpy().view(np.uint16).reshape(v_all.shape)
    ref_k, ref_v = ref_k.reshape(k_all.shape), ref_v.reshape(v_all.shape)
    # pages belong to one sequence each, slots past new_len are written by neither side: whole caches compare
    np.testing.assert_array_equal(got_k, ref_k)
    np.testing.assert_array_equal(got_v, ref_v)
    for b in range(attn.batch):                                # and the committed rows are where they belong
        for j, node in enumerate(ref["path_nodes"][b, :ref["accept_len"][b] + 1]):
            dst = W.kv_slot(attn, b, int(attn.prefix_len[b]) + j)
            src = W.kv_slot(attn, b, int(attn.prefix_len[b]) + int(node))
            np.testing.assert_array_equal(got_k[(0,) + dst], attn.k[src])
            np.testing.assert_array_equal(got_v[(0,) + dst], attn.v[src])


# ---- rank-head distribution summary -------------------------------------------------------------------

# fp32 sums over rows of up to 128256 terms: |err| <= 2e-5 * max(1, |ref|)
FEAT_TOL = 2e-5


def _check_features(scores, vocab=None):
    got = sb.sb_rank_features(torch.from_numpy(np.ascontiguousarray(scores)).cuda(), vocab=vocab)
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    ref = oracle.rank_features(scores, vocab=vocab)
    inf = np.isinf(ref)
    np.testing.assert_array_equal(got[inf], ref[inf])
    err = np.abs(got[~inf] - ref[~inf]) / np.maximum(1.0, np.abs(ref[~inf]))
    assert err.max() <= FEAT_TOL, f"feature error {err.max():.2e}"
    return got


def test_rank_features_config3_full_vocab():
    _, exp = W.config3_drafter()
    got = _check_features(exp.scores)
    assert (np.diff(got[:, :10], axis=1) <= 0).all()          # log-probs are listed in descending order


@pytest.mark.parametrize("vocab", [3, 17, 1000, 4099, 32000])
def test_rank_features_vocab_sizes_ties_nan_inf(vocab):
    rng = W.rng_for(90 + vocab)
    x = (rng.standard_normal((7, vocab + 5), dtype=np.float32) * 3).astype(np.float32)
    x[:, vocab:] = 1e9                      # padding beyond vocab
    x[1, :vocab] = np.round(x[1, :vocab])    # ties among the leaders
    x[2, :vocab:3] = np.nan
    x[3, :vocab] = -np.inf                   # no finite score: reported as uniform
    x[4, 2:vocab] = -np.inf                  # two finite scores only
    x[5, :vocab] = 4.0                       # exactly uniform
    x[6, 1] = 60.0                           # one token owns the distribution
    _check_features(x, vocab=vocab)


# ---- verifier-derived update signal (Sec. 3.4; Alg. 2 line 2) -----------------------------------------------

SIGNAL_TOL = 2e-5      # |r - r_ref| <= tol * max(r_ref, 1e-3) and |s - s_ref| <= tol: fp32 sums over the row


def _check_signal(scores, node_offsets, child_row, path_nodes, accept_len, bonus, max_depth, signal0, vocab=None):
    sig = torch.from_numpy(np.asarray(signal0, np.float32)).cuda()
    got = sb.sb_verifier_signal(torch.from_numpy(np.ascontiguousarray(scores)).cuda(), dev.i32_tensor(node_offsets),
                                dev.i32_tensor(child_row), dev.i32_tensor(path_nodes), dev.i32_tensor(accept_len),
                                dev.i32_tensor(bonus), max_depth, sig, vocab=vocab)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in got.items()}
    ref = oracle.verifier_signal(scores, node_offsets, child_row, path_nodes, accept_len, bonus, max_depth,
                                 signal=np.asarray(signal0, np.float32), vocab=vocab)
    np.testing.assert_array_equal(got["status"], ref["status"])
    none = ref["r_prob"] < 0
    np.testing.assert_array_equal(got["r_prob"][none], -1.0)
    err_r = np.abs(got["r_prob"][~none] - ref["r_prob"][~none]) / np.maximum(ref["r_prob"][~none], 1e-3)
    assert err_r.size == 0 or err_r.max() <= SIGNAL_TOL, f"r error {err_r.max():.2e}"
    assert np.abs(got["signal"] - ref["signal"]).max() <= SIGNAL_TOL
    return got, ref


def test_verifier_signal_after_accept_config2_and_config3_scores():
    """The signal chained on the device after sb_verify_accept, over full-vocabulary drafter rows."""
    par = W.config2_tree()
    ver = W.config2_logits(par=par, accept_len=3)
    _, exp = W.config3_drafter()                       # fp32 [32][128256] drafter scores
    rng = W.rng_for(95)
    child_row = rng.integers(-1, exp.scores.shape[0], len(par)).astype(np.int32)
    acc = sb.sb_verify_accept(_logits_tensor(ver.logits), dev.i32_tensor(ver.node_offsets), dev.i32_tensor(ver.parent),
                              dev.i32_tensor(ver.tok), ver.max_depth)
    best = int(acc["path_nodes"].cpu().numpy()[0, int(acc["accept_len"].cpu().numpy()[0])])
    child_row[best] = 7                                  # the row that predicted the rejected position
    sig = torch.full((1,), 0.25, dtype=torch.float32, device="cuda")
    got = sb.sb_verifier_signal(torch.from_numpy(exp.scores).cuda(), dev.i32_tensor(ver.node_offsets),
                                dev.i32_tensor(child_row), acc["path_nodes"], acc["accept_len"], acc["bonus"],
                                ver.max_depth, sig)
    torch.cuda.synchronize()
    ref_acc = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
    ref = oracle.verifier_signal(exp.scores, ver.node_offsets, child_row, ref_acc["path_nodes"], ref_acc["accept_len"],
                                 ref_acc["bonus"], ver.max_depth, signal=[0.25])
    assert int(got["status"].cpu()[0]) == 0 and ref["status"][0] == 0
    r, r_ref = float(got["r_prob"].cpu()[0]), ref["r_prob"][0]
    assert abs(r - r_ref) <= SIGNAL_TOL * max(r_ref, 1e-3)
    assert abs(float(got["signal"].cpu()[0]) - ref["signal"][0]) <= SIGNAL_TOL


@pytest.mark.parametrize("vocab", [1, 5, 1000, 4099, 32000, 128256])
def test_verifier_signal_vocab_sizes_batch_and_degenerate_rows(vocab):
    rng = W.rng_for(96 + vocab)
    R, B, n, max_depth = 9, 11, 6, 5
    x = (rng.standard_normal((R, vocab + 3), dtype=np.float32) * 3).astype(np.float32)
    x[:, vocab:] = 1e9                       # padding beyond vocab must be ignored
    x[1, :vocab:3] = np.nan
    x[2, :vocab] = -np.inf                   # no finite score: flat
    x[3, :vocab] = 2.0                       # exactly flat
    x[4, :vocab] = -np.inf
    x[4, vocab // 2] = 1.0                   # one finite score
    x[5, vocab - 1] = 70.0                   # one token owns the row, in the last CTA's tail
    node_offsets = np.arange(B + 1, dtype=np.int32) * n
    child_row = rng.integers(0, R, B * n).astype(np.int32)
    accept_len = rng.integers(0, max_depth + 1, B).astype(np.int32)
    path = rng.integers(0, n, (B, max_depth + 1)).astype(np.int32)
    bonus = rng.integers(0, vocab, B).astype(np.int32)
    for b in range(min(B, R)):               # sequence b reads row b, so every special row is used
        child_row[b * n + path[b, accept_len[b]]] = b
    bonus[4] = vocab // 2
    bonus[5] = vocab - 1
    bonus[6] = vocab + 2                     # outside the drafter's vocabulary: r = 0
    child_row[7 * n + path[7, accept_len[7]]] = -1      # nothing drafted there
    child_row[9 * n + path[9, accept_len[9]]] = R       # row out of range
    accept_len[10] = max_depth + 1                      # accept length out of range
    got, ref = _check_signal(x, node_offsets, child_row, path, accept_len, bonus, max_depth,
                             rng.random(B).astype(np.float32), vocab=vocab)
    assert list(got["status"][[9, 10]]) == [5, 5] and got["r_prob"][7] == -1.0
    if vocab > 1:
        assert got["r_prob"][6] == 0.0 and abs(got["r_prob"][5] - 1.0) < 1e-6


def test_verifier_signal_unaligned_rows_and_host_errors():
    rng = W.rng_for(97)
    x = (rng.standard_normal((4, 1001), dtype=np.float32)).astype(np.float32)   # odd stride: rows 1..3 unaligned
    node_offsets = np.asarray([0, 3, 6], np.int32)
    child_row = np.asarray([1, 2, 3, 3, 2, 1], np.int32)
    path = np.asarray([[0, 1, 2], [2, 1, 0]], np.int32)
    accept_len = np.asarray([2, 1], np.int32)
    _check_signal(x, node_offsets, child_row, path, accept_len, np.asarray([5, 999], np.int32), 2, [0.0, 1.5],
                  vocab=999)
    t = torch.from_numpy(x).cuda()
    sig = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(sb.SbError):
        sb.sb_verifier_signal(t, dev.i32_tensor(node_offsets), dev.i32_tensor(child_row), dev.i32_tensor(path),
                              dev.i32_tensor(accept_len), dev.i32_tensor([1, 1]), 2, sig, vocab=2000)
    with pytest.raises(sb.SbError):
        sb.sb_verifier_signal(t, dev.i32_tensor(node_offsets), dev.i32_tensor(child_row), dev.i32_tensor(path),
                              dev.i32_tensor(accept_len), dev.i32_tensor([1, 1]), 99, sig)


# ---- stochastic verification (temperature > 0) ---------------------------------------------------------------

def _robust_uniforms(rng, case_args, temperature, max_depth, total, batch, vocab=None, eps=2e-3, tries=40):
    """Acceptance uniforms whose every decision in the oracle has a relative margin of eps: the walk is
    the same with all of them scaled by 1 - eps and 1 + eps (acceptance is monotone in u, so the three
    runs follow the same path and every comparison on it holds with that margin).  The GPU decides
    in fp32 (about 1e-5 relative on a ratio of sums over the vocabulary)."""
    u_b = rng.random(batch).astype(np.float32) * np.float32(0.98) + np.float32(0.01)
    for _ in range(tries):
        u_a = rng.random(total).astype(np.float32) * np.float32(0.98) + np.float32(0.01)
        runs = [oracle.verify_sample(*case_args, temperature, (u_a * np.float32(s)).astype(np.float32), u_b,
                                     max_depth, vocab=vocab) for s in (1.0, 1.0 - eps, 1.0 + eps)]
        if all(np.array_equal(runs[0][k], r[k]) for r in runs[1:] for k in ("status", "accept_len", "path_nodes")):
            return u_a, u_b, runs[0]
    raise AssertionError("no robust uniforms found")


def _check_sample(rng, logits, scores, node_offsets, parent, tok, child_row, temperature, max_depth, vocab=None,
                  delta=1e-3):
    """The walk (status, accept_len, path, accepted tokens) must equal the oracle's.  The bonus token is
    an inverse-CDF draw whose cell can be far narrower than fp32 sums over the vocabulary resolve, so it
    is checked as a draw: it must lie between the oracle's draws for u_bonus (1 - delta) and (1 + delta)
    (the draw is monotone in u_bonus)."""
    total = len(parent)
    batch = len(node_offsets) - 1
    args = (logits, scores, node_offsets, parent, tok, child_row)
    u_a, u_b, ref = _robust_uniforms(rng, args, temperature, max_depth, total, batch, vocab=vocab)
    got = sb.sb_verify_sample(_logits_tensor(logits), torch.from_numpy(np.ascontiguousarray(scores)).cuda(),
                              dev.i32_tensor(node_offsets), dev.i32_tensor(parent), dev.i32_tensor(tok),
                              dev.i32_tensor(child_row), temperature, torch.from_numpy(u_a).cuda(),
                              torch.from_numpy(u_b).cuda(), max_depth, vocab=vocab)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in got.items()}
    for key in ("status", "accept_len", "path_nodes"):
        np.testing.assert_array_equal(got[key], ref[key], err_msg=key)
    lo = oracle.verify_sample(*args, temperature, u_a, (u_b * np.float32(1 - delta)).astype(np.float32), max_depth,
                              vocab=vocab)["bonus"]
    hi = oracle.verify_sample(*args, temperature, u_a, (u_b * np.float32(1 + delta)).astype(np.float32), max_depth,
                              vocab=vocab)["bonus"]
    for b in range(batch):
        a = int(ref["accept_len"][b])
        if ref["status"][b] != 0:
            np.testing.assert_array_equal(got["out_tokens"][b], ref["out_tokens"][b])
            assert got["bonus"][b] == ref["bonus"][b] == -1
            continue
        np.testing.assert_array_equal(got["out_tokens"][b, :a], ref["out_tokens"][b, :a])
        assert lo[b] <= got["bonus"][b] <= hi[b], (b, lo[b], got["bonus"][b], hi[b])
        assert got["out_tokens"][b, a] == got["bonus"][b] and (got["out_tokens"][b, a + 1:] == -1).all()
    return ref, got


def _sample_case(rng, parents, vocab, dtype, std=2.0, stride_pad=0):
    """Target logits that favour the drafted tokens (so that walks go deep) and drafter scores that
    favour them too; child_row = the node's own index."""
    n_nodes = [len(p) for p in parents]
    total = sum(n_nodes)
    node_offsets = np.concatenate([[0], np.cumsum(n_nodes)]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    tok = np.zeros(total, np.int32)
    logits = (rng.standard_normal((total, vocab + stride_pad), dtype=np.float32) * std).astype(np.float32)
    scores = (rng.standard_normal((total, vocab + stride_pad), dtype=np.float32) * std).astype(np.float32)
    if stride_pad:
        logits[:, vocab:] = 1e9
        scores[:, vocab:] = 1e9
    for b, par in enumerate(parents):
        o = node_offsets[b]
        for a in range(len(par)):
            kids = [c for c in range(len(par)) if par[c] == a]
            toks = rng.choice(vocab, size=len(kids), replace=False) if kids else []
            for c, t in zip(kids, toks):
                tok[o + c] = t
                logits[o + a, t] += 6.0 + rng.random() * 2          # the target likes its children ...
                scores[o + a, t] += 5.0 + rng.random() * 3          # ... and so does the drafter
    child_row = np.arange(total, dtype=np.int32)
    if dtype == "bf16":
        logits = W.f32_to_bf16_bits(logits)
    return logits, scores, node_offsets, parent, tok, child_row


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_verify_sample_matches_oracle_small_vocab(dtype):
    rng = W.rng_for(110)
    parents = [W.random_tree(rng, 40, 7), W.chain_tree(6), np.asarray([-1], np.int32), W.random_tree(rng, 128, 12)]
    case = _sample_case(rng, parents, 1000, dtype, stride_pad=3)
    depths = set()
    exact = 0
    for rep in range(6):
        ref, got = _check_sample(rng, *case, temperature=1.0, max_depth=8, vocab=1000)
        depths.update(int(a) for a in ref["accept_len"])
        exact += int((got["bonus"] == ref["bonus"]).sum())
    assert len(depths) >= 3, depths          # the walks really differ: rejections, residual draws, deep accepts
    assert exact >= 20, exact                # and almost every bonus draw is the oracle's own (24 draws)
    _check_sample(rng, *case, temperature=0.5, max_depth=3, vocab=1000)
    _check_sample(rng, *case, temperature=2.0, max_depth=8, vocab=1000)


def test_verify_sample_full_vocabulary_config2_tree():
    rng = W.rng_for(111)
    par = W.config2_tree()
    case = _sample_case(rng, [par], 128256, "bf16")
    for rep in range(2):
        _check_sample(rng, *case, temperature=1.0, max_depth=8)


def test_verify_sample_errors_and_degenerate_rows():
    rng = W.rng_for(112)
    parents = [W.random_tree(rng, 12, 4), W.random_tree(rng, 9, 3), W.chain_tree(4)]
    logits, scores, node_offsets, parent, tok, child_row = _sample_case(rng, parents, 257, "f32")
    bad_parent = parent.copy()
    bad_parent[node_offsets[1] + 3] = 5                  # parent index not below its child
    child_row2 = child_row.copy()
    child_row2[node_offsets[2]] = -1                     # the chain's root has children but no drafter row
    logits2 = logits.copy()
    logits2[0, :] = np.nan                               # a target row without a finite value: flat
    scores2 = scores.copy()
    scores2[0, :] = -np.inf
    ref, _ = _check_sample(rng, logits2, scores2, node_offsets, bad_parent, tok, child_row2, temperature=1.0, max_depth=6)
    assert list(ref["status"]) == [0, 4, 5]
    t = torch.from_numpy(logits).cuda()
    s = torch.from_numpy(scores).cuda()
    u = torch.zeros(len(parent), dtype=torch.float32, device="cuda")
    ub = torch.zeros(3, dtype=torch.float32, device="cuda")
    with pytest.raises(sb.SbError):
        sb.sb_verify_sample(t, s, dev.i32_tensor(node_offsets), dev.i32_tensor(parent), dev.i32_tensor(tok),
                            dev.i32_tensor(child_row), 0.0, u, ub, 6)
    with pytest.raises(sb.SbError):
        sb.sb_verify_sample(t, s, dev.i32_tensor(node_offsets), dev.i32_tensor(parent), dev.i32_tensor(tok),
                            dev.i32_tensor(child_row), 1.0, u, ub, 6,
                            workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))


# ---- layer-wise shift projection (Sec. 3.1) -----------------------------------------------------------------

def _check_shift(rng, R, d, d_out, K, w_std=0.02):
    h = W.f32_to_bf16_bits(rng.standard_normal((R, d), dtype=np.float32))
    w = W.f32_to_bf16_bits(rng.standard_normal((d_out, 2 * d if K > 0 else d), dtype=np.float32) * np.float32(w_std))
    got, status = sb.sb_shift_project(dev.bf16_tensor(h), dev.bf16_tensor(w), K)
    torch.cuda.synchronize()
    assert int(status.cpu()[0]) == 0
    got = got.float().cpu().numpy().astype(np.float64)
    ref = oracle.shift_project(h, w, K)
    err = np.abs(got - ref)
    tol = 1e-2 + 1e-2 * np.abs(ref)          # bf16 output of an fp32 accumulation
    assert (err <= tol).all(), f"max err {err.max():.3e} at |ref| {np.abs(ref).flat[err.argmax()]:.3e}"
    return got, ref


@pytest.mark.parametrize("R,K", [(32, 4), (4, 4), (60, 4), (128, 8), (17, 1)])
def test_shift_project_8b_shape(R, K):
    """d = d_out = 4096 (the 8B drafter's width): 64 MB of weights streamed once."""
    _check_shift(W.rng_for(120 + R), R, 4096, 4096, K)


@pytest.mark.parametrize("d,d_out", [(64, 128), (192, 384), (1024, 256), (5120, 128)])
def test_shift_project_other_shapes_and_plain_projection(d, d_out):
    rng = W.rng_for(130 + d)
    _check_shift(rng, 24, d, d_out, 4, w_std=0.05)
    _check_shift(rng, 9, d, d_out, 0, w_std=0.05)       # plain projection, n_rows not a multiple of 16


def test_shift_project_pure_shift_and_host_errors():
    rng = W.rng_for(140)
    d = 256
    h = W.f32_to_bf16_bits(rng.standard_normal((12, d), dtype=np.float32))
    eye, zero = np.eye(d, dtype=np.float32), np.zeros((d, d), np.float32)
    got, _ = sb.sb_shift_project(dev.bf16_tensor(h), dev.bf16_tensor(W.f32_to_bf16_bits(np.hstack([zero, eye]))), 4)
    torch.cuda.synchronize()
    prev = np.asarray([r - 1 if r % 4 else r for r in range(12)])
    np.testing.assert_array_equal(got.view(torch.int16).cpu().numpy().view(np.uint16), h[prev])   # bit-exact copy
    ht, wt = dev.bf16_tensor(h), dev.bf16_tensor(W.f32_to_bf16_bits(np.hstack([zero, eye])))
    with pytest.raises(sb.SbError):
        sb.sb_shift_project(ht[:, :100].contiguous(), wt[:, :200].contiguous(), 4)      # d not a multiple of 64
    with pytest.raises(sb.SbError):
        sb.sb_shift_project(torch.cat([ht] * 11), wt, 4)                                 # more than 128 rows
    with pytest.raises(sb.SbError):
        sb.sb_shift_project(ht, wt, 4, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))


@pytest.mark.parametrize("vocab", [2, 3, 40, 300])
def test_verify_sample_tiny_vocabularies(vocab):
    """Vocabularies smaller than the cluster's 256 segments (most warps own nothing)."""
    rng = W.rng_for(150 + vocab)
    parents = [W.random_tree(rng, 10, 4), W.chain_tree(3)]
    n_children = max(np.bincount(np.concatenate([p[p >= 0] for p in parents])).max(), 1)
    if n_children > vocab:                       # siblings carry distinct tokens
        parents = [W.chain_tree(6), W.chain_tree(3)]
    case = _sample_case(rng, parents, vocab, "f32", std=1.0)
    for rep in range(3):
        _check_sample(rng, *case, temperature=1.0, max_depth=6)


def test_shift_project_single_row_and_smallest_shapes():
    rng = W.rng_for(160)
    _check_shift(rng, 1, 64, 128, 1, w_std=0.1)
    _check_shift(rng, 1, 4096, 128, 0)
    _check_shift(rng, 128, 64, 128, 128, w_std=0.1)


# ---- the drafter's fused per-position input (Sec. 3.1, the equation for h^(0)) ------------------------------------

def _check_fuse(rng, S, K, d, d_out, *, gains=True, eps=1e-5, w_std=0.02):
    c = W.f32_to_bf16_bits(rng.standard_normal((S, d), dtype=np.float32) * np.float32(3.0))
    e = W.f32_to_bf16_bits(rng.standard_normal((S, d), dtype=np.float32) * np.float32(0.05))
    q = W.f32_to_bf16_bits(rng.standard_normal((K, d), dtype=np.float32))
    w = W.f32_to_bf16_bits(rng.standard_normal((d_out, 3 * d), dtype=np.float32) * np.float32(w_std))
    g = [rng.uniform(0.5, 1.5, d).astype(np.float32) if gains else None for _ in range(3)]
    gt = [None if x is None else torch.from_numpy(x).cuda() for x in g]
    ct, et, qt, wt = (dev.bf16_tensor(a) for a in (c, e, q, w))
    q_term = torch.full((K, d_out), float("nan"), dtype=torch.float32, device="cuda")
    full, status = sb.sb_fuse_project(ct, et, qt, wt, gain_c=gt[0], gain_e=gt[1], gain_q=gt[2], eps=eps, q_term=q_term)
    torch.cuda.synchronize()
    assert int(status.cpu()[0]) == 0
    ref = oracle.fuse_project(c, e, q, w, *g, eps=eps)
    got = full.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    # The normalised rows are rounded to bf16 before the tensor-core product (relative 2^-9 per element,
    # independent): an absolute error of about 1e-3 of the outputs' root mean square, whatever |ref| is.
    # The absolute term of the bound therefore scales with that root mean square (about 9 sigma).
    scale = max(1.0, float(np.sqrt(np.mean(ref * ref))))
    tol = 1e-2 * scale + 1e-2 * np.abs(ref)
    assert (err <= tol).all(), f"max err/tol {(err / tol).max():.3f}"
    # the cached query term: two thirds of the weights streamed, the same bits out
    assert bool(torch.isfinite(q_term).all())
    again, status2 = sb.sb_fuse_project(ct, et, qt, wt, gain_c=gt[0], gain_e=gt[1], gain_q=gt[2], eps=eps, q_term=q_term,
                                        q_term_valid=True)
    torch.cuda.synchronize()
    assert int(status2.cpu()[0]) == 0
    assert torch.equal(again.view(torch.int16), full.view(torch.int16))
    # the query term itself: W_q norm(q_k), i.e. the oracle with the other two thirds of W zeroed
    wq = W.bf16_bits_to_f32(w).copy()
    wq[:, :2 * d] = 0
    ref_q = oracle.fuse_project(c[:1], e[:1], q, W.f32_to_bf16_bits(wq), *g, eps=eps)
    errq = np.abs(q_term.cpu().numpy().astype(np.float64) - ref_q)
    assert (errq <= 1e-2 * scale + 1e-2 * np.abs(ref_q)).all()
    return got, ref


@pytest.mark.parametrize("S,K", [(8, 4), (1, 4), (16, 4), (3, 8), (128, 1)])
def test_fuse_project_8b_shape(S, K):
    """d = d_out = 4096 (the 8B drafter's width): 96 MB of weights, 64 MB with the query term cached."""
    _check_fuse(W.rng_for(170 + S), S, K, 4096, 4096)


@pytest.mark.parametrize("d,d_out", [(64, 128), (192, 384), (1024, 256)])
def test_fuse_project_other_shapes(d, d_out):
    rng = W.rng_for(180 + d)
    _check_fuse(rng, 5, 4, d, d_out, w_std=0.05)
    _check_fuse(rng, 2, 7, d, d_out, gains=False, eps=0.0, w_std=0.05)   # more positions than starts, no gains


def test_fuse_project_selector_weights_and_host_errors():
    rng = W.rng_for(190)
    S, K, d = 3, 4, 128
    eye, zero = np.eye(d, dtype=np.float32), np.zeros((d, d), np.float32)
    c = W.f32_to_bf16_bits(np.stack([np.tile([3.0, 4.0], d // 2), np.full(d, -2.0), np.full(d, 0.25)]).astype(np.float32))
    e = W.f32_to_bf16_bits(rng.standard_normal((S, d), dtype=np.float32))
    q = W.f32_to_bf16_bits(rng.standard_normal((K, d), dtype=np.float32))
    ct, et, qt = dev.bf16_tensor(c), dev.bf16_tensor(e), dev.bf16_tensor(q)
    wt = dev.bf16_tensor(W.f32_to_bf16_bits(np.hstack([eye, zero, zero])))
    got, _ = sb.sb_fuse_project(ct, et, qt, wt, eps=0.0)
    torch.cuda.synchronize()
    got = got.float().cpu().numpy().reshape(S, K, d)
    want = np.stack([np.tile([3.0, 4.0], d // 2) / np.sqrt(12.5), np.full(d, -1.0), np.full(d, 1.0)])
    for k in range(K):                                   # the prefix broadcast: every position sees the same c
        np.testing.assert_allclose(got[:, k], want, rtol=2.0 ** -8)
    with pytest.raises(sb.SbError):
        sb.sb_fuse_project(ct[:, :100].contiguous(), et[:, :100].contiguous(), qt[:, :100].contiguous(),
                           wt[:, :300].contiguous())                                  # d not a multiple of 64
    with pytest.raises(sb.SbError):
        sb.sb_fuse_project(ct, et, qt, wt, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    with pytest.raises(sb.SbError):
        sb.sb_fuse_project(ct, et, qt, wt, q_term_valid=True)                         # no q_term to read


@pytest.mark.parametrize("n_starts,block_k", [(256, 4), (300, 4), (5, 7), (64, 16), (1, 1)])
def test_expand_many_rows_and_other_block_lengths(n_starts, block_k):
    """Up to 1024 rows one CTA per row finishes the expansion; beyond that a single CTA does
    (256 x 4 = 1024 rows is the last size of the first kind, 300 x 4 the second kind)."""
    rng = W.rng_for(200 + n_starts)
    case = W.make_expand_case(rng, n_starts=n_starts, block_k=block_k, vocab=700, bmap=[2, 3, 4, 0],
                              node_budget=128, existing_parent=W.random_tree(rng, 9, 3), tie_rows=3)
    _check_expand(case)
    roomy = W.make_expand_case(rng, n_starts=n_starts, block_k=block_k, vocab=90, bmap=[1, 2, 3, 1],
                               node_budget=128 if n_starts > 20 else 4096)
    _check_expand(roomy)


def test_expand_with_features_in_one_pass():
    """sb_tree_expand_features = sb_tree_expand + sb_rank_features from one scan: same tree, same summaries."""
    for case in (W.config3_drafter()[1],
                 W.make_expand_case(W.rng_for(230), n_starts=5, block_k=3, vocab=777, bmap=[2, 3, 4, 0], node_budget=40,
                                    existing_parent=W.random_tree(W.rng_for(231), 6, 3), tie_rows=2),
                 W.make_expand_case(W.rng_for(232), n_starts=300, block_k=4, vocab=90, bmap=[1, 2, 1, 0], node_budget=4000,
                                    existing_parent=np.concatenate([[-1], np.zeros(299, np.int32)]),
                                    start_parent=np.arange(300, dtype=np.int32))):   # > 1024 rows: one finishing CTA
        R, V = case.scores.shape
        scores = torch.from_numpy(case.scores).cuda()

        def fresh_tree():
            n0 = 0 if case.tree is None else len(case.tree["tok"])
            t = {k: torch.full((case.node_budget,), -1, dtype=torch.int32, device="cuda")
                 for k in ("tok", "parent", "depth", "node_row", "node_rank")}
            if case.tree is not None:
                for k in t:
                    t[k][:n0] = dev.i32_tensor(case.tree[k])
            t["n_nodes"] = torch.tensor([n0], dtype=torch.int32, device="cuda")
            return t

        args = (scores, case.block_k, torch.from_numpy(case.bucket).cuda(), case.bmap, dev.i32_tensor(case.start_parent),
                case.node_budget)
        t_sep, t_fused = fresh_tree(), fresh_tree()
        tok_a, val_a, st_a = sb.sb_tree_expand(*args, t_sep)
        feat_sep = sb.sb_rank_features(scores)
        feat_fused = torch.full((R, 15), float("nan"), dtype=torch.float32, device="cuda")
        child_row = torch.full((case.node_budget,), -1, dtype=torch.int32, device="cuda")
        tok_b, val_b, st_b = sb.sb_tree_expand(*args, t_fused, features=feat_fused, child_row=child_row, row_base=1000)
        torch.cuda.synchronize()
        assert int(st_a.cpu()[0]) == 0 and int(st_b.cpu()[0]) == 0
        assert torch.equal(tok_a, tok_b) and torch.equal(val_a, val_b)
        n_old = 0 if case.tree is None else len(case.tree["tok"])
        n_now = int(t_sep["n_nodes"].cpu()[0])
        for k in t_sep:
            if k == "node_row":    # the fused call numbers the rows from its row_base; the old nodes keep theirs
                assert torch.equal(t_sep[k][:n_old], t_fused[k][:n_old])
                assert torch.equal(t_sep[k][n_old:n_now] + 1000, t_fused[k][n_old:n_now])
                assert torch.equal(t_sep[k][n_now:], t_fused[k][n_now:])
            else:
                assert torch.equal(t_sep[k], t_fused[k]), k
        assert torch.equal(feat_sep.view(torch.int32), feat_fused.view(torch.int32))
        # the row that proposed each node's children: derived from the oracle's tree
        ref_t = oracle.tree_expand(case.scores, case.block_k, case.bucket, case.bmap, case.start_parent, case.node_budget,
                                   tree=case.tree)
        n0 = 0 if case.tree is None else len(case.tree["tok"])
        want_rows = np.full(case.node_budget, -1, np.int32)
        for c in range(n0, ref_t["n_nodes"]):
            if ref_t["parent"][c] >= 0:
                want_rows[ref_t["parent"][c]] = 1000 + ref_t["node_row"][c]
        unique_starts = len(set(int(x) for x in case.start_parent if x >= 0)) == sum(1 for x in case.start_parent if x >= 0)
        assert unique_starts or R == 15                 # only the small random case may let two starts share a node
        if unique_starts:
            np.testing.assert_array_equal(child_row.cpu().numpy(), want_rows)
        ref = oracle.rank_features(case.scores)
        got = feat_fused.cpu().numpy().astype(np.float64)
        fin = np.isfinite(ref)
        assert (np.abs(got[fin] - ref[fin]) <= 2e-5 * np.maximum(1, np.abs(ref[fin]))).all()
        assert (got[~fin] == ref[~fin]).all()


@pytest.mark.parametrize("vocab,dtype,pad", [(131071, "f32", 3), (130000, "bf16", 5), (131072, "f32", 0), (200000, "bf16", 0)])
def test_verify_sample_large_vocabularies_and_unaligned_rows(vocab, dtype, pad):
    """Segments of exactly 512 tokens take the register-resident runs (with 16-byte loads only where the
    rows allow them: odd vocabularies and padded strides fall back to scalar loads inside the run);
    more than 131072 tokens take the scalar passes."""
    rng = W.rng_for(240 + pad + vocab % 97)
    parents = [W.random_tree(rng, 14, 4), W.chain_tree(5)]
    case = _sample_case(rng, parents, vocab, dtype, stride_pad=pad)
    for rep in range(2):
        _check_sample(rng, *case, temperature=1.0, max_depth=5, vocab=vocab)


def test_path_rows_against_the_oracle_and_error_cases():
    """Two sequences (the second with its own first row), every accepted length, then the error cases: a path
    node without a row (the root), a node outside the tree, rows that do not increase, an accepted length
    beyond max_depth."""
    require_gpu()
    # K = 4: block 1 rows 0..3 under the root (row 0 proposes the siblings 1 and 2), block 2 rows 4..7 under node 2
    node_row = np.array([-1, 0, 0, 1, 2, 3, 4, 4, 5], np.int32)
    n, md = len(node_row), 4
    offs = np.array([0, n, 2 * n], np.int32)
    row_begin = np.array([0, 100], np.int32)
    rows_all = np.concatenate([node_row, np.where(node_row >= 0, node_row + 100, -1)]).astype(np.int32)
    paths = {4: [0, 1, 3, 4, 5], 3: [0, 2, 6, 8, -1], 2: [0, 2, 7, -1, -1], 1: [0, 2, -1, -1, -1], 0: [0, -1, -1, -1, -1]}
    dev_args = [torch.from_numpy(x).cuda() for x in (offs, rows_all)]
    rb = torch.from_numpy(row_begin).cuda()

    def both(pn, acc):
        pn, acc = np.array(pn, np.int32), np.array(acc, np.int32)
        ref = oracle.path_rows(offs, rows_all, pn, acc, md, row_begin=row_begin)
        got, st = sb.sb_path_rows(*dev_args, torch.from_numpy(pn).cuda(), torch.from_numpy(acc).cuda(), md, row_begin=rb)
        np.testing.assert_array_equal(got.cpu().numpy(), ref["path_rows"])
        np.testing.assert_array_equal(st.cpu().numpy(), ref["status"])
        return ref

    for a0 in range(5):
        for a1 in range(5):
            assert both([paths[a0], paths[a1]], [a0, a1])["status"].tolist() == [0, 0]
    assert both([paths[2], paths[3]], [2, 3])["path_rows"].tolist() == [[0, 1, 5, -1, -1], [0, 1, 5, 6, -1]]
    for path, a in (([0, 0, -1, -1, -1], 1),      # the root has no row
                    ([0, 1, 9, -1, -1], 2),       # node 9 does not exist
                    ([0, 3, 1, -1, -1], 2),       # rows 1 then 0
                    ([0, 1, 3, 4, 5], 5)):        # longer than max_depth
        ref = both([paths[4], path], [4, a])
        assert ref["status"].tolist() == [0, 4] and ref["path_rows"][1].tolist() == [0, -1, -1, -1, -1]   # SB_ERR_INVALID_TREE


def test_accept_and_compact_with_empty_sequences_in_the_batch():
    """A sequence without nodes has no root: acceptance reports an invalid tree for it (accept_len 0, -1 elsewhere)
    and compaction leaves its cache and length alone, while the neighbours are processed as usual."""
    require_gpu()
    rng = W.rng_for(78)
    none = np.zeros(0, np.int32)
    parents = [W.random_tree(rng, 12, 4), none, W.chain_tree(6), none]
    total = sum(len(p) for p in parents)
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    logits = rng.standard_normal((total, 97), dtype=np.float32)
    tok = rng.integers(0, 97, total).astype(np.int32)
    par = np.concatenate(parents).astype(np.int32)
    for c in range(13, 18):                               # the chain accepts its first three tokens
        if c - 12 <= 3:
            logits[c - 1, tok[c]] = 50.0
    case = W.VerifyCase(logits, tok, offs, par, 5, None, None, None)
    got = _check_accept(case)
    assert list(got["status"]) == [0, 4, 0, 4] and got["accept_len"][2] == 3
    attn = W.make_attn_case(rng, parents=parents, prefix_lens=[10, 4, 33, 0], n_q_heads=4, n_kv_heads=2, head_dim=64)
    tb, _q, _kw = dev.attention_args(attn)
    k0 = attn.k.copy()
    new_len, st = sb.sb_kv_compact(tb, 1, int(attn.k.size), torch.from_numpy(got["path_nodes"]).cuda(),
                                   torch.from_numpy(got["accept_len"]).cuda(), 5)
    torch.cuda.synchronize()
    ref_c, ref_len, ref_st = oracle.kv_compact(
        n_kv_heads=2, head_dim=64, cache=k0.reshape(-1), n_layers=1, layer_stride_elems=int(attn.k.size),
        kv_capacity=attn.kv_capacity, prefix_len=attn.prefix_len, node_offsets=offs, path_nodes=got["path_nodes"],
        accept_len=got["accept_len"], max_depth=5)
    np.testing.assert_array_equal(st.cpu().numpy(), ref_st)
    np.testing.assert_array_equal(new_len.cpu().numpy(), ref_len)
    got_k = tb.k_cache.view(torch.int16).cpu().numpy().view(np.uint16).reshape(len(parents), -1)
    row = 2 * 64
    for b in range(len(parents)):
        np.testing.assert_array_equal(got_k[b, :ref_len[b] * row], ref_c.reshape(len(parents), -1)[b, :ref_len[b] * row])
