"""GPU parity of sb_tree_attention / sb_tree_ancestors against the CPU oracle, through the C ABI.

Tolerance (stated by the benchmark spec): bf16 outputs |err| <= 1e-2 + 1e-2*|ref|, fp32 log-sum-exp
|err| <= 1e-5*max(1,|ref|).  Status words and ancestor masks are compared exactly."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import device_inputs as dev
from paper_2605_07243_b200 import workloads as W

from gpu_helpers import (assert_attention_close, check_attention, gpu_attention, require_gpu,
                         sample_rows)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _read_fig4(golden_dir):
    rows, parent = [], None
    for line in open(os.path.join(golden_dir, "fig4_mask.txt")):
        line = line.strip()
        if not line or line.startswith("#") or line.startswith("pos"):
            continue
        if line.startswith("parent"):
            parent = np.asarray([int(t) for t in line.split()[1:]], np.int32)
        else:
            rows.append([int(c) for c in line])
    return np.asarray(rows), parent


def test_fig4_ancestors_on_gpu(golden_dir):
    mask, parent = _read_fig4(golden_dir)
    P, n = 2, len(parent)
    anc, depth, status = sb.sb_tree_ancestors(dev.i32_tensor([0, n]), dev.i32_tensor(parent), n)
    anc = anc.cpu().numpy().view(np.uint32)
    ref_anc, ref_depth, _ = oracle.tree_ancestors(parent)
    np.testing.assert_array_equal(anc, ref_anc)
    np.testing.assert_array_equal(depth.cpu().numpy(), ref_depth)
    assert status.cpu().numpy()[0] == 0
    for i in range(n):
        row = [1] * P + [(int(anc[i, a // 32]) >> (a % 32)) & 1 for a in range(n)]
        assert row == list(mask[P + i])


def test_fig4_visibility_read_out_on_gpu(golden_dir):
    """q = 0 and one-hot value rows: the output reveals the visible set of every row."""
    mask, parent = _read_fig4(golden_dir)
    P, n, D = 2, len(parent), 64
    case = W.make_attn_case(W.rng_for(1), parents=[parent], prefix_lens=[P], n_q_heads=2,
                            n_kv_heads=1, head_dim=D)
    v = np.zeros((1, P + n, 1, D), np.float32)
    for j in range(P + n):
        v[0, j, 0, j] = 1.0
    case.v = W.f32_to_bf16_bits(v)
    case.q[:] = 0
    out, lse, st = gpu_attention(case)
    assert st[0] == 0
    for i in range(n):
        vis = mask[P + i].astype(np.float64)
        for h in range(2):
            np.testing.assert_allclose(out[i, h, :P + n], vis / vis.sum(), atol=2e-3)
            assert abs(lse[i, h] - np.log(vis.sum())) < 1e-5
            assert np.all(out[i, h, :P + n][vis == 0] == 0.0)


def test_ancestors_batch_with_invalid_tree():
    rng = W.rng_for(40)
    pars = [W.random_tree(rng, 128, 12), np.asarray([-1, 0, 2, 1], np.int32), W.chain_tree(1),
            W.random_tree(rng, 77, 30)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in pars])])
    anc, depth, status = sb.sb_tree_ancestors(dev.i32_tensor(offs), dev.i32_tensor(np.concatenate(pars)), 128)
    anc, depth, status = anc.cpu().numpy().view(np.uint32), depth.cpu().numpy(), status.cpu().numpy()
    assert list(status) == [0, 4, 0, 0]
    for b, p in enumerate(pars):
        ra, rd, rc = oracle.tree_ancestors(p)
        np.testing.assert_array_equal(anc[offs[b]:offs[b + 1]], ra)
        np.testing.assert_array_equal(depth[offs[b]:offs[b + 1]], rd)


def test_config1_tiny():
    attn, _ = W.config1_tiny()
    check_attention(attn, "config 1")
    check_attention(attn, "config 1, 2 splits", num_splits=2)


@pytest.mark.parametrize("num_splits", [0, 1, 2, 3, 7])
@pytest.mark.parametrize("prefix", [300, 0, 1, 63, 64, 129])
def test_block_tree_small_prefixes_and_splits(prefix, num_splits):
    """8B-shaped heads, 60-node K=4 block tree; prefixes that put the tree slots at the start of,
    across and at the end of 64-key tiles; every chunking merges to the same result."""
    par = W.config2_tree()
    case = W.config2_verify_layer(layer=prefix, prefix=prefix, par=par)
    check_attention(case, f"P={prefix} splits={num_splits}", num_splits=num_splits)


def test_config2_full_layer():
    check_attention(W.config2_verify_layer(), "config 2 layer 0")


def test_config3_drafter_blocks_with_cached_nodes():
    attn, _ = W.config3_drafter()
    check_attention(attn, "config 3")
    check_attention(attn, "config 3, 5 splits", num_splits=5)


@pytest.mark.parametrize("page_size", [64, 16, 256])
def test_ragged_paged_batch_small(page_size):
    rng = W.rng_for(41)
    sizes = [1, 33, 96, 64, 17]
    parents = [W.random_tree(rng, n, 10) for n in sizes]
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[0, 700, 130, 64, 511], n_q_heads=32,
                            n_kv_heads=8, head_dim=128, page_size=page_size)
    check_attention(case, f"ragged paged {page_size}")
    check_attention(case, f"ragged paged {page_size}, 4 splits", num_splits=4)


def test_group_of_eight_and_128_nodes():
    """Long-context config's head shape (64 query / 8 KV heads) and a full 128-node tree."""
    rng = W.rng_for(42)
    parents = [W.random_tree(rng, 128, 12), W.random_tree(rng, 128, 12)]
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[1000, 37], n_q_heads=64, n_kv_heads=8,
                            head_dim=128, page_size=64)
    check_attention(case, "G=8 N=128", num_splits=3)


@pytest.mark.parametrize("heads", [(4, 4), (6, 2), (8, 1)])
def test_head_dim_64_and_other_group_sizes(heads):
    rng = W.rng_for(43)
    hq, hkv = heads
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 50, 8), W.chain_tree(9)],
                            prefix_lens=[200, 77], n_q_heads=hq, n_kv_heads=hkv, head_dim=64, scale=0.3)
    check_attention(case, f"D=64 heads={heads}")
    check_attention(case, f"D=64 heads={heads} split", num_splits=3)


def test_peaky_softmax():
    rng = W.rng_for(44)
    case = W.make_attn_case(rng, parents=[W.block_tree(rng, 60)], prefix_lens=[500], n_q_heads=32,
                            n_kv_heads=8, head_dim=128, q_std=4.0)
    check_attention(case, "q x4", num_splits=4)


@pytest.mark.parametrize("prefix", [40, 64, 100, 127])
def test_mask_leaks_are_order_one(prefix):
    """Adversarial: every tree key is made dominant for every query row (k = c*q/|q| is not
    possible for all rows at once, so tree keys get a huge common component that all queries
    share) and carries V = +-100 with random signs.  A single leaked off-path key, or a missing
    on-path key, moves the output by O(10), far outside the tolerance, whose absolute term is
    scaled by the value magnitude 100 here (1.0 instead of 1e-2)."""
    rng = W.rng_for(45)
    par = W.random_tree(rng, 64, 6)
    case = W.make_attn_case(rng, parents=[par], prefix_lens=[prefix], n_q_heads=8, n_kv_heads=2,
                            head_dim=128)
    q = W.bf16_bits_to_f32(case.q)
    q[:, :, 0] = 4.0                                   # shared component of every query
    case.q = W.f32_to_bf16_bits(q)
    k = W.bf16_bits_to_f32(case.k)
    v = W.bf16_bits_to_f32(case.v)
    k[0, prefix:, :, 0] = 16.0                          # tree keys: score + 64*scale ~ +5.7
    v[0, prefix:prefix + len(par)] = 100.0 * rng.choice([-1.0, 1.0], size=(len(par), 2, 128))
    case.k, case.v = W.f32_to_bf16_bits(k), W.f32_to_bf16_bits(v)
    for splits in (1, 2, 5):
        check_attention(case, f"adversarial P={prefix} splits={splits}", num_splits=splits,
                        value_scale=100.0)


def _dominant_tree_keys(rng, parents, prefix_lens, **shape):
    """Every tree key overwhelms the whole prefix for every query row (one shared query component of 8
    against a key component of 32: a score of +22 before the usual N(0,1) part, against at most 33k prefix
    keys of weight ~1) and carries V = +-100 with random signs: an output row is then a short weighted
    average of +-100 over the row's own ancestors.  One leaked off-path key, or one missing on-path key,
    moves it by O(10); the tolerance's absolute term is 1.0 here (value_scale = 100)."""
    case = W.make_attn_case(rng, parents=parents, prefix_lens=prefix_lens, **shape)
    q = W.bf16_bits_to_f32(case.q)
    q[:, :, 0] = 8.0
    case.q = W.f32_to_bf16_bits(q)
    k, v = W.bf16_bits_to_f32(case.k), W.bf16_bits_to_f32(case.v)
    for b, par in enumerate(parents):
        for i in range(len(par)):
            slot = W.kv_slot(case, b, int(prefix_lens[b]) + i)
            k[slot][:, 0] = 32.0
            v[slot] = 100.0 * rng.choice([-1.0, 1.0], size=v[slot].shape)
    case.k, case.v = W.f32_to_bf16_bits(k), W.f32_to_bf16_bits(v)
    return case


@pytest.mark.parametrize("page_size", [0, 16, 64])
@pytest.mark.parametrize("two_tiles", [False, True])
def test_mask_leaks_are_order_one_across_tiles_pages_and_blocks(page_size, two_tiles, request):
    """The tree's cache slots straddle a page boundary, a 128-key block boundary and a chunk boundary,
    on the one-tile and on the two-tile kernel (whose window-application code is its own), contiguous
    and paged.  G = 8 with up to 60 nodes gives one to four row tiles per KV head."""
    if two_tiles:
        request.getfixturevalue("test_build").setenv("SB_ATTN_TWO_TILES", "1")
    rng = W.rng_for(4600 + page_size + (1 if two_tiles else 0))
    shape = dict(n_q_heads=16, n_kv_heads=2, head_dim=128, page_size=page_size)
    for prefix in ([13, 120], [60, 250], [127, 1000], [128, 5]):
        parents = [W.random_tree(rng, 60, 7), W.block_tree(rng, 40)]
        case = _dominant_tree_keys(rng, parents, prefix, **shape)
        for splits in (1, 2, 3):
            check_attention(case, f"dominant tree keys, page {page_size}, two tiles {two_tiles}, P={prefix}, splits={splits}",
                            num_splits=splits, value_scale=100.0)


@pytest.mark.parametrize("prefix", [8000, 33000])
@pytest.mark.parametrize("two_tiles", [False, True])
def test_mask_leaks_are_order_one_behind_a_long_prefix(prefix, two_tiles, request):
    """Long prefixes are where the float tolerance alone cannot see a leaked key (one key among 33k moves
    the output by 3e-5): here the tree sits in the last of 16 chunks behind 8k / 33k prefix keys, with the
    128-node trees and eight heads per KV head of the long-context configuration, paged as it is."""
    if two_tiles:
        request.getfixturevalue("test_build").setenv("SB_ATTN_TWO_TILES", "1")
    rng = W.rng_for(4700 + prefix // 1000 + (1 if two_tiles else 0))
    case = _dominant_tree_keys(rng, [W.random_tree(rng, 128, 12)], [prefix], n_q_heads=16, n_kv_heads=2,
                               head_dim=128, page_size=64)
    for splits in (16, 0):
        check_attention(case, f"dominant tree keys behind P={prefix}, two tiles {two_tiles}, splits={splits}",
                        num_splits=splits, value_scale=100.0)


def test_chunk_without_visible_key():
    """P = 0 and many chunks: most chunks hold no key a given row may see."""
    rng = W.rng_for(46)
    par = W.random_tree(rng, 128, 3)
    case = W.make_attn_case(rng, parents=[par], prefix_lens=[0], n_q_heads=4, n_kv_heads=4, head_dim=64)
    check_attention(case, "P=0, 2 chunks", num_splits=2)


@pytest.mark.parametrize("impl", ["mma", "tc"])
def test_both_tensor_core_paths(test_build, impl):
    """The tcgen05 kernel is the library's only backend; the test build also holds an mma.sync kernel,
    an independent implementation that must agree with the oracle on the same cases."""
    test_build.setenv("SB_ATTN_IMPL", impl)
    attn, _ = W.config1_tiny()
    check_attention(attn, f"{impl}: config 1", num_splits=2)
    check_attention(W.config2_verify_layer(prefix=777), f"{impl}: 8B-shaped, P=777")
    check_attention(W.config2_verify_layer(prefix=777), f"{impl}: 8B-shaped, P=777, 16 chunks", num_splits=16)
    rng = W.rng_for(50)
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 128, 12), W.chain_tree(5), W.random_tree(rng, 40, 6)],
                            prefix_lens=[333, 0, 2000], n_q_heads=64, n_kv_heads=8, head_dim=128, page_size=64)
    check_attention(case, f"{impl}: ragged paged G=8", num_splits=5)


def test_simple_kernel_path(test_build):
    test_build.setenv("SB_ATTN_IMPL", "simple")
    attn, _ = W.config1_tiny()
    check_attention(attn, "simple kernel, config 1")
    rng = W.rng_for(47)
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 20, 5), W.chain_tree(3)], prefix_lens=[90, 5],
                            n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16)
    check_attention(case, "simple kernel, paged")


def test_errors_are_flagged_per_sequence_and_zero_filled():
    rng = W.rng_for(48)
    pars = [np.asarray([-1, 0, 1, 1], np.int32), W.random_tree(rng, 10, 4), W.chain_tree(5)]
    case = W.make_attn_case(rng, parents=pars, prefix_lens=[30, 100, 64], n_q_heads=8, n_kv_heads=2,
                            head_dim=128)
    case.parent[2] = 3                                  # sequence 0: parent after child
    case.prefix_len = np.asarray([30, 100, 64 + 1000], np.int32)   # sequence 2: beyond capacity
    for splits in (1, 3):
        tb, q, kw = dev.attention_args(case)
        tb.max_kv_len = 2000
        out, lse, status = sb.sb_tree_attention(tb, q, num_splits=splits, **kw)
        torch.cuda.synchronize()
        out, lse, status = out.float().cpu().numpy(), lse.cpu().numpy(), status.cpu().numpy()
        assert list(status) == [4, 0, 5]
        ref_out, ref_lse, ref_status = oracle.tree_attention(**case.oracle_kwargs())
        assert list(ref_status) == [4, 0, 5]
        assert not out[:4].any() and not out[14:].any() and not lse[:4].any()
        assert_attention_close(out[4:14], lse[4:14], ref_out[4:14], ref_lse[4:14], "valid sequence")


def test_bad_page_id_is_reported_without_fault():
    rng = W.rng_for(49)
    case = W.make_attn_case(rng, parents=[W.chain_tree(4), W.chain_tree(4)], prefix_lens=[100, 100],
                            n_q_heads=4, n_kv_heads=1, head_dim=64, page_size=16)
    good = gpu_attention(case)
    case.page_table[1, 2] = case.num_pages + 5
    out, lse, status = gpu_attention(case)
    assert list(status) == [0, 5]
    # the contract for a page id outside the pool: reported, every read redirected into the pool (so the
    # call cannot fault), that sequence's rows unspecified -- and the other sequence's rows untouched
    np.testing.assert_array_equal(out[:4], good[0][:4])
    np.testing.assert_array_equal(lse[:4], good[1][:4])
    assert np.isfinite(out[4:]).all()


def test_host_argument_errors():
    big = W.config2_verify_layer(prefix=1500)
    tb, q, kw = dev.attention_args(big)
    assert sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], 8) == 0      # one cluster: no scratch
    assert sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], 16) > 0      # two clusters: partials
    with pytest.raises(sb.SbError) as e:
        sb.sb_tree_attention(tb, q, num_splits=16, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 3
    attn, _ = W.config1_tiny()
    tb, q, kw = dev.attention_args(attn)
    tb.head_dim = 48
    with pytest.raises(sb.SbError) as e:
        sb.sb_tree_attention(tb, q)
    assert e.value.code == 2
    tb.head_dim = 64
    tb.n_kv_heads = 3
    with pytest.raises(sb.SbError) as e:
        sb.sb_tree_attention(tb, q)
    assert e.value.code == 1


# ---- full-size configurations, every output element (the oracle takes seconds on them) ----------

def test_config4_batched_full_size():
    """All 16 ragged paged sequences, every row: the launch configuration the bench times (the library's
    own choice of chunks) and an explicit split."""
    attn, _ = W.config4_batched(with_logits=False)
    ref = oracle.tree_attention(**attn.oracle_kwargs())
    for what, kw in (("config 4, library's chunks", {}), ("config 4, 3 chunks", dict(num_splits=3))):
        out, lse, status = gpu_attention(attn, **kw)
        np.testing.assert_array_equal(status, ref[2])
        assert_attention_close(out, lse, ref[0], ref[1], what)


def test_config5_long_context_full_size():
    """All four 32k-token sequences, every row, with the 16 chunks the configuration prescribes and with
    the chunk count the library chooses (one chunk: 257 key blocks per CTA)."""
    attn, _ = W.config5_long(with_logits=False)
    ref = oracle.tree_attention(**attn.oracle_kwargs())
    for what, kw in (("config 5, 16 chunks", dict(num_splits=16)), ("config 5, library's chunks", {})):
        out, lse, status = gpu_attention(attn, **kw)
        np.testing.assert_array_equal(status, ref[2])
        assert_attention_close(out, lse, ref[0], ref[1], what)


def test_two_tiles_per_cta_kernel(test_build):
    """The throughput kernel (two row tiles per CTA, P written over S in tensor memory, chunks merged
    from fp32 partials), forced on shapes that would otherwise take the one-tile kernel."""
    test_build.setenv("SB_ATTN_TWO_TILES", "1")
    check_attention(W.config2_verify_layer(prefix=777), "two tiles: 8B-shaped, P=777, 1 chunk", num_splits=1)
    check_attention(W.config2_verify_layer(prefix=777), "two tiles: 8B-shaped, P=777, 3 chunks", num_splits=3)
    check_attention(W.config2_verify_layer(prefix=2048), "two tiles: 8B-shaped, library's chunks")
    check_attention(W.config2_verify_layer(prefix=300), "two tiles: more chunks than blocks", num_splits=16)
    rng = W.rng_for(70)
    # ragged trees: 1, 2, 3 and 8 row tiles in one batch (a last pair with a single tile), paged, G = 8
    parents = [W.random_tree(rng, 128, 12), W.chain_tree(5), W.random_tree(rng, 40, 6), W.random_tree(rng, 24, 4)]
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[333, 0, 2000, 129], n_q_heads=64, n_kv_heads=8,
                            head_dim=128, page_size=64)
    check_attention(case, "two tiles: ragged paged G=8", num_splits=5)
    check_attention(case, "two tiles: ragged paged G=8, one chunk", num_splits=1)
    # G = 3 does not divide 128: Q tiles are gathered; head_dim 64; page 16
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 100, 9), W.random_tree(rng, 50, 5)], prefix_lens=[700, 64],
                            n_q_heads=6, n_kv_heads=2, head_dim=64, page_size=16, scale=0.2)
    check_attention(case, "two tiles: G=3, D=64, page 16", num_splits=2)
    # no prefix at all: every block is masked
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 128, 10)], prefix_lens=[0], n_q_heads=8, n_kv_heads=2,
                            head_dim=128)
    check_attention(case, "two tiles: P=0")


def test_two_tiles_per_cta_long_chunks(test_build):
    """Many blocks per CTA (the steady state of the two-tile pipeline), peaky scores so that the
    reference maximum moves and accumulators are rescaled."""
    test_build.setenv("SB_ATTN_TWO_TILES", "1")
    rng = W.rng_for(71)
    case = W.make_attn_case(rng, parents=[W.random_tree(rng, 96, 10), W.random_tree(rng, 33, 10)],
                            prefix_lens=[6000, 3001], n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=64, q_std=4.0)
    check_attention(case, "two tiles: long chunks, peaky", num_splits=1)
    check_attention(case, "two tiles: long chunks, peaky, 2 chunks", num_splits=2)


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_against_oracle(seed, request):
    """Seeded random shapes: batch, head layout, head_dim, page size, tree sizes, prefix lengths, query
    range, chunk count and kernel variant all drawn at random; element-wise parity on every one."""
    rng = W.rng_for(9000 + seed)
    B = int(rng.integers(1, 5))
    hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 3, 4, 8]))
    D = int(rng.choice([64, 128]))
    page = int(rng.choice([0, 0, 16, 64, 128, 256]))
    parents, prefix, qbegin = [], [], []
    for _ in range(B):
        n = int(rng.integers(1, 129))
        parents.append(W.random_tree(rng, n, int(rng.integers(1, 14))))
        prefix.append(int(rng.choice([0, 1, 15, 16, 17, 127, 128, 129, int(rng.integers(0, 3000))])))
        qbegin.append(int(rng.integers(0, n)) if rng.random() < 0.3 else 0)
    use_qbegin = any(qbegin)
    case = W.make_attn_case(rng, parents=parents, prefix_lens=prefix, n_q_heads=hkv * G, n_kv_heads=hkv, head_dim=D,
                            page_size=page, q_node_begin=qbegin if use_qbegin else None,
                            q_std=float(rng.choice([1.0, 1.0, 4.0])), capacity_pad=int(rng.integers(0, 40)))
    splits = int(rng.choice([0, 0, 1, 2, 3, 5, 8, 16]))
    if rng.random() < 0.4:   # the forced two-tile kernel lives in the test build; the rest runs on the library proper
        request.getfixturevalue("test_build").setenv("SB_ATTN_TWO_TILES", "1")
    check_attention(case, f"random shape {seed}: B={B} Hkv={hkv} G={G} D={D} page={page} splits={splits}",
                    num_splits=splits)


def test_settled_flags_give_the_same_bits():
    """The flags only move the fetch of the sequence lengths, and of key blocks inside the prefix, ahead of
    the dependency wait: same results, on the compile-time variant (config 2, with chunks that lie inside
    the prefix, straddle its end, or hold tree rows only), a paged ragged batch and a drafter call with
    cached nodes."""
    rng = W.rng_for(431)
    ragged = W.make_attn_case(rng, parents=[W.random_tree(rng, 40, 6), W.chain_tree(7), W.random_tree(rng, 90, 9)],
                              prefix_lens=[700, 33, 0], n_q_heads=16, n_kv_heads=4, head_dim=128, page_size=64)
    for case in (W.config2_verify_layer(prefix=600), W.config2_verify_layer(prefix=130), W.config2_verify_layer(),
                 ragged, W.config3_drafter(prefix=900)[0]):
        plain = gpu_attention(case)
        for flags in (dict(index_arrays_settled=True), dict(index_arrays_settled=True, prefix_rows_settled=True),
                      dict(prefix_rows_settled=True)):
            flagged = gpu_attention(case, **flags)
            for a, b in zip(plain, flagged):
                np.testing.assert_array_equal(a, b)
        assert (plain[2] == 0).all()


@pytest.mark.parametrize("page_size", [0, 64])
@pytest.mark.parametrize("num_splits", [0, 1, 3])
def test_empty_sequences_inside_a_batch(page_size, num_splits, monkeypatch):
    """Sequences without any tree node (and one whose query range is empty) between ordinary ones: they own no
    output row, report status 0 and leave their neighbours' rows alone -- on the one-tile and the two-tile kernel."""
    rng = W.rng_for(77 + page_size + num_splits)
    none = np.zeros(0, np.int32)
    parents = [none, W.random_tree(rng, 70, 6), none, W.chain_tree(9), W.random_tree(rng, 20, 4), none]
    case = W.make_attn_case(rng, parents=parents, prefix_lens=[40, 300, 0, 0, 129, 5], n_q_heads=8, n_kv_heads=2,
                            head_dim=128, page_size=page_size, q_node_begin=[0, 0, 0, 3, 20, 0])
    check_attention(case, f"empty sequences, page {page_size}, splits {num_splits}", num_splits=num_splits)
    with sb.build_variant("test"):
        monkeypatch.setenv("SB_ATTN_TWO_TILES", "1")
        check_attention(case, f"empty sequences, page {page_size}, splits {num_splits}, two tiles", num_splits=num_splits)
