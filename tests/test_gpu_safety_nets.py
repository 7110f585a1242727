"""Memory-safety evidence and failure paths that need a GPU but never fault one.

This pool has no compute-sanitizer, so two things stand in for it: the CHECKED build of the library
(every index a kernel computes from device data is verified against the extent of what it indexes
before the access; violations are counted and skipped) and canary-padded buffers (every cache, query,
output and workspace buffer sits between guard bands whose pattern must survive the call).  Both run on
small ragged / paged / partial-last-page cases and on the in-place compaction, and every result is still
compared with the oracle.  The bounded device wait is made to run out in a kernel of the TEST build."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import device_inputs as dev
from paper_2605_07243_b200 import workloads as W

from gpu_helpers import assert_attention_close, require_gpu

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side
PATTERN = 0xA5


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


class Guarded:
    """A device buffer between two guard bands.  `view` is the usable part (16-byte aligned)."""

    def __init__(self, src: torch.Tensor = None, *, nbytes=None, dtype=torch.uint8):
        if src is not None:
            nbytes, dtype = src.numel() * src.element_size(), src.dtype
        self.nbytes = nbytes
        pad = (-nbytes) % 16
        self.raw = torch.full((GUARD + nbytes + pad + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.view = self.raw[GUARD:GUARD + nbytes].view(dtype)
        if src is not None:
            self.view.copy_(src.reshape(-1))
            self.view = self.view.view(src.shape)

    def intact(self) -> bool:
        lo, hi = self.raw[:GUARD], self.raw[GUARD + self.nbytes:]
        return bool((lo == PATTERN).all()) and bool((hi == PATTERN).all())


def _guarded_attention(case, num_splits):
    tb, q, kw = dev.attention_args(case)
    g = {"k": Guarded(tb.k_cache), "v": Guarded(tb.v_cache), "q": Guarded(q),
         "out": Guarded(nbytes=q.numel() * 2, dtype=torch.bfloat16),
         "lse": Guarded(nbytes=q.shape[0] * case.n_q_heads * 4, dtype=torch.float32)}
    tb.k_cache, tb.v_cache = g["k"].view, g["v"].view
    need = sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], num_splits)
    g["ws"] = Guarded(nbytes=max(need, 256))
    # the workspace must be 256-byte aligned: GUARD is a multiple of 256 and torch allocations are 512-aligned
    out = g["out"].view.view(q.shape)
    lse = g["lse"].view.view(q.shape[0], case.n_q_heads)
    status = torch.zeros(case.batch, dtype=torch.int32, device="cuda")
    sb.sb_tree_attention(tb, g["q"].view, out, lse, num_splits=num_splits, workspace=g["ws"].view, status=status, **kw)
    torch.cuda.synchronize()
    return tb, g, out, lse, status


def _attention_cases():
    rng = W.rng_for(9100)
    yield "ragged paged 16, partial last page", W.make_attn_case(
        rng, parents=[W.random_tree(rng, 37, 6), W.chain_tree(3), W.random_tree(rng, 90, 9)],
        prefix_lens=[205, 0, 1001], n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16), (0, 3)
    yield "paged 64, G=3 (gathered Q tile)", W.make_attn_case(
        rng, parents=[W.random_tree(rng, 50, 5), W.random_tree(rng, 21, 4)], prefix_lens=[130, 63],
        n_q_heads=6, n_kv_heads=2, head_dim=64, page_size=64), (0, 2)
    yield "contiguous, two row tiles, 12 chunks (partials + merge kernel)", W.make_attn_case(
        rng, parents=[W.block_tree(rng, 60)], prefix_lens=[1500], n_q_heads=16, n_kv_heads=4, head_dim=128), (0, 12)
    # more (sequence, KV head, row tile) units than SMs and up to three row tiles per KV head: the two-tile kernel,
    # alone (library's choice) and with bf16 partials and the merge kernel (2 chunks)
    sizes = [70, 33, 96, 41, 64, 50, 88, 37, 72, 45]
    yield "ragged paged batch on the two-tile kernel", W.make_attn_case(
        rng, parents=[W.random_tree(rng, n, 8) for n in sizes],
        prefix_lens=[130, 517, 64, 300, 0, 255, 129, 700, 31, 402], n_q_heads=32, n_kv_heads=8, head_dim=128,
        page_size=64), (0, 2)
    attn, _ = W.config1_tiny()
    yield "tiny configuration", attn, (0, 2)


@pytest.mark.parametrize("variant", [None, "checked"])
def test_attention_stays_inside_its_buffers(variant):
    """Library proper: canaries only.  Checked build: canaries, zero refused accesses, same parity."""
    import contextlib
    ctx = sb.build_variant(variant) if variant else contextlib.nullcontext()
    with ctx:
        if variant:
            sb.sb_checked_violations()   # clear
        for what, case, splits_list in _attention_cases():
            ref_out, ref_lse, ref_status = oracle.tree_attention(**case.oracle_kwargs())
            for splits in splits_list:
                tb, g, out, lse, status = _guarded_attention(case, splits)
                np.testing.assert_array_equal(status.cpu().numpy(), ref_status)
                assert_attention_close(out.float().cpu().numpy().astype(np.float64),
                                       lse.cpu().numpy().astype(np.float64), ref_out, ref_lse, f"{what}, splits={splits}")
                for name, buf in g.items():
                    assert buf.intact(), f"{what}, splits={splits}: guard band of {name} was written"
        if variant:
            assert sb.sb_checked_violations() == 0


@pytest.mark.parametrize("variant", [None, "checked"])
@pytest.mark.parametrize("page_size", [0, 16])
def test_accept_then_in_place_compaction_stays_inside_its_buffers(variant, page_size):
    import contextlib
    ctx = sb.build_variant(variant) if variant else contextlib.nullcontext()
    rng = W.rng_for(9200 + page_size)
    parents = [W.random_tree(rng, 40, 8), W.chain_tree(9), W.random_tree(rng, 17, 5)]
    attn = W.make_attn_case(rng, parents=parents, prefix_lens=[77, 15, 300], n_q_heads=4, n_kv_heads=2, head_dim=64,
                            page_size=page_size)
    ver = W.make_verify_case(rng, parents=parents, vocab=3001, dtype="bf16")
    n_layers = 3
    with ctx:
        if variant:
            sb.sb_checked_violations()
        tb = dev.tree_batch(attn)
        layer_elems = tb.k_cache.numel()
        k_layers = torch.stack([tb.k_cache.clone().reshape(-1) for _ in range(n_layers)])
        for l in range(n_layers):
            k_layers[l] = k_layers[l].roll(l)          # distinct contents per layer
        v_layers = k_layers.flip(0).contiguous()
        gk, gv = Guarded(k_layers), Guarded(v_layers)
        host_k, host_v = gk.view.cpu(), gv.view.cpu()
        tb.k_cache, tb.v_cache = gk.view[0], gv.view[0]
        assert ver.logits.dtype == np.uint16
        logits = Guarded(torch.from_numpy(ver.logits.view(np.int16)).cuda().view(torch.bfloat16))
        ws = Guarded(nbytes=sb.sb_verify_accept_workspace_bytes(int(ver.node_offsets[-1]), ver.logits.shape[1]))
        r = sb.sb_verify_accept(logits.view, dev.i32_tensor(ver.node_offsets), dev.i32_tensor(ver.parent),
                                dev.i32_tensor(ver.tok), ver.max_depth, workspace=ws.view)
        new_len, cstatus = sb.sb_kv_compact(tb, n_layers, layer_elems, r["path_nodes"], r["accept_len"], ver.max_depth)
        torch.cuda.synchronize()
        ref = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
        for key in ("amax", "accept_len", "path_nodes", "out_tokens", "bonus", "status"):
            np.testing.assert_array_equal(r[key].cpu().numpy(), ref[key], err_msg=key)
        for name, g, host in (("k", gk, host_k), ("v", gv, host_v)):
            ref_cache, ref_len, ref_st = oracle.kv_compact(
                n_kv_heads=attn.n_kv_heads, head_dim=attn.head_dim, cache=host.view(torch.int16).numpy().view(np.uint16).reshape(-1),
                n_layers=n_layers, layer_stride_elems=layer_elems, kv_capacity=attn.kv_capacity, prefix_len=attn.prefix_len,
                node_offsets=attn.node_offsets, path_nodes=ref["path_nodes"], accept_len=ref["accept_len"],
                max_depth=ver.max_depth, page_size=attn.page_size, page_table=attn.page_table, num_pages=attn.num_pages,
                max_pages=attn.max_pages)
            got = g.view.cpu().view(torch.int16).numpy().view(np.uint16).reshape(n_layers, -1)
            refc = ref_cache.reshape(n_layers, -1)
            np.testing.assert_array_equal(new_len.cpu().numpy(), ref_len)
            np.testing.assert_array_equal(cstatus.cpu().numpy(), ref_st)
            # rows below the new length are defined; compare them position by position
            for b in range(attn.batch):
                for pos in range(int(ref_len[b])):
                    i0, i1 = W.kv_slot(attn, b, pos)
                    row = attn.n_kv_heads * attn.head_dim
                    lo = (i0 * attn.k.shape[1] + i1) * row
                    np.testing.assert_array_equal(got[:, lo:lo + row], refc[:, lo:lo + row], err_msg=f"{name} b={b} pos={pos}")
            assert g.intact(), f"guard band of the {name} cache was written"
        assert logits.intact() and ws.intact()
        if variant:
            assert sb.sb_checked_violations() == 0


def test_checked_build_guard_fires():
    with sb.build_variant("checked"):
        sb.sb_checked_violations()
        status = sb.sb_checked_selftest()
        assert sb.sb_checked_violations() == 1
        s = status.cpu().numpy()
        assert s[0] == 5 and sb.sb_status_string(5).startswith("position or page")   # SB_ERR_BOUNDS
        assert s[1] == 1                                                           # only the in-range access ran
        assert sb.sb_checked_violations() == 0


def test_bounded_device_wait_runs_out_and_reports():
    """A wait on a barrier nobody arrives at gives up after its limit, sets the status word the way the
    product kernels do, releases the other waiting warp through the abort flag, and leaves the context
    usable.  Nothing traps or hangs."""
    limit_ns = 3_000_000                                      # 3 ms
    with sb.build_variant("test"):
        status, elapsed = sb.sb_test_wait_expires(limit_ns)
        torch.cuda.synchronize()
        e = elapsed.cpu().numpy()
        assert int(status[0]) == 6 and sb.sb_status_string(6) == "CUDA call failed"    # SB_ERR_CUDA
        assert limit_ns <= e[0] < 20 * limit_ns, e                                    # gave up at its own limit
        assert e[1] < 20 * limit_ns, e                                                # released by the abort flag, not after 2 s
        with pytest.raises(sb.SbError):
            sb.sb_test_wait_expires(10)                                               # below the allowed range
    # the context is intact: an ordinary call still works and matches the oracle
    attn, _ = W.config1_tiny()
    tb, q, kw = dev.attention_args(attn)
    out, lse, st = sb.sb_tree_attention(tb, q, **kw)
    torch.cuda.synchronize()
    ref_out, ref_lse, ref_status = oracle.tree_attention(**attn.oracle_kwargs())
    np.testing.assert_array_equal(st.cpu().numpy(), ref_status)
    assert_attention_close(out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), ref_out, ref_lse)
