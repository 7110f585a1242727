"""The whole verify iteration through pipeline.VerifyStep (the sequence of C-ABI calls bench.py times):
device-resident inputs against the oracle, and the host-buffer path against the device-resident one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import workloads as W
from paper_2605_07243_b200.pipeline import VerifyStep

pytestmark = pytest.mark.gpu


def _small_step(keep_host):
    par = W.config2_tree()
    layers = [W.config2_verify_layer(layer=l, par=par, prefix=300) for l in range(3)]
    ver = W.config2_logits(par=par, vocab=5000, accept_len=3)
    _, exp = W.config3_drafter()
    exp_small = W.ExpandCase(exp.scores[:, :4099].copy(), exp.block_k, exp.bucket, exp.bmap, exp.start_parent,
                             exp.node_budget, exp.tree)
    return layers, ver, exp_small, VerifyStep(layers, ver, exp_small, keep_host=keep_host)


def test_verify_step_device_path_matches_oracle():
    layers, ver, exp, step = _small_step(False)
    k0 = [c.k.copy() for c in layers]
    step.run_device()
    torch.cuda.synchronize()
    assert int(step.attn_status.max()) == 0 and int(step.compact_status.max()) == 0
    for l, case in enumerate(layers):
        ref_out, ref_lse, _ = oracle.tree_attention(**case.oracle_kwargs())
        got = step.out_all[l].float().cpu().numpy().astype(np.float64)
        assert (np.abs(got - ref_out) <= 1e-2 + 1e-2 * np.abs(ref_out)).all(), f"layer {l}"
        assert (np.abs(step.lse_all[l].cpu().numpy() - ref_lse) <= 1e-5 * np.maximum(1, np.abs(ref_lse))).all()
    ref = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
    for key in ("amax", "accept_len", "path_nodes", "out_tokens", "bonus", "status"):
        np.testing.assert_array_equal(step.accept[key].cpu().numpy(), ref[key], err_msg=key)
    assert int(ref["accept_len"][0]) == 3
    # compaction of every layer's K against the out-of-place gather
    c0 = layers[0]
    all_k = np.stack(k0).reshape(-1)
    ref_k, ref_len, _ = oracle.kv_compact(
        n_kv_heads=c0.n_kv_heads, head_dim=c0.head_dim, cache=all_k, n_layers=len(layers),
        layer_stride_elems=int(c0.k.size), kv_capacity=c0.kv_capacity, prefix_len=c0.prefix_len,
        node_offsets=c0.node_offsets, path_nodes=ref["path_nodes"], accept_len=ref["accept_len"],
        max_depth=ver.max_depth)
    got_k = step.k_all.view(torch.int16).cpu().numpy().view(np.uint16).reshape(len(layers), -1)
    new_len = int(ref_len[0])
    row = c0.n_kv_heads * c0.head_dim
    np.testing.assert_array_equal(step.new_len.cpu().numpy(), ref_len)
    np.testing.assert_array_equal(got_k[:, :new_len * row], ref_k.reshape(len(layers), -1)[:, :new_len * row])
    # the expansion next to it
    e = step.expand
    ref_e = oracle.tree_expand(exp.scores, exp.block_k, exp.bucket, exp.bmap, exp.start_parent, exp.node_budget,
                               tree=exp.tree)
    assert int(e["n_nodes"].cpu()[0]) == ref_e["n_nodes"]
    np.testing.assert_array_equal(e["tree"]["tok"].cpu().numpy()[:ref_e["n_nodes"]], ref_e["tok"][:ref_e["n_nodes"]])


def test_verify_step_from_host_buffers_equals_device_path():
    """run_from_host() pipelines host-to-device copies, kernels and device-to-host copies over three
    streams: its results in host memory must be bit-identical to the device-resident run, twice in a row
    (the second call overwrites the buffers the first one compacted in place)."""
    _, _, _, step = _small_step(True)
    step.run_device()
    torch.cuda.synchronize()
    want = dict(out=step.out_all.cpu(), lse=step.lse_all.cpu(), new_len=step.new_len.cpu(),
                **{k: v.cpu() for k, v in step.accept.items()})
    for rep in range(2):
        step.host["out"].zero_()
        step.host["lse"].zero_()
        step.run_from_host()
        torch.cuda.current_stream().synchronize()
        assert torch.equal(step.host["out"], want["out"]) and torch.equal(step.host["lse"], want["lse"])
        assert torch.equal(step.host["new_len"], want["new_len"])
        for k in step.accept:
            assert torch.equal(step.host["res"][k], want[k]), k
    h2d, d2h = step.host_bytes()
    assert h2d > 3 * 2 * step.k_all[0].numel() * 2 and d2h >= step.out_all.numel() * 2


def test_graph_replay_of_the_step_is_bit_stable():
    """The step as one CUDA graph, replayed 2000 times back to back (every layer's attention a programmatic
    dependent of the one before, lengths and prefix keys requested under the predecessor's tail): every
    output keeps its bits and every status word stays zero.  The first replays are left out of the
    comparison because compaction moves cache rows in place until the accepted rows have settled."""
    _, _, _, step = _small_step(False)
    stream = torch.cuda.Stream()

    def snapshot():
        e = step.expand
        t = [o.clone() for o in step.out_all] + [l.clone() for l in step.lse_all]
        t += [v.clone() for v in step.accept.values()] + [step.new_len.clone(), e["n_nodes"].clone(), e["topk_tok"].clone()]
        return t + [e["tree"][k].clone() for k in sorted(e["tree"])]

    with torch.cuda.stream(stream):
        step.run_device()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step.run_device()
        for _ in range(10):
            graph.replay()
        stream.synchronize()
        ref = snapshot()
        for _ in range(2000):
            graph.replay()
        stream.synchronize()
        now = snapshot()
    for a, b in zip(ref, now):
        assert torch.equal(a, b)
    for s in (step.attn_status, step.accept["status"], step.compact_status, step.expand["status"]):
        assert int(s.max()) == 0
