"""sb_verify_accept_static: the variant of sb_verify_accept for callers that cannot allocate device
memory (its argmax partials live in a fixed array inside the library).  Collected last on purpose.

Called through the C ABI twice in a row on different inputs; every result must equal what the
workspace-taking entry point returns for the same inputs (integer results: exact equality), which
also shows that the shared array needs no clearing between calls -- and what the CPU oracle computes
from the same host arrays."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import device_inputs as dev
from paper_2605_07243_b200 import workloads as W

pytestmark = pytest.mark.gpu

KEYS = ("amax", "accept_len", "path_nodes", "out_tokens", "bonus", "status")


def _empty_out(total, batch, max_depth):
    i32 = dict(dtype=torch.int32, device="cuda")
    return dict(amax=torch.full((total,), -7, **i32), accept_len=torch.full((batch,), -7, **i32),
                path_nodes=torch.full((batch, max_depth + 1), -7, **i32),
                out_tokens=torch.full((batch, max_depth + 1), -7, **i32), bonus=torch.full((batch,), -7, **i32),
                status=torch.full((batch,), -7, **i32))


def _both_ways(case):
    logits = dev.bf16_tensor(case.logits) if case.logits.dtype == np.uint16 else torch.from_numpy(case.logits).cuda()
    offs, par, tok = dev.i32_tensor(case.node_offsets), dev.i32_tensor(case.parent), dev.i32_tensor(case.tok)
    total, batch = logits.shape[0], offs.numel() - 1
    ref = sb.sb_verify_accept(logits, offs, par, tok, case.max_depth)
    got = sb.sb_verify_accept_static(logits, offs, par, tok, case.max_depth, _empty_out(total, batch, case.max_depth))
    torch.cuda.synchronize()
    want = oracle.verify_accept(case.logits, case.node_offsets, case.parent, case.tok, case.max_depth)
    for k in KEYS:
        np.testing.assert_array_equal(got[k].cpu().numpy(), ref[k].cpu().numpy(), err_msg=k)
        np.testing.assert_array_equal(got[k].cpu().numpy(), want[k], err_msg=f"{k} against the oracle")
    return got


def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row():
    if not torch.cuda.is_available():
        raise RuntimeError("GPU tests need a CUDA device")
    rng = W.rng_for(91)
    # call 1: the 8B-shaped verify logits (60 nodes x 128256 bf16), planted acceptance length 5
    first = W.config2_logits(accept_len=5)
    got = _both_ways(first)
    assert int(got["accept_len"][0]) == int(first.planted_len[0])
    # call 2, straight after, different shape and dtype: a ragged fp32 batch with an invalid tree in it
    parents = [W.random_tree(rng, 33, 6), np.asarray([-1, 0, 3, 1], np.int32), W.random_tree(rng, 128, 10)]
    second = W.make_verify_case(rng, parents=[parents[0], W.chain_tree(4), parents[2]], vocab=5003, dtype="f32",
                                max_depth=10)
    second.parent[33:37] = parents[1]
    got = _both_ways(second)
    assert list(got["status"].cpu().numpy()) == [0, 4, 0]
    # and the first problem again: the array still holds call 2's partials, which must not matter
    _both_ways(first)


def test_static_scratch_variant_refuses_what_does_not_fit():
    if not torch.cuda.is_available():
        raise RuntimeError("GPU tests need a CUDA device")
    total, vocab = 60000, 8             # 60000 rows of partials do not fit the fixed array
    assert sb.sb_verify_accept_workspace_bytes(total, vocab) > sb.SB_STATIC_SCRATCH_BYTES
    logits = torch.zeros((total, vocab), dtype=torch.float32, device="cuda")  # never read: refused first
    offs = dev.i32_tensor([0, total])
    par = dev.i32_tensor(np.zeros(total, np.int32))
    with pytest.raises(sb.SbError) as e:
        lib = sb.load()
        import ctypes as C
        rc = lib.sb_verify_accept_static(C.c_void_p(logits.data_ptr()), C.c_int(1), C.c_int64(vocab), C.c_int32(vocab),
                                         C.c_int32(1), C.c_int32(total), C.c_void_p(offs.data_ptr()),
                                         C.c_void_p(par.data_ptr()), C.c_void_p(par.data_ptr()), C.c_int32(4),
                                         C.c_void_p(par.data_ptr()), C.c_void_p(par.data_ptr()),
                                         C.c_void_p(par.data_ptr()), C.c_void_p(par.data_ptr()),
                                         C.c_void_p(par.data_ptr()), C.c_void_p(par.data_ptr()), None)
        if rc != 0:
            raise sb.SbError(rc, "sb_verify_accept_static")
    assert e.value.code == 3
