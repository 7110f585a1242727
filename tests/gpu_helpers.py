"""Shared pieces of the GPU parity tests: run the CUDA library through its binding, run the
oracle on the same host arrays, compare with the stated tolerances."""
import numpy as np
import torch

import oracle
from paper_2605_07243_b200 import binding as sb
from paper_2605_07243_b200 import device_inputs as dev

# bf16 attention outputs: |err| <= 1e-2 + 1e-2*|ref|; fp32 log-sum-exp: |err| <= 1e-5*max(1,|ref|)
OUT_ATOL, OUT_RTOL, LSE_RTOL = 1e-2, 1e-2, 1e-5


def require_gpu():
    if not torch.cuda.is_available():
        raise RuntimeError("GPU tests need a CUDA device")
    sb.load()


def gpu_attention(case, **kw):
    tb, q, args = dev.attention_args(case)
    args.update(kw)
    out, lse, status = sb.sb_tree_attention(tb, q, **args)
    torch.cuda.synchronize()
    return (out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64),
            status.cpu().numpy())


def assert_attention_close(out, lse, ref_out, ref_lse, what="", value_scale=1.0):
    """value_scale: magnitude of the V entries when it is not ~1 (the absolute term of the
    tolerance is stated for unit-variance values; rounding the probabilities to bf16 before the
    P.V product gives an absolute error proportional to |V|)."""
    err = np.abs(out - ref_out)
    bound = OUT_ATOL * value_scale + OUT_RTOL * np.abs(ref_out)
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, f"{what}: out error {err.max():.3e} is {worst:.2f}x the tolerance"
    lerr = np.abs(lse - ref_lse)
    lbound = LSE_RTOL * np.maximum(1.0, np.abs(ref_lse))
    lworst = float((lerr / lbound).max()) if lerr.size else 0.0
    assert lworst <= 1.0, f"{what}: lse error {lerr.max():.3e} is {lworst:.2f}x the tolerance"
    return worst, lworst


def check_attention(case, what="", sel=None, value_scale=1.0, **kw):
    """Full (or sampled, sel = int32 [n,3] of (b,node,head)) element-wise parity."""
    out, lse, status = gpu_attention(case, **kw)
    ref_out, ref_lse, ref_status = oracle.tree_attention(**case.oracle_kwargs(), sel=sel)
    np.testing.assert_array_equal(status, ref_status)
    if sel is not None:
        qoff = case.q_offsets if case.q_offsets is not None else case.node_offsets
        q0 = case.q_node_begin if case.q_node_begin is not None else np.zeros(case.batch, np.int32)
        rows = np.asarray([qoff[b] + i - q0[b] for b, i, _h in sel])
        heads = sel[:, 2]
        out, lse = out[rows, heads], lse[rows, heads]
    return assert_attention_close(out, lse, ref_out, ref_lse, what, value_scale)


def sample_rows(case, n, seed=0):
    """n random (b, node, head) triples among the rows that have a query."""
    rng = np.random.default_rng(seed)
    sizes = np.diff(case.node_offsets)
    q0 = case.q_node_begin if case.q_node_begin is not None else np.zeros(case.batch, np.int32)
    sel = []
    for _ in range(n):
        b = int(rng.integers(case.batch))
        sel.append((b, int(rng.integers(q0[b], sizes[b])), int(rng.integers(case.n_q_heads))))
    return np.asarray(sel, np.int32)
