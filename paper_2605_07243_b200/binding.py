"""ctypes binding of libspecblock.so -- argument marshalling only.

Every function here has the name of the C entry point it calls (include/specblock.h) and does
nothing but turn torch CUDA tensors into device pointers, size the workspace and raise on a
non-zero return code.  All computation happens in the CUDA library; there is no CPU fallback:
if the library is missing or no CUDA device is present these calls raise.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

SB_MAX_NODES = 128
SB_MAX_DEPTH = 32
SB_KMAX = 16
SB_BF16, SB_F32 = 0, 1

STATUS_NAMES = {0: "SB_OK", 1: "SB_ERR_INVALID_ARG", 2: "SB_ERR_UNSUPPORTED", 3: "SB_ERR_WORKSPACE",
                4: "SB_ERR_INVALID_TREE", 5: "SB_ERR_BOUNDS", 6: "SB_ERR_CUDA"}


class SbError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")


class _TreeBatch(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("page_size", C.c_int32), ("max_pages", C.c_int32), ("kv_capacity", C.c_int64),
        ("num_pages", C.c_int32), ("total_nodes", C.c_int32), ("page_table", C.c_void_p),
        ("prefix_len", C.c_void_p), ("node_offsets", C.c_void_p), ("parent", C.c_void_p),
        ("max_nodes", C.c_int32), ("max_kv_len", C.c_int32),
        ("index_arrays_settled", C.c_int32), ("prefix_rows_settled", C.c_int32),
    ]


_lib = None


def lib_path() -> str:
    return _build.LIB


def _open(path: str):
    lib = C.CDLL(path)
    lib.sb_status_string.restype = C.c_char_p
    lib.sb_version.restype = C.c_int32
    lib.sb_kernel_launch_count.restype = C.c_int64
    for name in ("sb_tree_attention_workspace_bytes", "sb_tree_expand_workspace_bytes",
                 "sb_verify_accept_workspace_bytes", "sb_rank_features_workspace_bytes",
                 "sb_verify_sample_workspace_bytes", "sb_shift_project_workspace_bytes",
                 "sb_fuse_project_workspace_bytes"):
        getattr(lib, name).restype = C.c_size_t
    for name in ("sb_tree_ancestors", "sb_tree_attention", "sb_tree_expand", "sb_verify_accept",
                 "sb_verify_accept_static", "sb_kv_compact", "sb_path_rows", "sb_rank_features", "sb_verifier_signal",
                 "sb_verify_sample", "sb_shift_project", "sb_fuse_project", "sb_tree_expand_features"):
        getattr(lib, name).restype = C.c_int
    return lib


def load(build_if_missing: bool = True):
    """Load libspecblock.so (building it in-tree with nvcc when it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build() if build_if_missing else _build.LIB
    if not os.path.exists(path):
        raise RuntimeError("libspecblock.so is not built: run python -m paper_2605_07243_b200.build")
    _lib = _open(path)
    return _lib


_variants = {}


@contextlib.contextmanager
def build_variant(name: str):
    """Inside the block every call of this module goes to another build of the same sources:
    "test" (libspecblock_test.so: the mma.sync and one-warp-per-row attention kernels as independent
    cross-checks, the environment switches SB_ATTN_IMPL / SB_ATTN_TWO_TILES / SB_ATTN_MAX_CLUSTER /
    SB_NO_PDL / SB_DEBUG, and the wait-expiry kernel) or "checked" (libspecblock_checked.so: every
    computed index verified before use).  For tests; the library proper is what load() returns."""
    global _lib
    load()
    if name not in _variants:
        _variants[name] = _open(_build.build(variant=name))
    saved, _lib = _lib, _variants[name]
    try:
        yield _lib
    finally:
        _lib = saved


EXPORTED = ("sb_tree_ancestors", "sb_tree_attention", "sb_tree_attention_workspace_bytes",
            "sb_tree_expand", "sb_tree_expand_workspace_bytes", "sb_verify_accept",
            "sb_verify_accept_workspace_bytes", "sb_verify_accept_static", "sb_kv_compact", "sb_path_rows",
            "sb_rank_features", "sb_rank_features_workspace_bytes", "sb_verifier_signal", "sb_verify_sample",
            "sb_verify_sample_workspace_bytes", "sb_shift_project", "sb_shift_project_workspace_bytes",
            "sb_fuse_project", "sb_fuse_project_workspace_bytes", "sb_tree_expand_features", "sb_status_string",
            "sb_version",
            "sb_kernel_launch_count")


def _ptr(t: Optional[torch.Tensor], dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code, where):
    if code != 0:
        raise SbError(code, where)


def sb_kernel_launch_count() -> int:
    return int(load().sb_kernel_launch_count())


def sb_version() -> int:
    return int(load().sb_version())


def sb_status_string(code: int) -> str:
    return load().sb_status_string(C.c_int(code)).decode()


@dataclass
class TreeBatch:
    """Device-side description of a ragged batch of trees over one layer's KV cache; mirrors the
    C struct sb_tree_batch field for field.  k_cache / v_cache: bf16 tensors."""
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    k_cache: torch.Tensor
    v_cache: torch.Tensor
    prefix_len: torch.Tensor          # int32 [B]
    node_offsets: torch.Tensor        # int32 [B+1]
    parent: torch.Tensor              # int32 [total_nodes]
    total_nodes: int
    max_nodes: int
    max_kv_len: int
    page_size: int = 0
    kv_capacity: int = 0
    page_table: Optional[torch.Tensor] = None   # int32 [B, max_pages]
    num_pages: int = 0
    max_pages: int = 0

    def c_struct(self, k_cache=None, v_cache=None, settled=False, prefix_settled=False) -> _TreeBatch:
        k = self.k_cache if k_cache is None else k_cache
        v = self.v_cache if v_cache is None else v_cache
        s = _TreeBatch()
        s.batch = self.prefix_len.numel()
        s.n_q_heads, s.n_kv_heads, s.head_dim = self.n_q_heads, self.n_kv_heads, self.head_dim
        s.k_cache = _ptr(k, torch.bfloat16).value
        s.v_cache = _ptr(v, torch.bfloat16).value
        s.page_size, s.max_pages, s.kv_capacity = self.page_size, self.max_pages, self.kv_capacity
        s.num_pages, s.total_nodes = self.num_pages, self.total_nodes
        s.page_table = None if self.page_table is None else _ptr(self.page_table, torch.int32).value
        s.prefix_len = _ptr(self.prefix_len, torch.int32).value
        s.node_offsets = _ptr(self.node_offsets, torch.int32).value
        s.parent = _ptr(self.parent, torch.int32).value
        s.max_nodes, s.max_kv_len = self.max_nodes, self.max_kv_len
        s.index_arrays_settled = 1 if settled else 0
        s.prefix_rows_settled = 1 if (settled and prefix_settled) else 0
        return s


def sb_tree_ancestors(node_offsets, parent, max_nodes, anc_mask=None, depth=None, status=None):
    """-> (anc_mask int32 [total,4] holding the uint32 words, depth int32 [total], status [B])."""
    batch = node_offsets.numel() - 1
    total = parent.numel()
    dev = parent.device
    anc_mask = torch.empty((total, 4), dtype=torch.int32, device=dev) if anc_mask is None else anc_mask
    depth = torch.empty(total, dtype=torch.int32, device=dev) if depth is None else depth
    status = torch.empty(batch, dtype=torch.int32, device=dev) if status is None else status
    rc = load().sb_tree_ancestors(C.c_int32(batch), _ptr(node_offsets, torch.int32),
                                  _ptr(parent, torch.int32), C.c_int32(max_nodes), _ptr(anc_mask),
                                  _ptr(depth, torch.int32), _ptr(status, torch.int32), _stream())
    _check(rc, "sb_tree_ancestors")
    return anc_mask, depth, status


def sb_tree_attention_workspace_bytes(tb: TreeBatch, total_q: int, num_splits: int = 0) -> int:
    s = tb.c_struct()
    return int(load().sb_tree_attention_workspace_bytes(C.byref(s), C.c_int32(total_q),
                                                        C.c_int32(num_splits)))


def sb_tree_attention(tb: TreeBatch, q, out=None, lse=None, *, q_node_begin=None, q_offsets=None,
                      scale=0.0, num_splits=0, workspace=None, status=None, want_lse=True,
                      k_cache=None, v_cache=None, index_arrays_settled=False, prefix_rows_settled=False):
    """q bf16 [total_q, Hq, D] -> (out bf16 like q, lse fp32 [total_q, Hq] or None, status [B]).
    k_cache / v_cache override the batch's layer (same layout) without rebuilding it.
    index_arrays_settled: the kernel enqueued just before this call does not write the batch's index
    arrays (e.g. it is the previous layer's attention): the lengths may be fetched under its tail.
    prefix_rows_settled (with index_arrays_settled): nor does it write cache rows below prefix_len: key
    blocks inside the prefix may be requested under its tail too."""
    total_q = q.shape[0]
    dev = q.device
    out = torch.empty_like(q) if out is None else out
    if lse is None and want_lse:
        lse = torch.empty((total_q, tb.n_q_heads), dtype=torch.float32, device=dev)
    status = torch.empty(tb.prefix_len.numel(), dtype=torch.int32, device=dev) if status is None else status
    s = tb.c_struct(k_cache, v_cache, index_arrays_settled, prefix_rows_settled)
    lib = load()
    if workspace is None:
        need = int(lib.sb_tree_attention_workspace_bytes(C.byref(s), C.c_int32(total_q),
                                                         C.c_int32(num_splits)))
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    rc = lib.sb_tree_attention(C.byref(s), _ptr(q_node_begin, torch.int32), _ptr(q_offsets, torch.int32),
                               C.c_int32(total_q), _ptr(q, torch.bfloat16), _ptr(out, torch.bfloat16),
                               _ptr(lse, torch.float32), C.c_float(scale), C.c_int32(num_splits),
                               _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()),
                               _ptr(status, torch.int32), _stream())
    _check(rc, "sb_tree_attention")
    return out, lse, status


def sb_verify_accept_workspace_bytes(total_nodes: int, vocab: int) -> int:
    return int(load().sb_verify_accept_workspace_bytes(C.c_int32(total_nodes), C.c_int32(vocab)))


def sb_verify_accept(logits, node_offsets, parent, tok, max_depth, *, vocab=None, workspace=None,
                     out=None):
    """logits [total_nodes, stride] bf16 or fp32 -> dict(amax, accept_len, path_nodes, out_tokens,
    bonus, status) of int32 device tensors (`out` may pass preallocated ones)."""
    total, stride = logits.shape
    vocab = stride if vocab is None else vocab
    batch = node_offsets.numel() - 1
    dev = logits.device
    dt = {torch.bfloat16: SB_BF16, torch.float32: SB_F32}[logits.dtype]
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = dict(amax=torch.empty(total, **i32), accept_len=torch.empty(batch, **i32),
                   path_nodes=torch.empty((batch, max_depth + 1), **i32),
                   out_tokens=torch.empty((batch, max_depth + 1), **i32),
                   bonus=torch.empty(batch, **i32), status=torch.empty(batch, **i32))
    lib = load()
    if workspace is None:
        need = sb_verify_accept_workspace_bytes(total, vocab)
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    rc = lib.sb_verify_accept(_ptr(logits), C.c_int(dt), C.c_int64(stride), C.c_int32(vocab),
                              C.c_int32(batch), C.c_int32(total), _ptr(node_offsets, torch.int32),
                              _ptr(parent, torch.int32), _ptr(tok, torch.int32), C.c_int32(max_depth),
                              _ptr(out["amax"]), _ptr(out["accept_len"]), _ptr(out["path_nodes"]),
                              _ptr(out["out_tokens"]), _ptr(out["bonus"]), _ptr(workspace),
                              C.c_size_t(workspace.numel()), _ptr(out["status"]), _stream())
    _check(rc, "sb_verify_accept")
    return out


def sb_rank_features_workspace_bytes(n_rows: int, vocab: int) -> int:
    return int(load().sb_rank_features_workspace_bytes(C.c_int32(n_rows), C.c_int32(vocab)))


def sb_rank_features(scores, *, vocab=None, features=None, workspace=None):
    """scores fp32 [R, stride] -> features fp32 [R, 15] (top-10 log-probs, 3 logit gaps, top
    probability, entropy)."""
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    dev = scores.device
    features = torch.empty((n_rows, 15), dtype=torch.float32, device=dev) if features is None else features
    if workspace is None:
        workspace = torch.empty(max(sb_rank_features_workspace_bytes(n_rows, vocab), 256), dtype=torch.uint8, device=dev)
    rc = load().sb_rank_features(_ptr(scores, torch.float32), C.c_int64(stride), C.c_int32(n_rows), C.c_int32(vocab),
                                 _ptr(features, torch.float32), _ptr(workspace), C.c_size_t(workspace.numel()),
                                 _stream())
    _check(rc, "sb_rank_features")
    return features


def sb_verifier_signal(scores, node_offsets, child_row, path_nodes, accept_len, bonus, max_depth, signal, *,
                       vocab=None, r_prob=None, status=None):
    """One iteration's term of s = sum (1 - r): signal fp32 [B] is updated in place.
    -> dict(r_prob, signal, status)."""
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    batch = node_offsets.numel() - 1
    dev = scores.device
    r_prob = torch.empty(batch, dtype=torch.float32, device=dev) if r_prob is None else r_prob
    status = torch.empty(batch, dtype=torch.int32, device=dev) if status is None else status
    rc = load().sb_verifier_signal(
        _ptr(scores, torch.float32), C.c_int64(stride), C.c_int32(n_rows), C.c_int32(vocab), C.c_int32(batch),
        C.c_int32(child_row.numel()), _ptr(node_offsets, torch.int32), _ptr(child_row, torch.int32),
        _ptr(path_nodes, torch.int32), _ptr(accept_len, torch.int32), _ptr(bonus, torch.int32),
        C.c_int32(max_depth), _ptr(r_prob, torch.float32), _ptr(signal, torch.float32), _ptr(status, torch.int32),
        _stream())
    _check(rc, "sb_verifier_signal")
    return dict(r_prob=r_prob, signal=signal, status=status)


def sb_verify_sample_workspace_bytes(batch: int, vocab: int, total_nodes: int, n_rows: int) -> int:
    return int(load().sb_verify_sample_workspace_bytes(C.c_int32(batch), C.c_int32(vocab), C.c_int32(total_nodes),
                                                       C.c_int32(n_rows)))


def sb_verify_sample(logits, scores, node_offsets, parent, tok, child_row, temperature, u_accept, u_bonus, max_depth,
                     *, vocab=None, workspace=None, out=None):
    """Stochastic tree verification (temperature > 0); the uniforms are inputs.
    -> dict(accept_len, path_nodes, out_tokens, bonus, status)."""
    total, stride = logits.shape
    n_rows, sstride = scores.shape
    vocab = stride if vocab is None else vocab
    batch = node_offsets.numel() - 1
    dev = logits.device
    dt = {torch.bfloat16: SB_BF16, torch.float32: SB_F32}[logits.dtype]
    if out is None:
        i32 = dict(dtype=torch.int32, device=dev)
        out = dict(accept_len=torch.empty(batch, **i32), path_nodes=torch.empty((batch, max_depth + 1), **i32),
                   out_tokens=torch.empty((batch, max_depth + 1), **i32), bonus=torch.empty(batch, **i32),
                   status=torch.empty(batch, **i32))
    if workspace is None:
        workspace = torch.empty(max(sb_verify_sample_workspace_bytes(batch, vocab, total, n_rows), 256), dtype=torch.uint8,
                                device=dev)
    rc = load().sb_verify_sample(
        _ptr(logits), C.c_int(dt), C.c_int64(stride), C.c_int32(vocab), _ptr(scores, torch.float32), C.c_int64(sstride),
        C.c_int32(n_rows), C.c_int32(batch), C.c_int32(total), _ptr(node_offsets, torch.int32),
        _ptr(parent, torch.int32), _ptr(tok, torch.int32), _ptr(child_row, torch.int32), C.c_float(temperature),
        _ptr(u_accept, torch.float32), _ptr(u_bonus, torch.float32), C.c_int32(max_depth), _ptr(out["accept_len"]),
        _ptr(out["path_nodes"]), _ptr(out["out_tokens"]), _ptr(out["bonus"]), _ptr(workspace),
        C.c_size_t(workspace.numel()), _ptr(out["status"]), _stream())
    _check(rc, "sb_verify_sample")
    return out


def sb_shift_project_workspace_bytes(n_rows: int, d: int, d_out: int, block_k: int) -> int:
    return int(load().sb_shift_project_workspace_bytes(C.c_int32(n_rows), C.c_int32(d), C.c_int32(d_out),
                                                       C.c_int32(block_k)))


def sb_shift_project(h, w, block_k, *, out=None, workspace=None, status=None):
    """h bf16 [R, d], w bf16 [d_out, 2d] (block_k > 0) or [d_out, d] (block_k = 0) -> out bf16 [R, d_out]."""
    n_rows, d = h.shape
    d_out = w.shape[0]
    dev = h.device
    out = torch.empty((n_rows, d_out), dtype=torch.bfloat16, device=dev) if out is None else out
    status = torch.zeros(1, dtype=torch.int32, device=dev) if status is None else status
    if w.shape[1] != (2 * d if block_k > 0 else d):
        raise ValueError("w must be [d_out, 2d] with block_k > 0 and [d_out, d] with block_k = 0")
    if workspace is None:
        workspace = torch.zeros(max(sb_shift_project_workspace_bytes(n_rows, d, d_out, block_k), 256), dtype=torch.uint8,
                                device=dev)
    rc = load().sb_shift_project(_ptr(h, torch.bfloat16), _ptr(w, torch.bfloat16), C.c_int32(n_rows), C.c_int32(d),
                                 C.c_int32(d_out), C.c_int32(block_k), _ptr(out, torch.bfloat16), _ptr(workspace),
                                 C.c_size_t(workspace.numel()), _ptr(status, torch.int32), _stream())
    _check(rc, "sb_shift_project")
    return out, status


def sb_fuse_project_workspace_bytes(n_starts: int, block_k: int, d: int, d_out: int, q_term_valid: bool) -> int:
    return int(load().sb_fuse_project_workspace_bytes(C.c_int32(n_starts), C.c_int32(block_k), C.c_int32(d),
                                                      C.c_int32(d_out), C.c_int32(1 if q_term_valid else 0)))


def sb_fuse_project(c, e, q, w, *, gain_c=None, gain_e=None, gain_q=None, eps=1e-6, q_term=None, q_term_valid=False,
                    out=None, workspace=None, status=None):
    """c, e bf16 [S, d], q bf16 [K, d], w bf16 [d_out, 3d] -> out bf16 [S*K, d_out] (row s*K + k).
    q_term fp32 [K, d_out]: written when q_term_valid is false, read (and a third of w skipped) when true."""
    n_starts, d = c.shape
    block_k = q.shape[0]
    d_out = w.shape[0]
    dev = c.device
    if e.shape != c.shape or q.shape[1] != d or w.shape[1] != 3 * d:
        raise ValueError("expected c, e [S, d], q [K, d], w [d_out, 3d]")
    if q_term is not None and tuple(q_term.shape) != (block_k, d_out):
        raise ValueError("q_term must be [K, d_out]")
    out = torch.empty((n_starts * block_k, d_out), dtype=torch.bfloat16, device=dev) if out is None else out
    status = torch.zeros(1, dtype=torch.int32, device=dev) if status is None else status
    if workspace is None:
        workspace = torch.zeros(max(sb_fuse_project_workspace_bytes(n_starts, block_k, d, d_out, q_term_valid), 256),
                                dtype=torch.uint8, device=dev)
    rc = load().sb_fuse_project(_ptr(c, torch.bfloat16), _ptr(e, torch.bfloat16), _ptr(q, torch.bfloat16),
                                _ptr(gain_c, torch.float32), _ptr(gain_e, torch.float32), _ptr(gain_q, torch.float32),
                                C.c_float(eps), _ptr(w, torch.bfloat16), C.c_int32(n_starts), C.c_int32(block_k),
                                C.c_int32(d), C.c_int32(d_out), _ptr(q_term, torch.float32),
                                C.c_int32(1 if q_term_valid else 0), _ptr(out, torch.bfloat16), _ptr(workspace),
                                C.c_size_t(workspace.numel()), _ptr(status, torch.int32), _stream())
    _check(rc, "sb_fuse_project")
    return out, status


SB_STATIC_SCRATCH_BYTES = 256 * 1024


def sb_verify_accept_static(logits, node_offsets, parent, tok, max_depth, out, *, vocab=None):
    """sb_verify_accept without a workspace, for callers that cannot allocate device memory: the
    library's own fixed scratch array is used (at most SB_STATIC_SCRATCH_BYTES of partials, else
    SB_ERR_WORKSPACE).  `out` must hold the preallocated result tensors (amax, accept_len,
    path_nodes, out_tokens, bonus, status): nothing is allocated here either.  Calls that may
    overlap on the GPU share that array and must be serialised by the caller."""
    total, stride = logits.shape
    vocab = stride if vocab is None else vocab
    batch = node_offsets.numel() - 1
    dt = {torch.bfloat16: SB_BF16, torch.float32: SB_F32}[logits.dtype]
    rc = load().sb_verify_accept_static(
        _ptr(logits), C.c_int(dt), C.c_int64(stride), C.c_int32(vocab), C.c_int32(batch), C.c_int32(total),
        _ptr(node_offsets, torch.int32), _ptr(parent, torch.int32), _ptr(tok, torch.int32),
        C.c_int32(max_depth), _ptr(out["amax"]), _ptr(out["accept_len"]), _ptr(out["path_nodes"]),
        _ptr(out["out_tokens"]), _ptr(out["bonus"]), _ptr(out["status"]), _stream())
    _check(rc, "sb_verify_accept_static")
    return out


def sb_kv_compact(tb: TreeBatch, n_layers, layer_stride_elems, path_nodes, accept_len, max_depth,
                  new_len=None, status=None):
    """In-place compaction of tb.k_cache / tb.v_cache (layer 0 of n_layers).  -> (new_len, status)."""
    batch = tb.prefix_len.numel()
    dev = tb.prefix_len.device
    new_len = torch.empty(batch, dtype=torch.int32, device=dev) if new_len is None else new_len
    status = torch.empty(batch, dtype=torch.int32, device=dev) if status is None else status
    s = tb.c_struct()
    rc = load().sb_kv_compact(C.byref(s), C.c_int32(n_layers), C.c_int64(layer_stride_elems),
                              _ptr(path_nodes, torch.int32), _ptr(accept_len, torch.int32),
                              C.c_int32(max_depth), _ptr(new_len, torch.int32),
                              _ptr(status, torch.int32), _stream())
    _check(rc, "sb_kv_compact")
    return new_len, status


def sb_path_rows(node_offsets, node_row, path_nodes, accept_len, max_depth, path_rows=None, status=None,
                 row_begin=None):
    """The accepted path in the drafter's row numbering: -> (path_rows int32 [B, max_depth+1], status [B])."""
    batch = node_offsets.numel() - 1
    dev = node_row.device
    if path_rows is None:
        path_rows = torch.empty((batch, max_depth + 1), dtype=torch.int32, device=dev)
    status = torch.empty(batch, dtype=torch.int32, device=dev) if status is None else status
    rc = load().sb_path_rows(C.c_int32(batch), _ptr(node_offsets, torch.int32), _ptr(node_row, torch.int32),
                             _ptr(row_begin, torch.int32), _ptr(path_nodes, torch.int32),
                             _ptr(accept_len, torch.int32), C.c_int32(max_depth), _ptr(path_rows, torch.int32),
                             _ptr(status, torch.int32), _stream())
    _check(rc, "sb_path_rows")
    return path_rows, status


def sb_tree_expand_workspace_bytes(n_rows: int, vocab: int) -> int:
    return int(load().sb_tree_expand_workspace_bytes(C.c_int32(n_rows), C.c_int32(vocab)))


def sb_tree_expand(scores, block_k, bucket, bmap, start_parent, node_budget, tree, *, vocab=None,
                   workspace=None, topk_tok=None, topk_val=None, status=None, features=None, child_row=None,
                   row_base=0):
    """scores fp32 [R, stride]; bucket uint8 [R]; bmap: 4 host ints; tree: dict of int32 device
    tensors n_nodes [1], tok, parent, depth, node_row, node_rank (capacity node_budget), updated
    in place.  -> (topk_tok [R,16], topk_val [R,16], status [1]).
    features fp32 [R, 15]: also filled (sb_tree_expand_features: one pass over the scores for both);
    the workspace must then hold sb_rank_features_workspace_bytes.  With features, child_row int32
    [node_budget] (initialised to -1 by the caller) receives row_base + row for the nodes whose children a row
    of this call proposes."""
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    dev = scores.device
    topk_tok = torch.empty((n_rows, SB_KMAX), dtype=torch.int32, device=dev) if topk_tok is None else topk_tok
    topk_val = torch.empty((n_rows, SB_KMAX), dtype=torch.float32, device=dev) if topk_val is None else topk_val
    status = torch.empty(1, dtype=torch.int32, device=dev) if status is None else status
    lib = load()
    if workspace is None:
        need = (sb_tree_expand_workspace_bytes if features is None else sb_rank_features_workspace_bytes)(n_rows, vocab)
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    bm = (C.c_int32 * 4)(*[int(x) for x in bmap])
    head = (_ptr(scores, torch.float32), C.c_int64(stride), C.c_int32(n_rows),
            C.c_int32(vocab), C.c_int32(block_k), _ptr(bucket, torch.uint8), bm,
            _ptr(start_parent, torch.int32), C.c_int32(node_budget),
            _ptr(tree["n_nodes"], torch.int32), _ptr(tree["tok"], torch.int32),
            _ptr(tree["parent"], torch.int32), _ptr(tree["depth"], torch.int32),
            _ptr(tree["node_row"], torch.int32), _ptr(tree["node_rank"], torch.int32),
            _ptr(topk_tok, torch.int32), _ptr(topk_val, torch.float32))
    tail = (_ptr(workspace), C.c_size_t(workspace.numel()), _ptr(status, torch.int32), _stream())
    if features is None:
        _check(lib.sb_tree_expand(*head, *tail), "sb_tree_expand")
    else:
        _check(lib.sb_tree_expand_features(*head, _ptr(features, torch.float32), _ptr(child_row, torch.int32),
                                           C.c_int32(row_base), *tail), "sb_tree_expand_features")
    return topk_tok, topk_val, status


# ---- hooks of the test and checked builds (include/specblock_test.h); use inside build_variant(...) ----

def sb_test_wait_expires(limit_ns: int):
    """Test build: lets a bounded device wait run out.  -> (status int32[1], elapsed_ns int64[2]) tensors."""
    lib = load()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    elapsed = torch.zeros(2, dtype=torch.int64, device="cuda")
    lib.sb_test_wait_expires.restype = C.c_int
    _check(lib.sb_test_wait_expires(C.c_int64(limit_ns), _ptr(status), _ptr(elapsed), _stream()), "sb_test_wait_expires")
    return status, elapsed


def sb_checked_violations() -> int:
    """Checked build: accesses refused since the last call (synchronises the device, clears the counter)."""
    lib = load()
    lib.sb_checked_violations.restype = C.c_int
    n = C.c_int64(-1)
    _check(lib.sb_checked_violations(C.byref(n)), "sb_checked_violations")
    return int(n.value)


def sb_checked_selftest():
    """Checked build: one refused access on purpose.  -> status int32[2] tensor."""
    lib = load()
    lib.sb_checked_selftest.restype = C.c_int
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    _check(lib.sb_checked_selftest(_ptr(status), _stream()), "sb_checked_selftest")
    return status
