"""ctypes loader for specblock_oracle.c -- TEST INFRASTRUCTURE ONLY.

Thin numpy marshalling around the C oracle; no arithmetic of the method lives here.
bf16 data travels as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "specblock_oracle.c")
_LIB = os.path.join(_HERE, "libspecblock_oracle.so")
_lock = threading.Lock()
_lib = None

KMAX = 16


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, OpenMP only to spread rows over cores)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = C.CDLL(build())
            _lib.sbo_num_threads.restype = C.c_int
            for name in ("sbo_tree_ancestors", "sbo_tree_attention", "sbo_accept_from_amax",
                         "sbo_tree_expand"):
                getattr(_lib, name).restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(_load().sbo_num_threads())


def tree_ancestors(parent):
    """-> (anc_mask uint32 [n,4], depth int32 [n], rc)."""
    parent = _i32(parent)
    n = parent.shape[0]
    anc = np.zeros((n, 4), np.uint32)
    depth = np.zeros(n, np.int32)
    rc = _load().sbo_tree_ancestors(_p(parent), C.c_int(n), _p(anc), _p(depth))
    return anc, depth, int(rc)


def tree_attention(*, n_q_heads, n_kv_heads, head_dim, k, v, page_size=0, max_pages=0,
                   num_pages=0, kv_capacity=0, page_table=None, prefix_len, node_offsets, parent,
                   q, q_node_begin=None, q_offsets=None, scale=0.0, sel=None):
    """k, v, q: uint16 bf16 bit patterns.  -> (out f64, lse f64, status int32 [B]).

    sel=None: out [total_q, Hq, D], lse [total_q, Hq]; else sel int32 [n,3] of (b, node, head)
    and out [n, D], lse [n].
    """
    k = np.ascontiguousarray(k, np.uint16)
    v = np.ascontiguousarray(v, np.uint16)
    q = np.ascontiguousarray(q, np.uint16)
    prefix_len, node_offsets, parent = _i32(prefix_len), _i32(node_offsets), _i32(parent)
    q_node_begin, q_offsets, page_table = _i32(q_node_begin), _i32(q_offsets), _i32(page_table)
    batch = prefix_len.shape[0]
    total_q = q.size // (n_q_heads * head_dim)
    if sel is None:
        n_sel = 0
        out = np.zeros((total_q, n_q_heads, head_dim), np.float64)
        lse = np.zeros((total_q, n_q_heads), np.float64)
    else:
        sel = _i32(sel).reshape(-1, 3)
        n_sel = sel.shape[0]
        out = np.zeros((n_sel, head_dim), np.float64)
        lse = np.zeros(n_sel, np.float64)
    status = np.zeros(batch, np.int32)
    _load().sbo_tree_attention(
        C.c_int(batch), C.c_int(n_q_heads), C.c_int(n_kv_heads), C.c_int(head_dim), _p(k), _p(v),
        C.c_int(page_size), C.c_int(max_pages), C.c_int(num_pages), C.c_int64(kv_capacity),
        _p(page_table), _p(prefix_len), _p(node_offsets), _p(parent), _p(q_node_begin),
        _p(q_offsets), _p(q), C.c_double(scale), C.c_int64(n_sel), _p(sel), _p(out), _p(lse),
        _p(status))
    return out, lse, status


def _logits_arg(logits):
    if logits.dtype == np.uint16:
        return np.ascontiguousarray(logits), 0
    if logits.dtype == np.float32:
        return np.ascontiguousarray(logits), 1
    raise TypeError("logits must be uint16 (bf16 bits) or float32")


def row_argmax(logits, vocab=None):
    logits, dt = _logits_arg(logits)
    n_rows, stride = logits.shape
    vocab = stride if vocab is None else vocab
    amax = np.zeros(n_rows, np.int32)
    _load().sbo_row_argmax(_p(logits), C.c_int(dt), C.c_int64(stride), C.c_int(vocab),
                           C.c_int64(n_rows), _p(amax))
    return amax


def row_topk(scores, vocab=None):
    scores = np.ascontiguousarray(scores, np.float32)
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    tok = np.zeros((n_rows, KMAX), np.int32)
    val = np.zeros((n_rows, KMAX), np.float32)
    _load().sbo_row_topk(_p(scores), C.c_int64(stride), C.c_int(n_rows), C.c_int(vocab), _p(tok),
                         _p(val))
    return tok, val


def rank_features(scores, vocab=None):
    """-> float64 [n_rows, 15]: top-10 log-probs, 3 logit gaps, top probability, entropy."""
    scores = np.ascontiguousarray(scores, np.float32)
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    feats = np.zeros((n_rows, 15), np.float64)
    _load().sbo_rank_features(_p(scores), C.c_int64(stride), C.c_int(n_rows), C.c_int(vocab), _p(feats))
    return feats


def shift_project(h, w, block_k):
    """h uint16 (bf16 bits) [R, d], w uint16 [d_out, 2d] (block_k > 0) or [d_out, d] (block_k = 0) -> f64 [R, d_out]."""
    h = np.ascontiguousarray(h, np.uint16)
    w = np.ascontiguousarray(w, np.uint16)
    n_rows, d = h.shape
    d_out, kin = w.shape
    assert kin == (2 * d if block_k > 0 else d)
    out = np.zeros((n_rows, d_out), np.float64)
    _load().sbo_shift_project(_p(h), _p(w), C.c_int(n_rows), C.c_int(d), C.c_int(d_out), C.c_int(block_k), _p(out))
    return out


def fuse_project(c, e, q, w, gain_c=None, gain_e=None, gain_q=None, eps=1e-6):
    """c, e uint16 (bf16 bits) [S, d], q uint16 [K, d], w uint16 [d_out, 3d], gains f32 [d] or None -> f64 [S*K, d_out]."""
    c, e, q, w = (np.ascontiguousarray(a, np.uint16) for a in (c, e, q, w))
    n_starts, d = c.shape
    block_k = q.shape[0]
    d_out = w.shape[0]
    assert e.shape == c.shape and q.shape[1] == d and w.shape[1] == 3 * d
    gains = [None if g is None else np.ascontiguousarray(g, np.float32) for g in (gain_c, gain_e, gain_q)]
    out = np.zeros((n_starts * block_k, d_out), np.float64)
    _load().sbo_fuse_project(_p(c), _p(e), _p(q), *[_p(g) for g in gains], C.c_double(eps),
                             _p(w), C.c_int(n_starts), C.c_int(block_k), C.c_int(d), C.c_int(d_out), _p(out))
    return out


def verifier_signal(scores, node_offsets, child_row, path_nodes, accept_len, bonus, max_depth, signal=None,
                    vocab=None):
    """-> dict(r_prob f64 [B], signal f64 [B] (= signal in + 1 - r), status int32 [B])."""
    scores = np.ascontiguousarray(scores, np.float32)
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    node_offsets, child_row = _i32(node_offsets), _i32(child_row)
    path_nodes, accept_len, bonus = _i32(path_nodes), _i32(accept_len), _i32(bonus)
    batch = node_offsets.shape[0] - 1
    r_prob = np.zeros(batch, np.float64)
    sig = np.zeros(batch, np.float64) if signal is None else np.array(signal, np.float64)
    status = np.zeros(batch, np.int32)
    _load().sbo_verifier_signal(_p(scores), C.c_int64(stride), C.c_int(n_rows), C.c_int(vocab), C.c_int(batch),
                                _p(node_offsets), _p(child_row), _p(path_nodes), _p(accept_len), _p(bonus),
                                C.c_int(max_depth), _p(r_prob), _p(sig), _p(status))
    return dict(r_prob=r_prob, signal=sig, status=status)


def verify_accept(logits, node_offsets, parent, tok, max_depth, vocab=None):
    """-> dict(amax, accept_len, path_nodes, out_tokens, bonus, status)."""
    logits, dt = _logits_arg(logits)
    node_offsets, parent, tok = _i32(node_offsets), _i32(parent), _i32(tok)
    batch = node_offsets.shape[0] - 1
    total, stride = logits.shape
    vocab = stride if vocab is None else vocab
    r = dict(amax=np.zeros(total, np.int32), accept_len=np.zeros(batch, np.int32),
             path_nodes=np.zeros((batch, max_depth + 1), np.int32),
             out_tokens=np.zeros((batch, max_depth + 1), np.int32),
             bonus=np.zeros(batch, np.int32), status=np.zeros(batch, np.int32))
    _load().sbo_verify_accept(_p(logits), C.c_int(dt), C.c_int64(stride), C.c_int(vocab),
                              C.c_int(batch), _p(node_offsets), _p(parent), _p(tok),
                              C.c_int(max_depth), _p(r["amax"]), _p(r["accept_len"]),
                              _p(r["path_nodes"]), _p(r["out_tokens"]), _p(r["bonus"]),
                              _p(r["status"]))
    return r


def verify_sample(logits, scores, node_offsets, parent, tok, child_row, temperature, u_accept, u_bonus, max_depth,
                  vocab=None):
    """Stochastic tree verification.  -> dict(accept_len, path_nodes, out_tokens, bonus, status)."""
    logits, dt = _logits_arg(logits)
    scores = np.ascontiguousarray(scores, np.float32)
    total, stride = logits.shape
    n_rows, sstride = scores.shape
    vocab = stride if vocab is None else vocab
    node_offsets, parent, tok, child_row = _i32(node_offsets), _i32(parent), _i32(tok), _i32(child_row)
    u_accept = np.ascontiguousarray(u_accept, np.float32)
    u_bonus = np.ascontiguousarray(u_bonus, np.float32)
    batch = node_offsets.shape[0] - 1
    r = dict(accept_len=np.zeros(batch, np.int32), path_nodes=np.zeros((batch, max_depth + 1), np.int32),
             out_tokens=np.zeros((batch, max_depth + 1), np.int32), bonus=np.zeros(batch, np.int32),
             status=np.zeros(batch, np.int32))
    _load().sbo_verify_sample(_p(logits), C.c_int(dt), C.c_int64(stride), C.c_int(vocab), _p(scores),
                              C.c_int64(sstride), C.c_int(n_rows), C.c_int(batch), _p(node_offsets), _p(parent),
                              _p(tok), _p(child_row), C.c_double(temperature), _p(u_accept), _p(u_bonus),
                              C.c_int(max_depth), _p(r["accept_len"]), _p(r["path_nodes"]), _p(r["out_tokens"]),
                              _p(r["bonus"]), _p(r["status"]))
    return r


def accept_from_amax(parent, tok, amax, max_depth):
    parent, tok, amax = _i32(parent), _i32(tok), _i32(amax)
    n = parent.shape[0]
    accept_len = np.zeros(1, np.int32)
    bonus = np.zeros(1, np.int32)
    path = np.zeros(max_depth + 1, np.int32)
    out = np.zeros(max_depth + 1, np.int32)
    rc = _load().sbo_accept_from_amax(C.c_int(n), _p(parent), _p(tok), _p(amax),
                                      C.c_int(max_depth), _p(accept_len), _p(path), _p(out),
                                      _p(bonus))
    return dict(accept_len=int(accept_len[0]), path_nodes=path, out_tokens=out,
                bonus=int(bonus[0]), status=int(rc))


def path_rows(node_offsets, node_row, path_nodes, accept_len, max_depth, row_begin=None):
    """node_row int32 [total_nodes]: the iteration-wide row that proposed each node (-1: root).
    -> dict(path_rows int32 [B, max_depth+1], status int32 [B])."""
    node_offsets, node_row = _i32(node_offsets), _i32(node_row)
    path_nodes, accept_len = _i32(path_nodes), _i32(accept_len)
    batch = node_offsets.shape[0] - 1
    rb = None if row_begin is None else _i32(row_begin)
    rows = np.zeros((batch, max_depth + 1), np.int32)
    status = np.zeros(batch, np.int32)
    _load().sbo_path_rows(C.c_int(batch), _p(node_offsets), _p(node_row), None if rb is None else _p(rb),
                          _p(path_nodes), _p(accept_len), C.c_int(max_depth), _p(rows), _p(status))
    return dict(path_rows=rows, status=status)


def kv_compact(*, n_kv_heads, head_dim, cache, n_layers, layer_stride_elems, page_size=0,
               max_pages=0, num_pages=0, kv_capacity=0, page_table=None, prefix_len,
               node_offsets, path_nodes, accept_len, max_depth):
    """cache: uint16 flat array holding all layers.  -> (new_cache, new_len, status)."""
    cache = np.ascontiguousarray(cache, np.uint16)
    new = cache.copy()
    prefix_len, node_offsets = _i32(prefix_len), _i32(node_offsets)
    path_nodes, accept_len, page_table = _i32(path_nodes), _i32(accept_len), _i32(page_table)
    batch = prefix_len.shape[0]
    new_len = np.zeros(batch, np.int32)
    status = np.zeros(batch, np.int32)
    _load().sbo_kv_compact(C.c_int(batch), C.c_int(n_kv_heads), C.c_int(head_dim), _p(cache),
                           _p(new), C.c_int(n_layers), C.c_int64(layer_stride_elems),
                           C.c_int(page_size), C.c_int(max_pages), C.c_int(num_pages),
                           C.c_int64(kv_capacity), _p(page_table), _p(prefix_len),
                           _p(node_offsets), _p(path_nodes), _p(accept_len), C.c_int(max_depth),
                           _p(new_len), _p(status))
    return new, new_len, status


def tree_expand(scores, block_k, bucket, bmap, start_parent, node_budget, tree=None, vocab=None):
    """tree: optional dict(tok, parent, depth, node_row, node_rank) of existing nodes.

    -> dict(n_nodes, tok, parent, depth, node_row, node_rank, topk_tok, topk_val, status).
    """
    scores = np.ascontiguousarray(scores, np.float32)
    n_rows, stride = scores.shape
    vocab = stride if vocab is None else vocab
    bucket = np.ascontiguousarray(bucket, np.uint8)
    bmap, start_parent = _i32(bmap), _i32(start_parent)
    arrs = {k: np.full(node_budget, -1, np.int32)
            for k in ("tok", "parent", "depth", "node_row", "node_rank")}
    n0 = 0
    if tree is not None:
        n0 = len(tree["tok"])
        for k in arrs:
            arrs[k][:n0] = tree[k]
    n_nodes = np.array([n0], np.int32)
    topk_tok = np.zeros((n_rows, KMAX), np.int32)
    topk_val = np.zeros((n_rows, KMAX), np.float32)
    rc = _load().sbo_tree_expand(_p(scores), C.c_int64(stride), C.c_int(n_rows), C.c_int(vocab),
                                 C.c_int(block_k), _p(bucket), _p(bmap), _p(start_parent),
                                 C.c_int(node_budget), _p(n_nodes), _p(arrs["tok"]),
                                 _p(arrs["parent"]), _p(arrs["depth"]), _p(arrs["node_row"]),
                                 _p(arrs["node_rank"]), _p(topk_tok), _p(topk_val))
    return dict(n_nodes=int(n_nodes[0]), topk_tok=topk_tok, topk_val=topk_val, status=int(rc),
                **arrs)
