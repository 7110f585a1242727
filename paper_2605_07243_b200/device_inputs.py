"""Host arrays of `workloads` -> CUDA tensors and `binding.TreeBatch` (copies only)."""
from __future__ import annotations

import numpy as np
import torch

from .binding import TreeBatch


def bf16_tensor(bits: np.ndarray, device="cuda", pin=False) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor of the same shape on `device`."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if pin:
        t = t.pin_memory()
    return t.to(device, non_blocking=pin)


def i32_tensor(a, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, np.int32)).to(device)


def tree_batch(case, device="cuda", k=None, v=None) -> TreeBatch:
    """Upload an AttnCase.  k / v: already-uploaded cache tensors to reuse."""
    return TreeBatch(
        n_q_heads=case.n_q_heads, n_kv_heads=case.n_kv_heads, head_dim=case.head_dim,
        k_cache=bf16_tensor(case.k, device) if k is None else k,
        v_cache=bf16_tensor(case.v, device) if v is None else v,
        prefix_len=i32_tensor(case.prefix_len, device),
        node_offsets=i32_tensor(case.node_offsets, device),
        parent=i32_tensor(case.parent, device),
        total_nodes=int(case.node_offsets[-1]), max_nodes=case.max_nodes,
        max_kv_len=case.max_kv_len, page_size=case.page_size, kv_capacity=case.kv_capacity,
        page_table=None if case.page_table is None else i32_tensor(case.page_table, device),
        num_pages=case.num_pages, max_pages=case.max_pages)


def attention_args(case, device="cuda"):
    """-> (TreeBatch, q tensor, kwargs for binding.sb_tree_attention)."""
    tb = tree_batch(case, device)
    q = bf16_tensor(case.q, device)
    kw = dict(scale=float(case.scale))
    if case.q_node_begin is not None:
        kw["q_node_begin"] = i32_tensor(case.q_node_begin, device)
        kw["q_offsets"] = i32_tensor(case.q_offsets, device)
    return tb, q, kw
