"""CPU fp64 oracle of the SpecBlock device steps -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares no code with the CUDA library and never imports it.
"""
from .oracle import (  # noqa: F401
    build,
    num_threads,
    tree_ancestors,
    tree_attention,
    row_argmax,
    row_topk,
    rank_features,
    verify_accept,
    verifier_signal,
    verify_sample,
    shift_project,
    fuse_project,
    accept_from_amax,
    kv_compact,
    path_rows,
    tree_expand,
)
