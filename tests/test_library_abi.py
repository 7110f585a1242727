"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every symbol that
include/specblock.h declares.  No compute call is made here."""
import ctypes
import os
import re

from paper_2605_07243_b200 import binding, build


def _declared_symbols():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "specblock.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sb_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    path = build.build()
    lib = ctypes.CDLL(path)
    declared = _declared_symbols()
    assert "sb_tree_attention" in declared and "sb_kv_compact" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in specblock.h but not exported"
    assert set(binding.EXPORTED) == set(declared)


def test_host_only_entry_points():
    lib = binding.load()
    assert binding.sb_version() >= 100
    assert binding.sb_status_string(0) == "ok"
    assert binding.sb_status_string(4) == "invalid tree"
    assert binding.sb_kernel_launch_count() >= 0
    # workspace queries are host arithmetic
    assert binding.sb_verify_accept_workspace_bytes(60, 128256) > 0
    assert binding.sb_tree_expand_workspace_bytes(32, 128256) > 0
    assert lib.sb_tree_attention_workspace_bytes(None, 1, 0) == 0
    # every other query: positive and 256-byte granular for valid shapes, 0 for shapes the call refuses
    expand = binding.sb_tree_expand_workspace_bytes(32, 128256)
    feats = binding.sb_rank_features_workspace_bytes(32, 128256)
    assert feats > expand and expand % 256 == 0 and feats % 256 == 0          # the fused call uses the larger one
    assert binding.sb_tree_expand_workspace_bytes(0, 128256) == 0
    sample = binding.sb_verify_sample_workspace_bytes(2, 128256, 120, 36)
    assert sample >= 2 * 128256 * 4 and sample % 256 == 0                      # a residual row per sequence + statistics
    assert binding.sb_verify_sample_workspace_bytes(2, 128256, 0, 36) == 0
    shift = binding.sb_shift_project_workspace_bytes(32, 4096, 4096, 4)
    plain = binding.sb_shift_project_workspace_bytes(32, 4096, 4096, 0)
    assert shift >= plain > 0 and shift % 256 == 0                             # fp32 partials of the K splits + a word
    assert binding.sb_shift_project_workspace_bytes(32, 4000, 4096, 4) == 0    # d not a multiple of 64
    assert binding.sb_shift_project_workspace_bytes(129, 4096, 4096, 4) == 0   # more than 128 rows
    fuse3 = binding.sb_fuse_project_workspace_bytes(8, 4, 4096, 4096, False)
    fuse2 = binding.sb_fuse_project_workspace_bytes(8, 4, 4096, 4096, True)
    assert fuse3 > fuse2 > 0                                                   # the cached query term saves a third
    assert binding.sb_fuse_project_workspace_bytes(8, 4, 4096, 100, False) == 0


def test_binding_struct_matches_header_layout():
    """Field order and natural alignment of the ctypes mirror of sb_tree_batch."""
    s = binding._TreeBatch
    names = [f[0] for f in s._fields_]
    assert names == ["batch", "n_q_heads", "n_kv_heads", "head_dim", "k_cache", "v_cache",
                     "page_size", "max_pages", "kv_capacity", "num_pages", "total_nodes",
                     "page_table", "prefix_len", "node_offsets", "parent", "max_nodes",
                     "max_kv_len", "index_arrays_settled", "prefix_rows_settled"]
    assert s.k_cache.offset == 16 and s.kv_capacity.offset == 40 and s.page_table.offset == 56
    assert s.max_nodes.offset == 88 and s.index_arrays_settled.offset == 96
    assert ctypes.sizeof(s) == 104


def _test_header_symbols():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "specblock_test.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sb_[a-z_]+)\s*\(", text)))


def test_build_variants_export_their_hooks_and_the_library_proper_does_not():
    """libspecblock_test.so / libspecblock_checked.so: the same ABI plus the hooks of specblock_test.h.
    The library proper exports none of the hooks, holds no check kernel and reads no environment."""
    hooks = _test_header_symbols()
    assert hooks == ["sb_checked_selftest", "sb_checked_violations", "sb_test_wait_expires"]
    proper = ctypes.CDLL(build.build())
    test = ctypes.CDLL(build.build(variant="test"))
    checked = ctypes.CDLL(build.build(variant="checked"))
    for name in _declared_symbols():
        assert hasattr(test, name) and hasattr(checked, name), name
    for name in hooks:
        assert not hasattr(proper, name), f"{name} must not be in the library proper"
    assert hasattr(test, "sb_test_wait_expires") and not hasattr(test, "sb_checked_violations")
    assert hasattr(checked, "sb_checked_violations") and hasattr(checked, "sb_checked_selftest")
    # the only getenv of the sources is the test build's switch reader
    csrc = os.path.join(os.path.dirname(build.__file__), "csrc")
    uses = [(f, i + 1) for f in sorted(os.listdir(csrc)) for i, line in enumerate(open(os.path.join(csrc, f)))
            if "getenv" in line]
    assert uses == [("common.cuh", uses[0][1])], uses
    common = open(os.path.join(csrc, "common.cuh")).read()
    assert common.index("#ifdef SB_TEST_KERNELS") < common.index("getenv") < common.index("#else", common.index("getenv") - 200)
