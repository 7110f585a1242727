"""SpecBlock draft-and-verify hot path for NVIDIA B200 (sm_100a).

`paper_2605_07243_b200.binding` marshals torch tensors into the C-ABI library built from
`csrc/` (declared in include/specblock.h); `paper_2605_07243_b200.workloads` draws the seeded
synthetic inputs.  Importing the package loads neither torch nor the CUDA library.
"""
__all__ = ["binding", "workloads", "build"]
