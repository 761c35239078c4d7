"""TEAM MoE-layer hot path for NVIDIA B200 (sm_100a): C-ABI CUDA library + thin ctypes binding.

`binding` mirrors include/team.h; `workloads` holds the seeded synthetic inputs; `build` compiles
the library in-tree.  Importing the package does not load the library; the first call does, and
raises if it is missing.
"""
__all__ = ["binding", "workloads", "build"]
