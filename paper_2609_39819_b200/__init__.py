"""B200-native hot path of a lifecycle-aware KV cache engine for ReAct agents: block hashing,
GPU block-table lookup, lifecycle classification, state-prioritised victim selection and paged KV
movement, behind the C ABI declared in include/kvt.h.

Submodules: `build` (compiles libkvt.so with nvcc for sm_100a), `binding` (ctypes front end; needs
a CUDA device), `workloads` (seeded synthetic traces and the replay driver; numpy only).
"""
__all__ = ["build", "binding", "workloads"]
