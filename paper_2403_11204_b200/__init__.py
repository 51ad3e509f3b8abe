"""Segment training with synthetic intermediate labels on NVIDIA B200 (sm_100a).

`binding` exposes the C ABI of libsegtrain.so (include/seg.h); `workloads` describes the
synthetic workloads; `build` compiles the library in-tree.
"""
__all__ = ["binding", "workloads", "build"]
