"""GoodSpeed verification hot path for NVIDIA B200 (sm_100a).

The compute lives in a C-ABI CUDA library (csrc/, declared in include/goodspeed.h);
`binding` marshals torch device pointers into it and `workloads` makes seeded
synthetic inputs.  Importing the package does not load the library; the first
call through `binding` does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
