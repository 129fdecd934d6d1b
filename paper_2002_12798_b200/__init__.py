"""Composed affine copies on B200: compose a chain of layout operators into one
affine access map on the host and run it as a single CUDA copy kernel.

The CUDA/C++ library is loaded lazily by `paper_2002_12798_b200.binding`;
`paper_2002_12798_b200.workloads` (plain data) imports without it.
"""
__all__ = ["binding", "workloads"]
