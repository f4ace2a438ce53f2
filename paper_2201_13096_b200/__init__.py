"""Batched SPDY dynamic program on B200 (sm_100a): Python binding over a C-ABI CUDA library.

``workloads`` (seeded synthetic inputs) imports without a GPU.  The solver entry points live in
``binding`` and load ``libspdy_dp.so`` on first use; they raise if it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
