"""MAGE per-block sparse-attention hot path for NVIDIA B200 (sm_100a).

The compute lives in ``libmage.so`` (hand-written CUDA behind a C ABI, declared
in ``include/mage.h``); :mod:`paper_2602_14209_b200.binding` marshals torch
tensors into it.  Importing this package does not load the library; the first
call does, and raises if it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
