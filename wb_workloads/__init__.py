"""Seeded synthetic workloads for the weight-remap path.

This package only *describes inputs*: checkpoint tensor tables, the trainer and
rollout source maps (lists of slice-copy operations, Section 3.1 of the paper),
procedural ``load_weights`` functions written with tensor ops, and seeded weight
values.  It holds none of the method's arithmetic (no correspondence, no
de-duplication, no planning, no cast), so both the CPU oracle and the CUDA
library can be fed from it without sharing code with each other.
"""
from .types import (SLICE_DTYPE, TENSOR_DTYPE, WB_F32, WB_BF16, CkptTensor,
                    Layout, Workload, dtype_size)
from .configs import make_workload, CONFIG_NAMES
from .rng import SplitMix64

__all__ = ["SLICE_DTYPE", "TENSOR_DTYPE", "WB_F32", "WB_BF16", "CkptTensor",
           "Layout", "Workload", "dtype_size", "make_workload", "CONFIG_NAMES",
           "SplitMix64"]
