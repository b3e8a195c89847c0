"""B200-native weight remap (trainer layout -> rollout layout) behind a small C ABI.

`binding` mirrors include/wb.h one to one; `device` holds the torch-side plumbing
(device memory for the virtual ranks, streams).  The package has no CPU fallback: it
needs libwb.so, built in-tree by `build.build()`.
"""
from . import binding
from .binding import (Layout, Plan, WbError, wb_layout_describe, wb_plan_build, wb_version,
                      wb_launches_per_call)

__all__ = ["binding", "Layout", "Plan", "WbError", "wb_layout_describe", "wb_plan_build",
           "wb_version", "wb_launches_per_call"]
