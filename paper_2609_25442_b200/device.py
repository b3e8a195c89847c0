"""Torch-side plumbing: device memory for the virtual ranks and plan binding.

PyTorch is used for allocation and streams only.  Every virtual rank of a side gets one
arena (a single device allocation); its local tensors are carved from it at 256-byte
boundaries, so the ranks are separate regions of the GPU's memory.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np
import torch

from . import binding as wb

_TORCH = {wb.WB_F32: torch.float32, wb.WB_BF16: torch.bfloat16}
_SIZE = {wb.WB_F32: 4, wb.WB_BF16: 2}


def require_cuda() -> torch.device:
    if not torch.cuda.is_available():
        raise RuntimeError("the weight-remap executors need a CUDA device (sm_100a); none is visible")
    return torch.device("cuda", torch.cuda.current_device())


class RankArenas:
    """Device memory of one side: one arena per virtual rank, tensors carved at 256 B."""

    def __init__(self, tensors: np.ndarray, device, fill_byte: int | None = None, align: int = 256):
        self.device = device
        ranks = sorted(set(int(t["rank"]) for t in tensors))
        offs: Dict[int, int] = {r: 0 for r in ranks}
        place = []
        for t in tensors:
            r = int(t["rank"])
            nbytes = int(t["numel"]) * _SIZE[int(t["dtype"])]
            place.append((r, offs[r], nbytes))
            offs[r] += (nbytes + align - 1) // align * align
        self.arenas: Dict[int, torch.Tensor] = {}
        for r in ranks:
            a = torch.empty(max(offs[r], align), dtype=torch.uint8, device=device)
            if fill_byte is not None:
                a.fill_(fill_byte)
            self.arenas[r] = a
        self.tensors: List[torch.Tensor] = []
        for t, (r, off, nbytes) in zip(tensors, place):
            view = self.arenas[r][off:off + nbytes].view(_TORCH[int(t["dtype"])])
            self.tensors.append(view)

    def pointers(self) -> List[int]:
        return [t.data_ptr() for t in self.tensors]

    def total_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.tensors)


def bind(plan: wb.Plan, src: RankArenas | Sequence[torch.Tensor], dst: RankArenas | Sequence[torch.Tensor]) -> None:
    """Bind a plan to device tensors (anything with data_ptr())."""
    s = src.tensors if isinstance(src, RankArenas) else src
    d = dst.tensors if isinstance(dst, RankArenas) else dst
    plan.bind([t.data_ptr() for t in s], [t.data_ptr() for t in d])


def current_stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream
