"""Helpers for the GPU parity tests: put a workload on the device, run the library through
its C ABI, bring results back as raw bits."""
import numpy as np
import torch

from helpers import ckpt_shapes, to_bits
from oracle import remap_oracle
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200.device import RankArenas, bind

CANARY = 0xCD


class DeviceCase:
    """A workload resident on the GPU: trainer arenas filled by the procedural
    load_weights from seeded checkpoint values, rollout arenas pre-filled with a canary."""

    def __init__(self, wl, device, values=None, trainer=None, rollout=None, **plan_opts):
        self.wl = wl
        self.device = device
        self.trainer = trainer if trainer is not None else wl.trainer
        self.rollout = rollout if rollout is not None else wl.rollout
        self.src = RankArenas(self.trainer.tensors, device, fill_byte=0)
        self.dst = RankArenas(self.rollout.tensors, device, fill_byte=CANARY)
        self.load_trainer(values or (lambda i: wl.ckpt_values(i, device)))
        self.plan = wb.Plan(wb.Layout(self.trainer.tensors, self.trainer.slices),
                            wb.Layout(self.rollout.tensors, self.rollout.slices), **plan_opts)
        bind(self.plan, self.src, self.dst)

    def load_trainer(self, values):
        def sink(k, t):
            self.src.tensors[k].copy_(t.to(self.src.tensors[k].dtype) if t.dtype != self.src.tensors[k].dtype else t)
        self.wl.load_side("trainer", values, sink)

    def reset_dst(self):
        for a in self.dst.arenas.values():
            a.fill_(CANARY)

    def src_bits(self):
        return [to_bits(t) for t in self.src.tensors]

    def dst_bits(self):
        return [to_bits(t) for t in self.dst.tensors]

    def gaps_intact(self):
        """Bytes of the rollout arenas outside every local tensor still hold the canary."""
        for r, arena in self.dst.arenas.items():
            mask = torch.ones(arena.numel(), dtype=torch.bool, device=arena.device)
            base = arena.data_ptr()
            for t, d in zip(self.dst.tensors, self.rollout.tensors):
                if int(d["rank"]) == r:
                    off = t.data_ptr() - base
                    mask[off:off + t.numel() * t.element_size()] = False
            if not bool((arena[mask] == CANARY).all()):
                return False
        return True


def prefill_bits(rollout, dtype_bits):
    pat = CANARY | (CANARY << 8)
    if dtype_bits == np.uint32:
        pat |= pat << 16
    return [np.full(int(t["numel"]), pat, dtype_bits) for t in rollout.tensors]


def oracle_for(case: DeviceCase):
    """The CPU oracle's rollout tensors for the trainer bits a case holds on the device."""
    bits = np.uint32 if case.dst.tensors[0].dtype == torch.float32 else np.uint16
    return remap_oracle(ckpt_shapes(case.wl), case.trainer.tensors, case.trainer.slices,
                        case.rollout.tensors, case.rollout.slices, case.src_bits(),
                        prefill_bits(case.rollout, bits))
