"""Buffer management around the C-ABI calls: allocate a round's device buffers with torch
and issue prepare / compress / aggregate / decompress in order.  No arithmetic here."""
from __future__ import annotations

import numpy as np
import torch

from . import thc
from .workloads import Workload


def context_for(w: Workload, workers: int | None = None, acc_bits: int = 0,
                exact_range: bool = False) -> thc.Context:
    return thc.Context(bits=w.bits, granularity=w.granularity, table=w.table, t_p=w.t_p,
                       log2_block=w.log2_block, seed=w.seed,
                       in_dtype=thc.THC_BF16 if w.in_dtype == "bf16" else thc.THC_F32,
                       workers=w.n if workers is None else workers, acc_bits=acc_bits,
                       range_mode=1 if exact_range else 0)


class Round:
    """Device buffers of one simulated cluster: n gradient buffers in one GPU's memory."""

    def __init__(self, ctx: thc.Context, n: int, d: int, in_dtype: str = "f32",
                 device: str = "cuda:0", want_rotated: bool = False):
        self.ctx, self.n, self.d = ctx, n, d
        self.sz = ctx.sizes(d, n)
        dev = torch.device(device)
        self.device = dev
        gdt = torch.float32 if in_dtype == "f32" else torch.bfloat16
        self.grads = [torch.zeros(d, dtype=gdt, device=dev) for _ in range(n)]
        self.scales = torch.zeros(self.sz.scales_count, dtype=torch.float32, device=dev)
        self.packed = [torch.zeros(self.sz.packed_bytes, dtype=torch.uint8, device=dev)
                       for _ in range(n)]
        self.total = torch.zeros(self.sz.sum_bytes, dtype=torch.uint8, device=dev)
        self.out = torch.zeros(d, dtype=torch.float32, device=dev)
        self.workspace = torch.zeros(self.sz.workspace_bytes, dtype=torch.uint8, device=dev)
        self.rotated = ([torch.zeros(self.sz.d_pad, dtype=torch.float32, device=dev)
                         for _ in range(n)] if want_rotated else None)

    # -- host <-> device helpers (copies only)
    def upload(self, x: np.ndarray):
        """x: [n, d] float32, or uint16 bf16 bit patterns for bf16 contexts."""
        for i in range(self.n):
            t = torch.from_numpy(np.ascontiguousarray(x[i]))
            if self.grads[i].dtype == torch.bfloat16:
                t = t.view(torch.int16).view(torch.bfloat16) if t.dtype != torch.bfloat16 else t
            self.grads[i].copy_(t)

    def sum_numpy(self) -> np.ndarray:
        dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[self.sz.acc_bits]
        return self.total.cpu().numpy().view(dt)

    # -- the four calls
    def prepare(self, stream=None):
        self.ctx.prepare(self.grads, self.d, self.scales, self.workspace, stream)

    def prepare_minmax(self, rnd: int = 0, stream=None):
        self.ctx.prepare_minmax(self.grads, self.d, rnd, self.scales, self.workspace,
                                rotated=self.rotated, stream=stream)

    def compress(self, rnd: int = 0, stream=None):
        self.ctx.compress(self.grads, self.d, rnd, self.scales, self.packed, self.workspace,
                          rotated=self.rotated, stream=stream)

    def prepare_compress(self, rnd: int = 0, stream=None):
        self.ctx.prepare_compress(self.grads, self.d, rnd, self.scales, self.packed, self.workspace,
                                  rotated=self.rotated, stream=stream)

    def quantize_rotated(self, rnd: int = 0, stream=None):
        self.ctx.quantize_rotated(self.rotated, self.d, rnd, self.scales, self.packed, stream=stream)

    def aggregate(self, stream=None):
        self.ctx.aggregate(self.packed, self.d, self.total, stream)

    def decompress(self, rnd: int = 0, stream=None):
        self.ctx.decompress(self.total, self.n, self.d, rnd, self.scales, self.out,
                            self.workspace, stream)

    def aggregate_decompress(self, rnd: int = 0, want_sums: bool = False, stream=None):
        self.ctx.aggregate_decompress(self.packed, self.d, rnd, self.scales, self.out, self.workspace,
                                      total=self.total if want_sums else None, stream=stream)

    def run(self, rnd: int = 0, with_prepare: bool = True, stream=None, fused: bool = False):
        if with_prepare and fused:
            self.prepare_compress(rnd, stream)
        else:
            if with_prepare:
                self.prepare(stream)
            self.compress(rnd, stream)
        self.aggregate(stream)
        self.decompress(rnd, stream)
