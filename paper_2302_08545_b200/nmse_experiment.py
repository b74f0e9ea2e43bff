"""NMSE of the decompressed average against the granularity g, per index width b: the shape of
the paper's granularity study (Section 8.5 / Appendix D: error falls as g grows and by about an
order of magnitude per extra bit), on synthetic lognormal gradients that stand in for the
paper's training gradients.

    python -m paper_2302_08545_b200.nmse_experiment [--log2-d 22] [--workers 10] [--p 0.0009765625]

Every point builds the optimal lookup table for (b, g, p) with the solver of tables.py
(Section 5.2), runs one full round of the library on the GPU (scales, compress, aggregate,
decompress) and reports  NMSE = ||out - mean_i x_i||^2 / ||mean_i x_i||^2 for 2, 3 and 4 bits
per index (the paper's three curves).  One JSON line per point.
"""
from __future__ import annotations

import argparse
import json

from . import tables
from .workloads import Workload

DEFAULT_POINTS = {2: (3, 4, 5, 6, 8, 10), 3: (7, 8, 10, 12, 14, 18, 22), 4: (15, 18, 22, 26, 30, 36, 44, 52)}


def lognormal_gradients(n: int, d: int, seed: int, device):
    """n vectors of d coordinates: random sign times exp(N(-7, 1)), plus a component common to
    all workers (so that the average is not just noise).  Seeded; generated on the device."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    common = torch.randn(d, generator=gen, device=device).mul_(1.0).add_(-7.0).exp_()
    common.mul_(torch.randint(0, 2, (d,), generator=gen, device=device, dtype=torch.int8).float().mul_(2).sub_(1))
    out = []
    for _ in range(n):
        own = torch.randn(d, generator=gen, device=device).add_(-7.0).exp_()
        own.mul_(torch.randint(0, 2, (d,), generator=gen, device=device, dtype=torch.int8).float().mul_(2).sub_(1))
        out.append((common + own).contiguous())
    return out


def nmse_point(bits: int, g: int, p: float, grads, log2_block: int = 20, rnd: int = 0) -> float:
    import torch
    from . import runner
    n, d = len(grads), grads[0].numel()
    table, _ = tables.optimal_table(bits, g, p)
    w = Workload(f"nmse_b{bits}_g{g}", n=n, d=d, log2_block=log2_block, bits=bits, granularity=g,
                 table=tuple(table), in_dtype="f32", data_seed=0, t_p=tables.t_p(p))
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d, device=str(grads[0].device))
    for dst, src in zip(r.grads, grads):
        dst.copy_(src)
    r.run(rnd, fused=True)
    torch.cuda.synchronize()
    mean = torch.zeros(d, dtype=torch.float64, device=grads[0].device)
    for gsrc in grads:
        mean += gsrc.double()
    mean /= n
    err = (r.out.double() - mean).pow(2).sum().item()
    return err / mean.pow(2).sum().item()


def run(points=None, log2_d: int = 22, workers: int = 10, p: float = 1.0 / 1024, seed: int = 77):
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    grads = lognormal_gradients(workers, 1 << log2_d, seed, dev)
    rows = []
    for bits, gs in sorted((points or DEFAULT_POINTS).items()):
        for g in gs:
            rows.append({"bits": bits, "granularity": g, "p": p, "workers": workers, "d": 1 << log2_d,
                         "nmse": nmse_point(bits, g, p, grads)})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--log2-d", type=int, default=22)
    ap.add_argument("--workers", type=int, default=10)
    ap.add_argument("--p", type=float, default=1.0 / 1024)
    a = ap.parse_args()
    for row in run(None, a.log2_d, a.workers, a.p):
        print(json.dumps(row), flush=True)


if __name__ == "__main__":
    main()
