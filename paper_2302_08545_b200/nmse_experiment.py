"""NMSE of the decompressed average against the granularity g, per index width b: the shape of
the paper's granularity study (Section 8.5 / Appendix D: error falls as g grows and by about an
order of magnitude per extra bit), on synthetic lognormal gradients that stand in for the
paper's training gradients.

    python -m paper_2302_08545_b200.nmse_experiment [--log2-d 22] [--workers 10] [--p 0.0009765625]
                                                   [--protocol paper|signed|mixed] [--repeats 10]

Protocols.  `paper` is Appendix D's: one lognormal vector (exp of a standard normal: all
coordinates positive) copied to every worker, the NMSE averaged over repeats with a fresh vector,
rotation and rounding draws each; `signed` is the same with a random sign per coordinate;
`mixed` gives every worker its own lognormal vector on top of a common one (one round).

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


def copied_gradient(n: int, d: int, seed: int, device, signed: bool):
    """Appendix D's input: one lognormal vector, the same for all n workers (the list holds the
    same tensor n times: the library only reads it)."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    x = torch.randn(d, generator=gen, device=device).exp_()
    if signed:
        x.mul_(torch.randint(0, 2, (d,), generator=gen, device=device, dtype=torch.int8).float().mul_(2).sub_(1))
    return [x.contiguous()] * n


def nmse_point(bits: int, g: int, p: float, grads, log2_block: int = 20, rnd: int = 0) -> float:
    import torch
    from . import runner
    n, d = len(grads), grads[0].numel()
    table, _ = tables.optimal_table(bits, g, p)
    w = Workload(f"nmse_b{bits}_g{g}", n=n, d=d, log2_block=log2_block, bits=bits, granularity=g,
                 table=tuple(table), in_dtype="f32", data_seed=0, t_p=tables.t_p(p))
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d, device=str(grads[0].device))
    if all(gsrc is grads[0] for gsrc in grads):
        r.grads[0].copy_(grads[0])
        r.grads = [r.grads[0]] * n                       # one buffer read n times
    else:
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


def run(points=None, log2_d: int = 22, workers: int = 10, p: float = 1.0 / 1024, seed: int = 77,
        protocol: str = "mixed", repeats: int = 1):
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    d = 1 << log2_d
    rows = []
    reps = 1 if protocol == "mixed" else repeats
    inputs = [lognormal_gradients(workers, d, seed, dev)] if protocol == "mixed" else \
        [copied_gradient(workers, d, seed + rep, dev, protocol == "signed") for rep in range(reps)]
    for bits, gs in sorted((points or DEFAULT_POINTS).items()):
        for g in gs:
            vals = [nmse_point(bits, g, p, grads, rnd=rep) for rep, grads in enumerate(inputs)]
            rows.append({"bits": bits, "granularity": g, "p": p, "workers": workers, "d": d,
                         "protocol": protocol, "repeats": reps, "nmse": sum(vals) / len(vals)})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--log2-d", type=int, default=22)
    ap.add_argument("--workers", type=int, default=10)
    ap.add_argument("--p", type=float, default=1.0 / 1024)
    ap.add_argument("--protocol", default="paper", choices=["paper", "signed", "mixed"])
    ap.add_argument("--repeats", type=int, default=10)
    a = ap.parse_args()
    for row in run(None, a.log2_d, a.workers, a.p, protocol=a.protocol, repeats=a.repeats):
        print(json.dumps(row), flush=True)


if __name__ == "__main__":
    main()
