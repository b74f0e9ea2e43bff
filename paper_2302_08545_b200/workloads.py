"""Seeded synthetic gradients and the parameter sets they are compressed with.

This module serves both the CUDA path and the CPU oracle, so it holds no arithmetic of the
method: only random inputs, shapes, and constants that are inputs to the method (lookup
tables, truncation thresholds).  It imports neither of them.

The gradients stand in for the real training gradients the THC paper measured on
(ImageNet / SST2 models): same sizes and segment structure as ResNet-50, VGG-16 and
GPT-2-medium parameter vectors, with the value distributions the benchmark definition
names.  NumPy ``Generator(PCG64)``; worker streams come from ``SeedSequence(seed).spawn``.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

THC_SEED = 0x0123456789ABCDEF

# t_p = Phi^-1(1 - p/2) (Section 5.2 of the THC paper) for the p values the paper uses.
T_P = {
    "1/32": 2.1538746940614564,
    "1/512": 3.0972690781987846,
    "1/1024": 3.2971933456919635,
}

# Lookup tables T_{b,g,p}: inputs to the method.  The identity tables are uniform THC
# (Section 4.2).  The (4, 30, 1/32) table is the minimiser of the Section 5.2 objective
# for the paper's prototype setting (b=4, g=30, p=1/32); tests re-derive it.
TABLES = {
    (1, 1): (0, 1),
    (2, 3): (0, 1, 2, 3),
    (2, 4): (0, 1, 3, 4),            # the paper's worked example T_2 (Section 4.3)
    (4, 15): tuple(range(16)),
    (4, 30): (0, 3, 5, 7, 9, 11, 13, 14, 15, 17, 19, 21, 23, 25, 27, 30),
    (8, 255): tuple(range(256)),
}


@dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration."""
    name: str
    n: int                     # simulated workers
    d: int                     # gradient elements per worker
    log2_block: int            # RHT block = 2^log2_block
    bits: int                  # b
    granularity: int           # g
    table: tuple
    t_p: float = T_P["1/32"]
    in_dtype: str = "f32"      # "f32" or "bf16"
    data_seed: int = 1000
    seed: int = THC_SEED
    segments: tuple = field(default=(), compare=False)   # (size, scale) description

    @property
    def block(self) -> int:
        return 1 << self.log2_block

    @property
    def d_pad(self) -> int:
        return -(-self.d // self.block) * self.block

    @property
    def nblocks(self) -> int:
        return self.d_pad // self.block

    @property
    def acc_bits(self) -> int:
        for w in (8, 16, 32):
            if self.n * self.granularity <= (1 << w) - 1:
                return w
        raise ValueError("n*g too large")

    def algorithmic_bytes(self) -> dict:
        """Bytes each step must move if every input is read once and every output is
        written once (intermediates excluded)."""
        s_in = 4 if self.in_dtype == "f32" else 2
        n, dp, b, w = self.n, self.d_pad, self.bits, self.acc_bits
        compress = n * dp * s_in + n * dp * b // 8
        aggregate = n * dp * b // 8 + dp * w // 8
        decompress = dp * w // 8 + 4 * dp
        prepare = n * dp * s_in
        return {"prepare": prepare, "compress": compress, "aggregate": aggregate,
                "decompress": decompress, "round": compress + aggregate + decompress}


def _f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16). A dtype
    conversion of the inputs, not a step of the method."""
    u = a.astype(np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def _worker_rngs(seed: int, n: int):
    return [np.random.Generator(np.random.PCG64(s)) for s in np.random.SeedSequence(seed).spawn(n)]


# --------------------------------------------------------------------------------------
# Generators.  Each returns an [n, d] array (float32, or uint16 bf16 bit patterns).
# --------------------------------------------------------------------------------------
def gen_outlier_normal(n: int, d: int, seed: int, sigma=1e-3, frac=1e-3, sigma_out=1e-1):
    """iid N(0, sigma^2) with a fixed fraction of coordinates replaced by N(0, sigma_out^2)."""
    out = np.empty((n, d), dtype=np.float32)
    n_out = int(round(frac * d))
    for i, rng in enumerate(_worker_rngs(seed, n)):
        x = rng.standard_normal(d, dtype=np.float32) * np.float32(sigma)
        pos = rng.choice(d, size=n_out, replace=False)
        x[pos] = rng.standard_normal(n_out, dtype=np.float32) * np.float32(sigma_out)
        out[i] = x
    return out


def resnet50_like_segments(d: int, seed: int, count=161):
    """161 layer segments with lognormal sizes and lognormal per-segment scales."""
    rng = np.random.Generator(np.random.PCG64(seed + 7))
    raw = rng.lognormal(0.0, 1.5, size=count)
    sizes = np.maximum(1, np.floor(raw / raw.sum() * d)).astype(np.int64)
    sizes[np.argmax(sizes)] += d - sizes.sum()
    assert sizes.sum() == d and sizes.min() >= 1
    scales = rng.lognormal(np.log(1e-3), 1.0, size=count)
    return sizes, scales


def gen_segmented_normal(n: int, sizes, scales, seed: int):
    d = int(np.sum(sizes))
    out = np.empty((n, d), dtype=np.float32)
    per_elem = np.repeat(np.asarray(scales, dtype=np.float32), sizes)
    for i, rng in enumerate(_worker_rngs(seed, n)):
        out[i] = rng.standard_normal(d, dtype=np.float32)
        out[i] *= per_elem
    return out


def vgg16_like_segments(d: int = 138_357_544):
    """16 segments; the three FC-shaped ones (89 % of the elements) come last."""
    fc = [102_764_544, 16_781_312, 4_097_000]
    rest = d - sum(fc)
    ratios = np.geomspace(1.0, 64.0, 13)
    conv = np.floor(ratios / ratios.sum() * rest).astype(np.int64)
    conv[-1] += rest - conv.sum()
    return np.concatenate([conv, np.asarray(fc, dtype=np.int64)])


def gen_laplace(n: int, d: int, seed: int, scale=5e-4):
    out = np.empty((n, d), dtype=np.float32)
    for i, rng in enumerate(_worker_rngs(seed, n)):
        out[i] = rng.laplace(0.0, scale, size=d).astype(np.float32)
    return out


def gen_student_t_bf16(n: int, d: int, seed: int, nu=3.0, scale=1e-4, chunk=1 << 24):
    out = np.empty((n, d), dtype=np.uint16)
    for i, rng in enumerate(_worker_rngs(seed, n)):
        for lo in range(0, d, chunk):
            hi = min(d, lo + chunk)
            x = (rng.standard_t(nu, size=hi - lo) * scale).astype(np.float32)
            out[i, lo:hi] = _f32_to_bf16_bits(x)
    return out


def gen_standard_normal(n: int, d: int, seed: int):
    out = np.empty((n, d), dtype=np.float32)
    for i, rng in enumerate(_worker_rngs(seed, n)):
        out[i] = rng.standard_normal(d, dtype=np.float32)
    return out


# --------------------------------------------------------------------------------------
# The five benchmark configurations.
# --------------------------------------------------------------------------------------
def config1() -> Workload:
    return Workload("cfg1_outlier_normal", n=4, d=65_536, log2_block=16, bits=4,
                    granularity=30, table=TABLES[(4, 30)], data_seed=1001)


def config2() -> Workload:
    return Workload("cfg2_resnet50", n=8, d=25_557_032, log2_block=20, bits=4,
                    granularity=30, table=TABLES[(4, 30)], data_seed=1002)


def config3(bits: int = 4) -> Workload:
    g = 30 if bits == 4 else 3
    return Workload(f"cfg3_vgg16_b{bits}", n=8, d=138_357_544, log2_block=20, bits=bits,
                    granularity=g, table=TABLES[(bits, g)], data_seed=1003)


def config4() -> Workload:
    return Workload("cfg4_gpt2m_bf16", n=16, d=355_000_000, log2_block=22, bits=4,
                    granularity=30, table=TABLES[(4, 30)], in_dtype="bf16", data_seed=1004)


SWEEP_G = {1: 1, 2: 3, 4: 30, 8: 255}


def sweep_point(d: int, bits: int, n: int) -> Workload:
    g = SWEEP_G[bits]
    return Workload(f"sweep_d{d}_b{bits}_n{n}", n=n, d=d, log2_block=20, bits=bits,
                    granularity=g, table=TABLES[(bits, g)], data_seed=1005)


def sweep_points():
    for d in (1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28):
        for bits in (1, 2, 4, 8):
            for n in (2, 4, 8, 16, 32):
                yield sweep_point(d, bits, n)


def generate(w: Workload, d_limit: int | None = None) -> np.ndarray:
    """Materialise a workload's gradients on the host.  ``d_limit`` truncates to the first
    d_limit coordinates (a prefix of the same random streams is NOT guaranteed; it is a
    smaller workload of the same recipe)."""
    d = w.d if d_limit is None else min(w.d, d_limit)
    if w.name.startswith("cfg1"):
        return gen_outlier_normal(w.n, d, w.data_seed)
    if w.name.startswith("cfg2"):
        sizes, scales = resnet50_like_segments(d, w.data_seed)
        return gen_segmented_normal(w.n, sizes, scales, w.data_seed)
    if w.name.startswith("cfg3"):
        return gen_laplace(w.n, d, w.data_seed)
    if w.name.startswith("cfg4"):
        return gen_student_t_bf16(w.n, d, w.data_seed)
    return gen_standard_normal(w.n, d, w.data_seed)


def scaled(w: Workload, d: int, n: int | None = None, log2_block: int | None = None) -> Workload:
    """Same recipe at a smaller size (for parity tests the oracle finishes in seconds)."""
    from dataclasses import replace
    return replace(w, d=d, n=w.n if n is None else n,
                   log2_block=w.log2_block if log2_block is None else log2_block)


# --------------------------------------------------------------------------------------
# Large workloads, generated in place on the GPU (the NumPy recipes above take minutes for
# 10^9..10^10 samples).  Same sizes and distributions, seeded torch generators; used by the
# full-size parity tests and by bench.py for every configuration but the default one.
# --------------------------------------------------------------------------------------
def fill_torch(w: Workload, grads, seed_offset: int = 0) -> None:
    """Fill the n device tensors in `grads` (fp32 or bf16, d elements each) in place."""
    import torch
    dev = grads[0].device
    chunk = 1 << 26
    for i, g in enumerate(grads):
        gen = torch.Generator(device=dev)
        gen.manual_seed(w.data_seed * 1000 + i + seed_offset)
        for lo in range(0, w.d, chunk):
            hi = min(w.d, lo + chunk)
            m = hi - lo
            if w.name.startswith("cfg3"):
                u = torch.rand(m, generator=gen, device=dev, dtype=torch.float32) - 0.5
                a = u.abs().clamp_(max=0.49999997)                              # keep log finite
                x = -5e-4 * torch.sign(u) * torch.log1p(-2.0 * a)               # Laplace(0, 5e-4)
            elif w.name.startswith("cfg4"):
                z = torch.randn(m, generator=gen, device=dev, dtype=torch.float32)
                chi2 = sum(torch.randn(m, generator=gen, device=dev, dtype=torch.float32) ** 2
                           for _ in range(3))
                x = 1e-4 * z / torch.sqrt(chi2 / 3.0)                            # Student-t(3) * 1e-4
            elif w.name.startswith("cfg2"):
                x = torch.randn(m, generator=gen, device=dev, dtype=torch.float32)
                sizes, scales = resnet50_like_segments(w.d, w.data_seed)
                per = torch.repeat_interleave(
                    torch.as_tensor(scales, dtype=torch.float32, device=dev),
                    torch.as_tensor(sizes, device=dev))[lo:hi]
                x = x * per
            elif w.name.startswith("cfg1"):
                x = torch.randn(m, generator=gen, device=dev, dtype=torch.float32) * 1e-3
                out_mask = torch.rand(m, generator=gen, device=dev) < 1e-3
                x = torch.where(out_mask, torch.randn(m, generator=gen, device=dev) * 1e-1, x)
            else:
                x = torch.randn(m, generator=gen, device=dev, dtype=torch.float32)
            g[lo:hi].copy_(x.to(g.dtype))
