"""Seeded random configurations (block size, length, workers, index width, table, accumulator
width, round, range mode) through the whole path on the GPU, each compared with the oracle:
scales or ranges, packed indices, sums, output (from the two calls and from the one-call tail)
and error feedback."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2302_08545_b200 import tables, workloads as W

pytestmark = pytest.mark.gpu


def _random_case(rng):
    k = int(rng.choice([3, 5, 7, 9, 11, 13, 14, 15, 16, 17, 18, 19, 20, 21, 22]))
    B = 1 << k
    nblk = int(rng.integers(1, 6 if k <= 16 else 3))
    if k >= 20:
        nblk = int(rng.integers(1, 3))
    d = (nblk - 1) * B + int(rng.integers(1, B + 1))
    n = int(rng.integers(1, 10 if k <= 18 else 4))
    bits = int(rng.choice([1, 2, 3, 4, 8]))
    levels = 1 << bits
    if rng.random() < 0.4:
        g = levels - 1
        table = tuple(range(levels))
    else:
        g = int(rng.integers(levels - 1, min(255, 4 * levels) + 1))
        inner = np.sort(rng.choice(np.arange(1, g), size=levels - 2, replace=False)) if levels > 2 else []
        table = (0,) + tuple(int(v) for v in inner) + (g,)
    acc = int(rng.choice([0, 0, 0, 16, 32]))
    if acc and n * g > (1 << acc) - 1:
        acc = 0
    return dict(k=k, d=d, n=n, bits=bits, g=g, table=table, acc=acc, rnd=int(rng.integers(0, 1 << 20)),
                exact=bool(rng.random() < 0.35), t_p=float(rng.choice([0.8, W.T_P["1/32"], 3.3])))


@pytest.mark.parametrize("case", range(96))
def test_random_configuration(case):
    import torch
    from paper_2302_08545_b200 import runner
    rng = np.random.default_rng(90_000 + case)
    p = _random_case(rng)
    w = W.Workload(f"rand{case}", n=p["n"], d=p["d"], log2_block=p["k"], bits=p["bits"], granularity=p["g"],
                   table=p["table"], in_dtype="f32", data_seed=case, t_p=p["t_p"])
    x = (rng.standard_normal((p["n"], p["d"])) * np.exp(rng.standard_normal((p["n"], p["d"])))).astype(np.float32)
    c = O.Config(bits=w.bits, granularity=w.granularity, table=tuple(w.table), t_p=w.t_p,
                 log2_block=w.log2_block, seed=w.seed)
    ctx = runner.context_for(w, acc_bits=p["acc"], exact_range=p["exact"])
    r = runner.Round(ctx, w.n, w.d)
    r.upload(x)
    rnd = p["rnd"]
    if p["exact"]:
        r.prepare_minmax(rnd)
    else:
        r.prepare()
    r.compress(rnd)
    r.aggregate()
    r.decompress(rnd)
    ef = [torch.zeros(w.d, dtype=torch.float32, device=r.device) for _ in range(w.n)]
    ctx.error_feedback(r.grads, r.packed, w.d, rnd, r.scales, ef, r.workspace)
    torch.cuda.synchronize()
    assert ctx.status() == 0, p
    nb = r.sz.nblocks
    s = r.scales.cpu().numpy()
    if p["exact"]:
        lo_ref, hi_ref = O.ranges(x, c, rnd)
        assert np.array_equal(s[:nb].view(np.uint32), lo_ref.view(np.uint32)), p
        assert np.array_equal(s[nb:].view(np.uint32), hi_ref.view(np.uint32)), p
        lo, hi = s[:nb], s[nb:]
    else:
        ref = O.scales(x, c)
        ulp = np.abs(s.view(np.int32).astype(np.int64) - ref.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1, p
        lo, hi = None, s
    packed = np.stack([q.cpu().numpy() for q in r.packed])
    exp_packed, _ = O.compress(x, hi, c, rnd, lo=lo)            # the GPU's own scales: bit-exact indices
    assert np.array_equal(packed, exp_packed), p
    total = r.sum_numpy()
    assert np.array_equal(total, O.aggregate(packed, r.sz.d_pad, c, r.sz.acc_bits)), p
    out_ref = O.decompress(total, w.n, w.d, hi, c, rnd, lo=lo)
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), out_ref.view(np.uint32)), p
    # the same tail as one call (sums into a fresh buffer on odd cases, not written on even ones)
    r.out.zero_()
    r.total.fill_(0x5A)
    r.aggregate_decompress(rnd, want_sums=bool(case & 1))
    torch.cuda.synchronize()
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), out_ref.view(np.uint32)), p
    if case & 1:
        assert np.array_equal(r.sum_numpy(), total), p
    for i in range(w.n):
        z = O.unpack(packed[i], r.sz.d_pad, w.bits)
        e = O.error_feedback(x[i], z, hi, c, rnd, lo=lo)
        assert np.array_equal(ef[i].cpu().numpy().view(np.uint32), e.view(np.uint32)), (p, i)


@pytest.mark.parametrize("case", range(12))
def test_random_bf16_configuration(case):
    """The same for bf16 gradients (widened exactly to fp32 on both sides)."""
    import torch
    from paper_2302_08545_b200 import runner
    rng = np.random.default_rng(70_000 + case)
    k = int(rng.choice([4, 9, 13, 14, 15, 16, 18, 20, 21, 22]))
    B = 1 << k
    nblk = int(rng.integers(1, 4 if k <= 18 else 3))
    d = (nblk - 1) * B + int(rng.integers(1, B + 1))
    n = int(rng.integers(1, 6 if k <= 18 else 3))
    rnd = int(rng.integers(0, 1 << 16))
    w = W.Workload(f"randbf{case}", n=n, d=d, log2_block=k, bits=4, granularity=30, table=W.TABLES[(4, 30)],
                   in_dtype="bf16", data_seed=case, t_p=W.T_P["1/32"])
    xf = (rng.standard_normal((n, d)) * 1e-2).astype(np.float32)
    bits16 = (xf.view(np.uint32) >> 16).astype(np.uint16)             # truncate to bf16
    x = O.bf16_to_f32(bits16)
    c = O.Config(bits=4, granularity=30, table=tuple(w.table), t_p=w.t_p, log2_block=k, seed=w.seed)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d, "bf16")
    r.upload(bits16)
    r.run(rnd)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    s = r.scales.cpu().numpy()
    ulp = np.abs(s.view(np.int32).astype(np.int64) - O.scales(x, c).view(np.int32).astype(np.int64))
    assert ulp.max() <= 1
    packed = np.stack([q.cpu().numpy() for q in r.packed])
    exp_packed, _ = O.compress(x, s, c, rnd)
    assert np.array_equal(packed, exp_packed), (k, d, n)
    total = r.sum_numpy()
    assert np.array_equal(total, O.aggregate(packed, r.sz.d_pad, c, r.sz.acc_bits))
    out_ref = O.decompress(total, n, d, s, c, rnd)
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), out_ref.view(np.uint32))
