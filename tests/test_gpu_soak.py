"""Repeated launches of the persistent pipeline: the same round several hundred times in a row
must give the same scales, packed indices and output every time with no status flag (a late
dependency, a lost completion signal or a buffer handed over too early would show here first),
for the fused scales + compress launch, run-time and compile-time geometries, exact-range mode
and the one-call tail."""
import pytest

from paper_2302_08545_b200 import workloads as W

pytestmark = pytest.mark.gpu

T = W.TABLES[(4, 30)]


@pytest.mark.parametrize("k,d,n,dtype,exact,iters", [
    (20, 5 * (1 << 20) + 777, 4, "f32", False, 400),      # fused scales + compress
    (16, (1 << 21) + 5, 4, "f32", False, 400),
    (18, (1 << 22) + 99, 3, "f32", False, 300),
    (21, (1 << 23) + 5, 2, "f32", False, 200),
    (22, 3 * (1 << 22) + 5, 2, "bf16", False, 150),        # six worker-blocks: the four-slot ring
    (20, (1 << 22) + 99, 3, "f32", True, 200),
])
def test_repeated_rounds_are_identical(k, d, n, dtype, exact, iters):
    import torch
    from paper_2302_08545_b200 import runner
    w = W.Workload(f"soak_k{k}", n=n, d=d, log2_block=k, bits=4, granularity=30, table=T, data_seed=k,
                   in_dtype=dtype)
    ctx = runner.context_for(w, exact_range=exact)
    r = runner.Round(ctx, n, d, dtype)
    W.fill_torch(w, r.grads)
    fused = bool(r.sz.fused_scales) and not exact

    def step():
        if exact:
            r.prepare_minmax(3)
            r.compress(3)
        elif fused:
            r.prepare_compress(3)
        else:
            r.prepare()
            r.compress(3)
        r.aggregate()
        r.decompress(3)

    step()
    torch.cuda.synchronize()
    ref_p = [p.clone() for p in r.packed]
    ref_o, ref_s = r.out.clone(), r.scales.clone()
    tail = torch.empty_like(r.out)
    for i in range(iters):
        step()
        if i % 4 == 0:
            ctx.aggregate_decompress(r.packed, d, 3, r.scales, tail, r.workspace)
            assert torch.equal(tail, ref_o), f"one-call tail, iteration {i}"
        assert torch.equal(r.scales, ref_s), f"scales, iteration {i}"
        assert all(torch.equal(a, b) for a, b in zip(r.packed, ref_p)), f"indices, iteration {i}"
        assert torch.equal(r.out, ref_o), f"output, iteration {i}"
    assert ctx.status() == 0
