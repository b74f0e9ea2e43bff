"""Repeated launches of the persistent pipeline: the same round several hundred times in a row
must give the same scales, packed indices and output every time with no status flag (a late
dependency, a lost completion signal or a buffer handed over too early would show here first),
for the fused scales + compress launch, run-time and compile-time geometries, exact-range mode
and the one-call tail.  And two contexts driven from two host threads on two streams at once."""
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


def test_two_contexts_on_two_host_threads_and_streams():
    """Contexts are independent: two host threads, each with its own context, buffers and
    stream, run rounds at the same time (the persistent kernels share the GPU); every round of
    both must equal the one computed alone."""
    import threading
    import torch
    from paper_2302_08545_b200 import runner
    cases = [W.Workload("thr_a", n=3, d=3 * (1 << 20) + 11, log2_block=20, bits=4, granularity=30, table=T, data_seed=1),
             W.Workload("thr_b", n=4, d=(1 << 21) + 7, log2_block=16, bits=4, granularity=30, table=T, data_seed=2)]
    rounds, refs = [], []
    for w in cases:
        ctx = runner.context_for(w)
        r = runner.Round(ctx, w.n, w.d)
        W.fill_torch(w, r.grads)
        r.run(7, fused=bool(r.sz.fused_scales))
        torch.cuda.synchronize()
        rounds.append((ctx, r))
        refs.append(([p.clone() for p in r.packed], r.out.clone()))
    errors = []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            ctx, r = rounds[i]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for it in range(150):
                    r.run(7, stream=stream, fused=bool(r.sz.fused_scales))
                    if it % 10 == 9:
                        stream.synchronize()
                        ok = all(torch.equal(a, b) for a, b in zip(r.packed, refs[i][0])) and torch.equal(r.out, refs[i][1])
                        if not ok:
                            errors.append((i, it))
                            return
                stream.synchronize()
            if ctx.status() != 0:
                errors.append((i, "status", ctx.status()))
        except Exception as e:                         # surfaced by the assert below
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not any(t.is_alive() for t in threads)
    assert errors == []
