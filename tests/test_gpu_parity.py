"""Parity of the CUDA path (through the C ABI) with the CPU oracle, on the same seeded inputs.

Bars (stated by the benchmark definition):
  * packed indices and aggregated sums: bit-exact when both sides quantise the same rotated
    input;
  * end to end: max |err| <= 1e-5 * M of the coordinate's block, at most 1e-6 of the
    indices differing.
Both sides are always given the same `scales` array (the GPU's), so a last-bit difference
in M cannot pass for index flips; thc_prepare is tested on its own.
"""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2302_08545_b200 import workloads as W

pytestmark = pytest.mark.gpu

T4_30 = W.TABLES[(4, 30)]


def _mk(n, d, k, bits=4, g=30, table=T4_30, in_dtype="f32", name="cfg1_x", t_p=W.T_P["1/32"]):
    return W.Workload(name, n=n, d=d, log2_block=k, bits=bits, granularity=g, table=tuple(table),
                      in_dtype=in_dtype, data_seed=4242 + d % 97 + k, t_p=t_p)


def _ocfg(w):
    return O.Config(bits=w.bits, granularity=w.granularity, table=tuple(w.table), t_p=w.t_p,
                    log2_block=w.log2_block, seed=w.seed)


def _inputs(w):
    x = W.generate(w)
    xf = O.bf16_to_f32(x) if w.in_dtype == "bf16" else x
    return x, xf


def _gpu_round(w, x, rnd=0, acc_bits=0, want_rotated=True):
    import torch
    from paper_2302_08545_b200 import runner
    ctx = runner.context_for(w, acc_bits=acc_bits)
    r = runner.Round(ctx, w.n, w.d, w.in_dtype, want_rotated=want_rotated)
    r.upload(x)
    r.run(rnd)
    torch.cuda.synchronize()
    return ctx, r


def _block_scale_per_coord(scl, w, count):
    return np.repeat(scl.astype(np.float64), w.block)[:count]


def check_round(w, rnd=0, acc_bits=0, expect_exact_rotation=True):
    x, xf = _inputs(w)
    ctx, r = _gpu_round(w, x, rnd, acc_bits)
    c = _ocfg(w)
    sz = r.sz
    scl = r.scales.cpu().numpy()

    # thc_prepare on its own: equal as fp32 up to summation order (<= 1 ulp, rare)
    scl_ref = O.scales(xf, c)
    ulp = np.abs(scl.view(np.int32).astype(np.int64) - scl_ref.view(np.int32).astype(np.int64))
    assert ulp.max() <= 1, "scale differs by more than one ulp"
    assert (ulp > 0).mean() <= max(1e-3, 1.0 / scl.size) or scl.size < 1000

    flips = 0
    total_idx = 0
    packed_gpu = np.stack([p.cpu().numpy() for p in r.packed])
    for i in range(w.n):
        rot_gpu = r.rotated[i].cpu().numpy()
        rot_ref = O.rht_forward(xf[i], c, rnd)
        if expect_exact_rotation:
            assert np.array_equal(rot_gpu.view(np.uint32), rot_ref.view(np.uint32)), \
                f"worker {i}: rotated coordinates differ from the oracle's"
        # T1: same rotated input on both sides -> packed bytes identical
        z_from_gpu_rot = O.pack(O.quantize(rot_gpu, scl, c, rnd, i), w.bits)
        assert np.array_equal(packed_gpu[i], z_from_gpu_rot), f"worker {i}: packed indices differ"
        z_ref = O.quantize(rot_ref, scl, c, rnd, i)
        z_gpu = O.unpack(packed_gpu[i], sz.d_pad, w.bits)
        flips += int((z_ref != z_gpu).sum())
        total_idx += z_ref.size
    assert flips <= 1e-6 * total_idx, f"{flips} of {total_idx} indices differ"

    # aggregate: exact integers
    wbits = sz.acc_bits
    sum_ref = O.aggregate(packed_gpu, sz.d_pad, c, wbits)
    sum_gpu = r.sum_numpy()
    assert np.array_equal(sum_gpu, sum_ref), "aggregated sums differ"

    # decompress of the same sums
    out_gpu = r.out.cpu().numpy()
    out_ref = O.decompress(sum_gpu, w.n, w.d, scl, c, rnd)
    M = _block_scale_per_coord(scl, w, w.d)
    err = np.abs(out_gpu.astype(np.float64) - out_ref.astype(np.float64))
    assert np.all(err <= 1e-5 * M + 0.0), f"decompress error {err.max()} vs bound"
    # end to end against the oracle's own round
    if flips == 0:
        assert np.array_equal(out_gpu.view(np.uint32), out_ref.view(np.uint32)) or np.all(err <= 1e-5 * M)
    return ctx, r


@pytest.mark.parametrize("k,d,n", [
    (3, 8, 1), (3, 200, 3), (4, 1000, 2), (5, 4096 + 32, 2), (8, 5000, 4), (10, 33_000, 3),
    (13, 20_000, 2), (14, 16_384, 2), (14, 70_001, 3),
])
def test_single_pass_blocks(k, d, n):
    check_round(_mk(n, d, k))


@pytest.mark.parametrize("k,d,n", [
    (15, 32_768, 2), (15, 100_000, 2), (16, 65_536 * 2 + 5, 3), (18, 300_000, 2),
    (20, (1 << 20) + 777, 2), (21, (1 << 22) + 3, 2), (22, (1 << 22), 1), (22, (1 << 23) + 11, 2),
])
def test_two_pass_blocks(k, d, n):
    check_round(_mk(n, d, k))


@pytest.mark.parametrize("bits,g,table", [
    (1, 1, (0, 1)), (1, 30, (0, 30)), (2, 3, (0, 1, 2, 3)), (2, 4, (0, 1, 3, 4)),
    (3, 7, tuple(range(8))), (3, 12, (0, 2, 4, 5, 6, 7, 9, 12)),
    (4, 15, tuple(range(16))), (4, 30, T4_30), (8, 255, tuple(range(256))),
    (4, 200, tuple(int(round(v)) for v in np.linspace(0, 200, 16))),
])
@pytest.mark.parametrize("k", [10, 16])
def test_bit_budgets_and_tables(bits, g, table, k):
    check_round(_mk(3, 70_000, k, bits=bits, g=g, table=table))


@pytest.mark.parametrize("n,acc", [(8, 0), (9, 0), (16, 16), (3, 32), (40, 0)])
def test_accumulator_widths(n, acc):
    w = _mk(n, 40_000, 12)
    ctx, r = check_round(w, acc_bits=acc)
    assert r.sz.acc_bits == (acc if acc else O.acc_bits(n, 30))


def test_bf16_gradients():
    w = _mk(3, 150_000, 16, in_dtype="bf16", name="cfg4_x")
    check_round(w)


def test_other_round_and_seed_change_the_result():
    w = _mk(2, 50_000, 12)
    x, _ = _inputs(w)
    _, r0 = _gpu_round(w, x, rnd=0)
    _, r1 = _gpu_round(w, x, rnd=1)
    assert not np.array_equal(r0.packed[0].cpu().numpy(), r1.packed[0].cpu().numpy())
    check_round(w, rnd=7)


def test_config1_full_size():
    """Benchmark configuration 1 at full size (n=4, d=65536, one block of 2^16)."""
    check_round(W.config1())


def test_degenerate_and_nonfinite_blocks():
    import torch
    from paper_2302_08545_b200 import runner, thc
    w = _mk(2, 4 * 1024, 10)
    x, _ = _inputs(w)
    x[:, 1024:2048] = 0.0                 # an all-zero block
    x[1, 2048 + 5] = np.inf               # a non-finite block
    x[0, 3072 + 9] = np.nan
    ctx = runner.context_for(w)
    r = runner.Round(ctx, w.n, w.d, want_rotated=False)
    r.upload(x)
    r.run(0)
    torch.cuda.synchronize()
    flags = ctx.status()
    assert flags & thc.STATUS_NONFINITE and flags & thc.STATUS_ZERO_BLOCK
    assert ctx.status() == 0              # read-and-clear
    scl = r.scales.cpu().numpy()
    assert scl[0] > 0 and scl[1] == 0 and scl[2] == 0 and scl[3] == 0
    out = r.out.cpu().numpy()
    assert np.all(out[1024:] == 0.0)
    packed = np.stack([p.cpu().numpy() for p in r.packed])
    assert np.all(packed[:, 1024 // 2:] == 0)
    c = _ocfg(w)
    ref = O.thc_round(x, c, 0, scl=scl)
    assert np.array_equal(packed, ref["packed"])
    assert np.array_equal(out.view(np.uint32), ref["out"].view(np.uint32))


def test_workers_can_be_compressed_in_separate_calls():
    """n_local = 1 calls with worker_base = i give the same bytes as one batched call."""
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(3, 90_000, 16)
    x, _ = _inputs(w)
    ctx, r = _gpu_round(w, x, 0, want_rotated=False)
    batched = [p.cpu().numpy().copy() for p in r.packed]
    for p in r.packed:
        p.zero_()
    for i in range(w.n):
        ctx.compress([r.grads[i]], w.d, 0, r.scales, [r.packed[i]], r.workspace, worker_base=i)
    torch.cuda.synchronize()
    for i in range(w.n):
        assert np.array_equal(batched[i], r.packed[i].cpu().numpy())


def test_quantize_rotated_entry_matches_oracle_on_oracle_rotation():
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(2, 40_000, 13)
    x, xf = _inputs(w)
    c = _ocfg(w)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, w.n, w.d, want_rotated=True)
    scl = O.scales(xf, c)
    r.scales.copy_(torch.from_numpy(scl))
    for i in range(w.n):
        r.rotated[i].copy_(torch.from_numpy(O.rht_forward(xf[i], c, 3)))
    ctx.quantize_rotated(r.rotated, w.d, 3, r.scales, r.packed)
    torch.cuda.synchronize()
    for i in range(w.n):
        ref = O.pack(O.quantize(r.rotated[i].cpu().numpy(), scl, c, 3, i), w.bits)
        assert np.array_equal(r.packed[i].cpu().numpy(), ref)


def test_partial_aggregation_uses_the_count_as_divisor():
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(5, 30_000, 12)
    x, _ = _inputs(w)
    ctx, r = _gpu_round(w, x, 0, want_rotated=False)
    c = _ocfg(w)
    scl = r.scales.cpu().numpy()
    subset = [0, 2, 3]
    ctx.aggregate([r.packed[i] for i in subset], w.d, r.total)
    ctx.decompress(r.total, len(subset), w.d, 0, r.scales, r.out, r.workspace)
    torch.cuda.synchronize()
    packed = np.stack([r.packed[i].cpu().numpy() for i in subset])
    sum_ref = O.aggregate(packed, r.sz.d_pad, c, r.sz.acc_bits)
    assert np.array_equal(r.sum_numpy(), sum_ref)
    out_ref = O.decompress(sum_ref, len(subset), w.d, scl, c, 0)
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), out_ref.view(np.uint32))


def test_unsatisfiable_dependency_times_out_and_the_context_stays_usable():
    """Host-side injection on a tiny launch: the task queue starts one task late, so the
    pass-B panels of the first worker-block wait for a pass-A tile nobody will produce.  The
    kernel's bounded wait must expire, set THC_STATUS_WAIT_TIMEOUT and return; afterwards
    the same context must run a correct round."""
    import time
    import torch
    from paper_2302_08545_b200 import runner, thc
    w = _mk(1, 2 << 15, 15)
    x, _ = _inputs(w)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, w.n, w.d, want_rotated=False)
    r.upload(x)
    r.prepare()
    torch.cuda.synchronize()
    ctx.debug_skip_tasks(1)
    t0 = time.time()
    r.compress(0)
    torch.cuda.synchronize()
    waited = time.time() - t0
    assert ctx.status() & thc.STATUS_WAIT_TIMEOUT
    assert waited < 30.0
    # the context recovers: counters were cleared by the last CTA
    r.run(0)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    c = _ocfg(w)
    ref = O.thc_round(x, c, 0, scl=r.scales.cpu().numpy())
    assert np.array_equal(np.stack([p.cpu().numpy() for p in r.packed]), ref["packed"])
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), ref["out"].view(np.uint32))


@pytest.mark.parametrize("k,d,n", [(10, 33_001, 3), (16, 150_000, 2), (20, (1 << 21) + 99, 2)])
def test_error_feedback_matches_oracle(k, d, n):
    """e_i = x_i - RHT^-1(X_i) (Algorithm 3) from the worker's own packed indices: bit-exact
    against the oracle on the same indices and scales; and x_i + e_i through
    thc_accumulate_error is the fp32 sum."""
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    ctx, r = _gpu_round(w, x, rnd=2, want_rotated=False)
    ef = [torch.zeros(d, dtype=torch.float32, device=r.device) for _ in range(n)]
    ctx.error_feedback(r.grads, r.packed, d, 2, r.scales, ef, r.workspace)
    torch.cuda.synchronize()
    c = _ocfg(w)
    scl = r.scales.cpu().numpy()
    for i in range(n):
        z = O.unpack(r.packed[i].cpu().numpy(), r.sz.d_pad, w.bits)
        ref = O.error_feedback(x[i], z, scl, c, 2)
        got = ef[i].cpu().numpy()
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), f"worker {i}"
    ctx.accumulate_error(r.grads, ef, d)
    torch.cuda.synchronize()
    for i in range(n):
        assert np.array_equal(r.grads[i].cpu().numpy(), x[i] + ef[i].cpu().numpy())


@pytest.mark.parametrize("n,nblk,tail", [(1, 13, 5), (2, 14, 12_345), (3, 9, 0), (8, 6, 77), (13, 2, 4096)])
def test_prepare_compress_fused_equals_the_two_calls(n, nblk, tail):
    """thc_prepare_compress (block norms summed inside the transform kernel, Section 5.3's
    overlap of the norm exchange with the RHT): its scales agree with thc_prepare's (fp64 sums
    in another order: equal, or one ulp apart in rare cases) and with the oracle's; the packed
    indices are bit-identical to thc_compress run on those same scales and to the oracle's."""
    import torch
    from paper_2302_08545_b200 import runner
    k = 20
    d = (nblk - 1) * (1 << k) + (tail if tail else (1 << k))
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d)
    assert r.sz.fused_scales == 1
    r.upload(x)
    r.prepare()
    torch.cuda.synchronize()
    s_two = r.scales.cpu().numpy().copy()
    r.scales.zero_()
    r.prepare_compress(rnd=1)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    s_fused = r.scales.cpu().numpy().copy()
    p_fused = [p.cpu().numpy().copy() for p in r.packed]
    ulp = np.abs(s_fused.view(np.int32).astype(np.int64) - s_two.view(np.int32).astype(np.int64))
    assert ulp.max() <= 1 and (ulp > 0).mean() <= 0.1, ulp
    c = _ocfg(w)
    s_or = O.scales(x, c)
    ulp_o = np.abs(s_fused.view(np.int32).astype(np.int64) - s_or.view(np.int32).astype(np.int64))
    assert ulp_o.max() <= 1
    for p in r.packed:
        p.zero_()
    r.compress(rnd=1)                      # same scales, separate call
    torch.cuda.synchronize()
    for i in range(n):
        assert np.array_equal(r.packed[i].cpu().numpy(), p_fused[i]), f"worker {i}"
    # and the oracle on the first and last blocks of two workers
    for i in (0, n - 1):
        for blk in (0, nblk - 1):
            lo, hi = blk << k, min(d, (blk + 1) << k)
            xb = np.zeros(1 << k, np.float32)
            xb[: hi - lo] = x[i, lo:hi]
            rot = O.rht_forward(xb, c, 1, j_base=lo)
            z = O.quantize(rot, s_fused[blk:blk + 1], c, worker=i, rnd=1, j_base=lo)
            got = O.unpack(p_fused[i][(lo * w.bits) // 8:((lo + (1 << k)) * w.bits) // 8], 1 << k, w.bits)
            assert np.array_equal(got, z), (i, blk)


def test_prepare_compress_falls_back_where_the_fused_kernel_does_not_apply():
    """Other block sizes (and problems too small for the longer pipeline) take the two calls
    inside the same entry point: results identical to calling them."""
    import torch
    from paper_2302_08545_b200 import runner
    for k, d, n in [(16, 300_000, 3), (20, (1 << 20) + 5, 2), (20, 2 * (1 << 20), 14)]:
        w = _mk(n, d, k)
        x, _ = _inputs(w)
        ctx = runner.context_for(w)
        r = runner.Round(ctx, n, d)
        assert r.sz.fused_scales == 0
        r.upload(x)
        r.prepare(); r.compress(rnd=3)
        torch.cuda.synchronize()
        s0 = r.scales.cpu().numpy().copy(); p0 = [p.cpu().numpy().copy() for p in r.packed]
        r.scales.zero_()
        for p in r.packed:
            p.zero_()
        r.prepare_compress(rnd=3)
        torch.cuda.synchronize()
        assert np.array_equal(r.scales.cpu().numpy(), s0)
        for i in range(n):
            assert np.array_equal(r.packed[i].cpu().numpy(), p0[i])


@pytest.mark.parametrize("bits,g", [(1, 1), (2, 3), (3, 7), (8, 255)])
def test_error_feedback_other_index_widths(bits, g):
    """The one-launch error-feedback path unpacks 1-, 2- and 8-bit indices as well."""
    import torch
    k, d, n = 16, 200_003, 2
    w = _mk(n, d, k, bits=bits, g=g, table=tuple(range(g + 1)) if bits > 1 else (0, 1))
    x, _ = _inputs(w)
    ctx, r = _gpu_round(w, x, rnd=5, want_rotated=False)
    ef = [torch.zeros(d, dtype=torch.float32, device=r.device) for _ in range(n)]
    ctx.error_feedback(r.grads, r.packed, d, 5, r.scales, ef, r.workspace)
    torch.cuda.synchronize()
    c = _ocfg(w)
    scl = r.scales.cpu().numpy()
    for i in range(n):
        z = O.unpack(r.packed[i].cpu().numpy(), r.sz.d_pad, w.bits)
        ref = O.error_feedback(x[i], z, scl, c, 5)
        assert np.array_equal(ef[i].cpu().numpy().view(np.uint32), ref.view(np.uint32)), f"worker {i}"


@pytest.mark.parametrize("k,d,n", [(5, 1000, 2), (10, 33_001, 3), (16, 150_000, 2), (20, (1 << 21) + 99, 2),
                                   (22, (1 << 22) + 12_345, 3)])      # six worker-blocks: the compress ring is shorter than the planned one
def test_exact_range_round_matches_oracle(k, d, n):
    """THC_RANGE_MINMAX contexts (Algorithm 1's preliminary stage on the rotated coordinates):
    the (min, max) planes equal the oracle's bit for bit (the rotated coordinates do), and so
    do the packed indices, the sums, the output and the error feedback computed from them."""
    import torch
    from paper_2302_08545_b200 import runner, thc
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    ctx = runner.context_for(w, exact_range=True)
    r = runner.Round(ctx, n, d)
    assert r.sz.scales_count == 2 * r.sz.nblocks and r.sz.fused_scales == 0
    r.upload(x)
    rnd = 4
    r.prepare_minmax(rnd)
    r.compress(rnd)
    r.aggregate()
    r.decompress(rnd)
    ef = [torch.zeros(d, dtype=torch.float32, device=r.device) for _ in range(n)]
    ctx.error_feedback(r.grads, r.packed, d, rnd, r.scales, ef, r.workspace)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    c = _ocfg(w)
    lo, hi = O.ranges(x, c, rnd)
    got = r.scales.cpu().numpy()
    nb = r.sz.nblocks
    assert np.array_equal(got[:nb].view(np.uint32), lo.view(np.uint32))
    assert np.array_equal(got[nb:].view(np.uint32), hi.view(np.uint32))
    ref = O.thc_round(x, c, rnd, exact_range=True)
    for i in range(n):
        assert np.array_equal(r.packed[i].cpu().numpy(), ref["packed"][i]), f"worker {i}"
    assert np.array_equal(r.sum_numpy(), ref["sum"])
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), ref["out"].view(np.uint32))
    for i in range(n):
        z = O.unpack(ref["packed"][i], r.sz.d_pad, w.bits)
        e = O.error_feedback(x[i], z, hi, c, rnd, lo=lo)
        assert np.array_equal(ef[i].cpu().numpy().view(np.uint32), e.view(np.uint32)), f"worker {i}"
    # no coordinate was clamped: the extreme indices occur, and only at the extremes
    with pytest.raises(thc.ThcError):
        r.prepare()                        # the norm-based call does not apply to this context


def test_exact_range_flags_non_finite_blocks():
    import torch
    from paper_2302_08545_b200 import runner, thc
    k, d, n = 16, 3 * (1 << 16), 2
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    x[1, (1 << 16) + 5] = np.inf
    x[0, 2 * (1 << 16):] = 0.0
    x[1, 2 * (1 << 16):] = 0.0
    ctx = runner.context_for(w, exact_range=True)
    r = runner.Round(ctx, n, d)
    r.upload(x)
    r.prepare_minmax(0)
    r.compress(0); r.aggregate(); r.decompress(0)
    torch.cuda.synchronize()
    flags = ctx.status()
    assert flags & thc.STATUS_NONFINITE and flags & thc.STATUS_ZERO_BLOCK
    s = r.scales.cpu().numpy()
    assert s[1] == 0.0 and s[3 + 1] == 0.0 and s[2] == 0.0 and s[3 + 2] == 0.0 and s[3] > s[0]
    out = r.out.cpu().numpy()
    assert np.all(out[(1 << 16):] == 0.0) and np.all(np.isfinite(out))


def test_error_feedback_loop_on_the_gpu_telescopes_and_matches_the_oracle():
    """Algorithm 3's worker loop over several rounds, all on the GPU: x = grad + e,
    compress, e = x - RHT^-1(X).  Every round's residual equals the oracle's run of the same
    loop bit for bit, and what was sent telescopes: sum_r RHT^-1(X^r) = R grad - e^R
    (up to fp32 rounding of the additions)."""
    import torch
    from paper_2302_08545_b200 import runner
    k, d, n, R = 16, 100_000, 2, 4
    w = _mk(n, d, k, t_p=0.9)                            # a tight clamp: large residuals
    g, _ = _inputs(w)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d)
    c = _ocfg(w)
    ef = [torch.zeros(d, dtype=torch.float32, device=r.device) for _ in range(n)]
    e_ref = np.zeros((n, d), np.float32)
    sent = np.zeros((n, d), np.float64)
    for rnd in range(R):
        r.upload(g)
        ctx.accumulate_error(r.grads, ef, d)             # x = grad + e
        r.prepare()
        r.compress(rnd)
        ctx.error_feedback(r.grads, r.packed, d, rnd, r.scales, ef, r.workspace)
        torch.cuda.synchronize()
        x_ref = g + e_ref                                # one fp32 addition, as on the GPU
        scl = r.scales.cpu().numpy()
        for i in range(n):
            assert np.array_equal(r.grads[i].cpu().numpy(), x_ref[i])
            z = O.unpack(r.packed[i].cpu().numpy(), r.sz.d_pad, w.bits)
            e_new = O.error_feedback(x_ref[i], z, scl, c, rnd)
            assert np.array_equal(ef[i].cpu().numpy().view(np.uint32), e_new.view(np.uint32)), (rnd, i)
            sent[i] += x_ref[i].astype(np.float64) - e_new.astype(np.float64)
            e_ref[i] = e_new
    assert ctx.status() == 0
    resid = sent - (R * g.astype(np.float64) - e_ref.astype(np.float64))
    assert np.abs(resid).max() <= 1e-5 * np.abs(g).max() * R


def test_step_can_be_captured_in_a_cuda_graph_and_replayed():
    """The hot calls only enqueue work on the given stream: after one eager step (which sets
    kernel attributes) the whole step is captured into a CUDA graph; replays on new inputs
    give the same bits as eager calls."""
    import torch
    from paper_2302_08545_b200 import runner
    for k, d, n in [(16, 65_536 * 3, 4), (20, 14 * (1 << 20) + 17, 2)]:
        w = _mk(n, d, k)
        x, _ = _inputs(w)
        ctx = runner.context_for(w)
        r = runner.Round(ctx, n, d)
        r.upload(x)
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            r.run(3, fused=True)                         # eager, on the capture stream
        side.synchronize()
        expect_packed = [p.clone() for p in r.packed]
        expect_out = r.out.clone()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            r.run(3, fused=True)
        for p in r.packed:
            p.zero_()
        r.out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for a, b in zip(r.packed, expect_packed):
            assert torch.equal(a, b)
        assert torch.equal(r.out, expect_out)
        r.upload(x[::-1].copy())                         # other inputs, same graph
        graph.replay()
        torch.cuda.synchronize()
        got_out = r.out.clone()
        r.run(3, fused=True)
        torch.cuda.synchronize()
        assert torch.equal(got_out, r.out)
        assert ctx.status() == 0


@pytest.mark.parametrize("bits,g,table,n", [
    (1, 1, (0, 1), 5), (1, 200, (0, 200), 1), (1, 3, (0, 3), 64), (2, 3, (0, 1, 2, 3), 64),
    (4, 30, T4_30, 17), (4, 30, T4_30, 64), (4, 15, tuple(range(16)), 64), (4, 127, tuple(range(15)) + (127,), 3),
    (8, 255, tuple(range(256)), 7), (8, 255, tuple(range(256)), 64),
    (3, 7, tuple(range(8)), 9), (3, 20, (0, 1, 5, 8, 10, 13, 17, 20), 13), (3, 60, (0, 9, 17, 26, 30, 41, 50, 60), 64),
])
def test_aggregate_fast_paths_on_random_indices(bits, g, table, n):
    """The byte-lane (SWAR) aggregation kernels against the oracle's plain loop on uniformly
    random packed indices: every index value, every lane, chunk boundaries of the 16-bit
    widening, and a ragged number of thread units."""
    import torch
    from paper_2302_08545_b200 import runner
    k = 7
    d = 128 * 1237                                        # not a multiple of the grid stride
    w = _mk(n, d, k, bits=bits, g=g, table=table)
    ctx = runner.context_for(w)
    sz = ctx.sizes(d, n)
    rng = np.random.default_rng(1000 * bits + n)
    packed = rng.integers(0, 256, size=(n, sz.packed_bytes), dtype=np.uint8)
    dev = torch.device("cuda", 0)
    bufs = [torch.from_numpy(packed[i]).to(dev) for i in range(n)]
    total = torch.zeros(sz.sum_bytes, dtype=torch.uint8, device=dev)
    ctx.aggregate(bufs, d, total)
    torch.cuda.synchronize()
    c = _ocfg(w)
    ref = O.aggregate(packed, sz.d_pad, c, sz.acc_bits)
    dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[sz.acc_bits]
    assert np.array_equal(total.cpu().numpy().view(dt), ref)


def test_prepare_compress_fused_degenerate_blocks():
    """All-zero and non-finite blocks through the fused scales path: the same scales, status
    bits and indices as the two separate calls."""
    import torch
    from paper_2302_08545_b200 import runner, thc
    k, n, nblk = 20, 2, 14
    d = nblk << k
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    x[:, 3 << k:4 << k] = 0.0
    x[1, (7 << k) + 12345] = np.inf
    x[0, (9 << k) + 5] = np.nan
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d)
    assert r.sz.fused_scales == 1
    r.upload(x)
    r.prepare(); r.compress(2)
    torch.cuda.synchronize()
    f0 = ctx.status()
    s0 = r.scales.cpu().numpy().copy(); p0 = [p.cpu().numpy().copy() for p in r.packed]
    r.scales.fill_(-1.0)
    for p in r.packed:
        p.fill_(255)
    r.prepare_compress(2)
    torch.cuda.synchronize()
    f1 = ctx.status()
    assert f0 == f1 == (thc.STATUS_NONFINITE | thc.STATUS_ZERO_BLOCK)
    s1 = r.scales.cpu().numpy()
    assert s1[3] == 0.0 and s1[7] == 0.0 and s1[9] == 0.0
    ulp = np.abs(s1.view(np.int32).astype(np.int64) - s0.view(np.int32).astype(np.int64))
    assert ulp.max() <= 1
    if ulp.max() == 0:
        for i in range(n):
            assert np.array_equal(r.packed[i].cpu().numpy(), p0[i])
    for blk in (3, 7, 9):
        for i in range(n):
            seg = r.packed[i].cpu().numpy()[(blk << k) // 2:((blk + 1) << k) // 2]
            assert not seg.any()


@pytest.mark.parametrize("k,d,n", [(10, 33_001, 2), (16, 150_000, 2), (20, (1 << 21) + 99, 2)])
def test_exact_range_with_rotated_output_needs_one_transform(k, d, n):
    """thc_prepare_minmax can hand out the rotated coordinates; thc_quantize_rotated on them
    gives the same packed indices as thc_compress (which transforms again)."""
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(n, d, k)
    x, _ = _inputs(w)
    ctx = runner.context_for(w, exact_range=True)
    r = runner.Round(ctx, n, d, want_rotated=True)
    r.upload(x)
    r.prepare_minmax(6)
    r.quantize_rotated(6)
    torch.cuda.synchronize()
    one_pass = [p.cpu().numpy().copy() for p in r.packed]
    rot = [t.cpu().numpy().copy() for t in r.rotated]
    for p in r.packed:
        p.zero_()
    r.compress(6)
    torch.cuda.synchronize()
    c = _ocfg(w)
    for i in range(n):
        assert np.array_equal(one_pass[i], r.packed[i].cpu().numpy())
        assert np.array_equal(rot[i].view(np.uint32), O.rht_forward(x[i], c, 6).view(np.uint32))
    assert ctx.status() == 0


@pytest.mark.parametrize("bits,g,table,n,k,d", [
    (4, 30, T4_30, 8, 20, (1 << 21) + 777),              # one launch, 8-bit sums
    (4, 30, T4_30, 17, 16, 3 * (1 << 16) + 5),           # 16-bit sums, run-time geometry
    (3, 20, (0, 1, 5, 8, 10, 13, 17, 20), 5, 20, 1 << 20),
    (2, 3, (0, 1, 2, 3), 64, 15, (1 << 17) + 1),
    (1, 200, (0, 200), 3, 20, (1 << 20) + 12345),        # 3 * 200 = 600: 16-bit sums
    (8, 255, tuple(range(256)), 64, 20, 1 << 20),        # 64 * 255: 16-bit sums
    (8, 255, tuple(range(256)), 2, 18, 1 << 19),
    (4, 30, T4_30, 6, 10, 33_001),                       # small blocks: the composed form
])
@pytest.mark.parametrize("want_sums", [False, True])
def test_aggregate_decompress_in_one_call(bits, g, table, n, k, d, want_sums):
    """thc_aggregate_decompress (Algorithm 2's PS line feeding the estimate line and the inverse
    RHT in one launch) on uniformly random packed indices: the output equals, bit for bit, the
    oracle's decompression of the oracle's sums and the library's two separate calls; the sums,
    when asked for, equal the oracle's."""
    import torch
    from paper_2302_08545_b200 import runner
    w = _mk(n, d, k, bits=bits, g=g, table=table)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d, "f32")
    rng = np.random.default_rng(7000 + 10 * bits + n + k)
    packed = rng.integers(0, 256, size=(n, r.sz.packed_bytes), dtype=np.uint8)
    for i in range(n):
        r.packed[i].copy_(torch.from_numpy(packed[i]))
    nblk = r.sz.nblocks
    scl = (0.5 + rng.random(nblk)).astype(np.float32)
    if nblk > 1:
        scl[nblk - 1] = 0.0                               # a degenerate block decodes to zeros
    r.scales.copy_(torch.from_numpy(scl))
    r.total.fill_(0xAB)
    r.aggregate_decompress(rnd=3, want_sums=want_sums)
    torch.cuda.synchronize()
    fused_out = r.out.cpu().numpy().copy()
    c = _ocfg(w)
    ref_sum = O.aggregate(packed, r.sz.d_pad, c, r.sz.acc_bits)
    ref_out = O.decompress(ref_sum, n, d, scl, c, 3)
    assert np.array_equal(fused_out.view(np.uint32), ref_out.view(np.uint32))
    dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[r.sz.acc_bits]
    got_sum = r.total.cpu().numpy().view(dt)
    if want_sums:
        assert np.array_equal(got_sum, ref_sum)
    elif k > 14 and bits == 4:
        assert np.all(r.total.cpu().numpy() == 0xAB)      # one launch, sums not asked for: not written
    r.out.zero_()
    r.aggregate()
    r.decompress(3)
    torch.cuda.synchronize()
    assert np.array_equal(r.out.cpu().numpy().view(np.uint32), fused_out.view(np.uint32))
    assert ctx.status() in (0, 2)
