"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run these sizes whole, so it runs sampled RHT blocks (the first, the last
-- which is the zero-padded one --, and seeded random ones): blocks are independent given
their global coordinates, so each sampled block is checked exactly like the small cases:
scale, packed indices and sums bit-exact, output within 1e-5 * M.
"""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2302_08545_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _ocfg(w):
    return O.Config(bits=w.bits, granularity=w.granularity, table=tuple(w.table), t_p=w.t_p,
                    log2_block=w.log2_block, seed=w.seed)


def _sample_blocks(w, count, seed):
    nb = w.nblocks
    picks = {0, nb - 1}
    rng = np.random.default_rng(seed)
    while len(picks) < min(count, nb):
        picks.add(int(rng.integers(0, nb)))
    return sorted(picks)


def _to_f32(t):
    import torch
    if t.dtype == torch.bfloat16:
        return O.bf16_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def check_full_size(w, blocks, rnd=0):
    import torch
    from paper_2302_08545_b200 import runner
    ctx = runner.context_for(w)
    r = runner.Round(ctx, w.n, w.d, w.in_dtype)
    W.fill_torch(w, r.grads)
    r.run(rnd)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    c = _ocfg(w)
    B = w.block
    scl_all = r.scales.cpu().numpy()
    wdt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[r.sz.acc_bits]
    T = np.asarray(w.table, dtype=np.int64)
    for blk in blocks:
        lo, hi = blk * B, min(w.d, blk * B + B)
        x = np.stack([_to_f32(g[lo:hi]) for g in r.grads])
        # preliminary stage
        scl_ref = O.scales(x, c)
        ulp = abs(int(scl_all[blk:blk + 1].view(np.int32)[0]) - int(scl_ref.view(np.int32)[0]))
        assert ulp <= 1, f"block {blk}: scale differs by {ulp} ulp"
        scl = scl_all[blk:blk + 1]
        # compress: same bytes as the oracle for every worker
        pb = B * w.bits // 8
        zsum = np.zeros(B, dtype=np.int64)
        for i in range(w.n):
            rot = O.rht_forward(x[i], c, rnd, j_base=lo)
            ref = O.pack(O.quantize(rot, scl, c, rnd, i, j_base=lo), w.bits)
            got = r.packed[i][blk * pb:(blk + 1) * pb].cpu().numpy()
            assert np.array_equal(got, ref), f"block {blk} worker {i}: packed indices differ"
            zsum += T[O.unpack(ref, B, w.bits)]
        # aggregate
        sb = B * r.sz.acc_bits // 8
        got_sum = r.total[blk * sb:(blk + 1) * sb].cpu().numpy().view(wdt)
        assert np.array_equal(got_sum.astype(np.int64), zsum), f"block {blk}: sums differ"
        # decompress
        est = O.estimate(got_sum, w.n, scl, c)
        out_ref = O.rht_inverse(est, hi - lo, c, rnd, j_base=lo)
        out_got = r.out[lo:hi].cpu().numpy()
        err = np.abs(out_got.astype(np.float64) - out_ref.astype(np.float64)).max()
        assert err <= 1e-5 * float(scl[0]), f"block {blk}: output error {err}"
    # the one-call tail (thc_aggregate_decompress) and the launch that also computes the scales
    # (thc_prepare_compress), at this size: the same bits as the separate calls checked above
    out_two_calls = r.out.clone()
    sums_two_calls = r.total.clone()
    r.out.zero_()
    r.total.zero_()
    r.aggregate_decompress(rnd, want_sums=True)
    torch.cuda.synchronize()
    assert torch.equal(r.out.view(torch.int32), out_two_calls.view(torch.int32))
    assert torch.equal(r.total, sums_two_calls)
    if r.sz.fused_scales:
        packed_two_calls = [p.clone() for p in r.packed]
        scales_two_calls = r.scales.clone()
        r.prepare_compress(rnd)
        torch.cuda.synchronize()
        ulps = (r.scales.view(torch.int32) - scales_two_calls.view(torch.int32)).abs().max().item()
        assert ulps <= 1
        if ulps == 0:
            assert all(torch.equal(a, b) for a, b in zip(r.packed, packed_two_calls))
    assert ctx.status() == 0
    del r
    torch.cuda.empty_cache()


def test_config2_full_size():
    w = W.config2()
    check_full_size(w, _sample_blocks(w, 5, 2))


@pytest.mark.parametrize("bits", [2, 4])
def test_config3_full_size(bits):
    w = W.config3(bits)
    check_full_size(w, _sample_blocks(w, 4, 3))


def test_config4_full_size_bf16():
    w = W.config4()
    check_full_size(w, _sample_blocks(w, 3, 4))


@pytest.mark.parametrize("log2d,bits,n", [(20, 1, 2), (22, 8, 4), (24, 2, 32), (26, 4, 16), (24, 8, 32)])
def test_sweep_points_full_size(log2d, bits, n):
    w = W.sweep_point(1 << log2d, bits, n)
    check_full_size(w, _sample_blocks(w, 3, 5))
