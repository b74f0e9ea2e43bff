"""thc_prepare_noalloc: the entry point for callers that may not allocate device memory (it
keeps its scratch in a fixed array inside the library instead of a caller workspace and
needs no context).  Checked through the C ABI against thc_prepare and against the CPU oracle
on the same inputs, on two calls in a row with different data: the shared scratch keeps the first call's contents, and
the second call must not be affected by them.  Collected last (file name) so that a failure
here cannot hide the other GPU tests in a stop-at-first-failure run."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2302_08545_b200 import thc, workloads as W

pytestmark = pytest.mark.gpu


def _within_one_ulp(a, b):
    ai = a.view(np.int32).astype(np.int64)
    bi = b.view(np.int32).astype(np.int64)
    return np.abs(ai - bi).max() <= 1


@pytest.mark.parametrize("k,d,n,dtype", [(20, 3 * (1 << 20) + 4321, 4, "f32"), (12, 70_001, 3, "f32"),
                                         (16, 200_000, 2, "bf16")])
def test_noalloc_prepare_matches_prepare_twice_in_a_row(k, d, n, dtype):
    import torch
    from paper_2302_08545_b200 import runner
    w = W.Workload("sweep_x", n=n, d=d, log2_block=k, bits=4, granularity=30,
                   table=W.TABLES[(4, 30)], in_dtype=dtype, data_seed=77)
    ctx = runner.context_for(w)
    r = runner.Round(ctx, n, d, dtype)
    scales2 = torch.full_like(r.scales, -1.0)
    status = torch.zeros(1, dtype=torch.int32, device=r.device)
    code = thc.THC_BF16 if dtype == "bf16" else thc.THC_F32
    cfg = O.Config(bits=4, granularity=30, table=tuple(W.TABLES[(4, 30)]), t_p=w.t_p, log2_block=k,
                   seed=w.seed)
    for call in range(2):
        W.fill_torch(w, r.grads, seed_offset=call * 100)
        if call == 1:
            r.grads[0][: min(d, 1 << k)].zero_()          # changes the first block's winner
        r.prepare()
        torch.cuda.synchronize()
        held = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]
        thc.prepare_noalloc(r.grads, d, k, code, w.t_p, scales2, status=status)
        torch.cuda.synchronize()
        if call == 1:                                     # the first call may load the module lazily
            assert torch.cuda.memory_allocated() == held
            assert torch.cuda.mem_get_info()[0] >= free_before
        a, b = r.scales.cpu().numpy(), scales2.cpu().numpy()
        assert np.all(b > 0)
        assert _within_one_ulp(a, b), f"call {call}: scales differ from thc_prepare"
        x = np.stack([g.float().cpu().numpy() for g in r.grads])
        assert _within_one_ulp(O.scales(x, cfg), b), f"call {call}: scales differ from the oracle"
        assert int(status.item()) == 0


def test_noalloc_prepare_sets_status_and_rejects_oversized_inputs():
    import torch
    dev = torch.device("cuda:0")
    d, k = 4096, 10
    g = [torch.ones(d, dtype=torch.float32, device=dev) for _ in range(2)]
    g[0][1024:2048] = 0
    g[1][1024:2048] = 0
    g[1][3000] = float("inf")
    scales = torch.zeros(4, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    thc.prepare_noalloc(g, d, k, thc.THC_F32, 2.0, scales, status=status)
    torch.cuda.synchronize()
    s = scales.cpu().numpy()
    assert s[0] > 0 and s[1] == 0 and s[2] == 0 and s[3] > 0
    assert int(status.item()) == (thc.STATUS_NONFINITE | thc.STATUS_ZERO_BLOCK)
    # too many partial sums for the built-in scratch: refused, nothing launched
    partials = thc.NOALLOC_SCRATCH_BYTES // 8
    big_d = (partials // 2 + 1) * (1 << 14)
    with pytest.raises(thc.ThcError) as e:
        thc.prepare_noalloc([g[0].data_ptr(), g[1].data_ptr()], big_d, 20, thc.THC_F32, 2.0, scales)
    assert e.value.code == thc.THC_EWORKSPACE
    with pytest.raises(thc.ThcError):
        thc.prepare_noalloc(g, d, 2, thc.THC_F32, 2.0, scales)
    with pytest.raises(thc.ThcError) as e:                # a length whose padding would wrap
        thc.prepare_noalloc([g[0].data_ptr(), g[1].data_ptr()], (1 << 64) - 5, 20, thc.THC_F32, 2.0, scales)
    assert e.value.code == thc.THC_EINVAL
