"""Shape of the NMSE-versus-granularity study (Section 8.5 / Appendix D) on the GPU path, and
agreement of the GPU's NMSE with the oracle's on a small case."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2302_08545_b200 import tables

pytestmark = pytest.mark.gpu


def test_nmse_falls_with_granularity_and_by_much_more_with_bits():
    from paper_2302_08545_b200 import nmse_experiment as E
    rows = E.run({2: (3, 6, 10), 3: (7, 14), 4: (15, 30, 52)}, log2_d=21, workers=10)
    nm = {(r["bits"], r["granularity"]): r["nmse"] for r in rows}
    # more grid points for the same number of bits: no worse (optimal tables nest in quality)
    assert nm[(2, 6)] <= nm[(2, 3)] * 1.02 and nm[(2, 10)] <= nm[(2, 6)] * 1.02
    assert nm[(4, 30)] <= nm[(4, 15)] * 1.02 and nm[(4, 52)] <= nm[(4, 30)] * 1.02
    # two more bits: far more than the gain from granularity (the paper: about 10x per bit)
    assert min(nm[(4, g)] for g in (15, 30, 52)) < 0.05 * min(nm[(2, g)] for g in (3, 6, 10))
    # three bits sit in between, each bit worth a large factor
    best = {b: min(v for (bb, _), v in nm.items() if bb == b) for b in (2, 3, 4)}
    assert best[4] < 0.5 * best[3] < 0.25 * best[2]
    assert all(0.0 < v < 1.0 for v in nm.values())


def test_gpu_nmse_equals_the_oracles_on_a_small_case():
    import torch
    from paper_2302_08545_b200 import nmse_experiment as E
    bits, g, p, n, k = 4, 26, 1.0 / 1024, 4, 16
    grads = E.lognormal_gradients(n, 3 * (1 << k) + 1234, 5, torch.device("cuda", 0))
    got = E.nmse_point(bits, g, p, grads, log2_block=k, rnd=2)
    table, _ = tables.optimal_table(bits, g, p)
    c = O.Config(bits=bits, granularity=g, table=tuple(table), t_p=tables.t_p(p), log2_block=k,
                 seed=0x0123456789ABCDEF)
    x = np.stack([t.cpu().numpy() for t in grads])
    out = O.thc_round(x, c, 2)["out"]
    mean = x.astype(np.float64).mean(axis=0)
    ref = float(((out.astype(np.float64) - mean) ** 2).sum() / (mean ** 2).sum())
    assert abs(got - ref) <= 1e-4 * ref, (got, ref)
