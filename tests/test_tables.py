"""The lookup-table solver (Section 5.2 / Appendix B) against brute force and the paper's
printed facts, and the tables the workloads use against the solver."""
import math

import pytest
from scipy import integrate
from scipy.stats import norm

from paper_2302_08545_b200 import tables, workloads as W


def test_t_p_values():
    for name, p in (("1/32", 1 / 32), ("1/512", 1 / 512), ("1/1024", 1 / 1024)):
        assert abs(tables.t_p(p) - W.T_P[name]) < 1e-9
        assert abs(tables.t_p(p) - norm.ppf(1 - p / 2)) < 1e-9


def test_interval_cost_closed_form_matches_quadrature():
    for l, h in ((-0.3, 0.9), (-2.0, -1.2), (0.0, 0.4), (1.1, 2.15)):
        ref = integrate.quad(lambda a: (a - l) * (h - a) * norm.pdf(a), l, h)[0]
        assert abs(tables.interval_cost(l, h) - ref) < 1e-12


def test_paper_worked_integral_is_the_interval_sum():
    """Appendix B writes the objective of T = [0,1,3,4] (b=2, g=4) as three integrals of
    p*(a-q1)^2 + (1-p)*(a-q0)^2, which is (a-q0)(q1-a) on each interval."""
    tp = tables.t_p(1 / 32)
    q = [-tp, -tp / 2, tp / 2, tp]

    def integrand(a, q0, q1):
        up = (a - q0) / (q1 - q0)
        return (up * (a - q1) ** 2 + (1 - up) * (a - q0) ** 2) * norm.pdf(a)

    ref = sum(integrate.quad(integrand, q[i], q[i + 1], args=(q[i], q[i + 1]))[0] for i in range(3))
    assert abs(tables.table_cost((0, 1, 3, 4), 4, tp) - ref) < 1e-12


def test_stars_and_bars_enumeration_is_complete_and_duplicate_free():
    for n, k in ((0, 3), (3, 1), (4, 3), (5, 4)):
        seen = list(tables.stars_and_bars(n, k))
        assert len(seen) == math.comb(n + k - 1, k - 1) == len(set(seen))
        assert all(sum(b) == n and min(b) >= 0 for b in seen)
    assert next(iter(tables.stars_and_bars(4, 3))) == (4, 0, 0)


@pytest.mark.parametrize("bits,g", [(1, 1), (1, 5), (2, 3), (2, 4), (2, 9), (3, 7), (3, 12), (3, 14)])
def test_dp_equals_brute_force(bits, g):
    for p in (1 / 32, 1 / 1024):
        t_dp, c_dp = tables.optimal_table(bits, g, p)
        t_bf, c_bf = tables.brute_force_table(bits, g, p)
        assert abs(c_dp - c_bf) < 1e-12
        assert t_dp == t_bf


def test_tables_used_by_the_workloads():
    t, _ = tables.optimal_table(4, 30, 1 / 32)
    assert t == W.TABLES[(4, 30)]
    assert tables.optimal_table(2, 3, 1 / 32)[0] == W.TABLES[(2, 3)]      # uniform is forced
    assert tables.optimal_table(4, 15, 1 / 32)[0] == W.TABLES[(4, 15)]
    # finer granularity can only help (the old grid points are still available when g doubles)
    assert tables.optimal_table(4, 30, 1 / 32)[1] <= tables.optimal_table(4, 15, 1 / 32)[1] + 1e-15
    # optimal tables are symmetric for odd g (Appendix B's symmetry argument)
    t51, _ = tables.optimal_table(4, 51, 1 / 32)
    assert all(a + b == 51 for a, b in zip(t51, reversed(t51)))
