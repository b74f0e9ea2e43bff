"""The lookup-table solver (Section 5.2 / Appendix B) against brute force and the paper's
printed facts, and the tables the workloads use against the solver."""
import math
from itertools import combinations

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


def increasing_tables(bits: int, g: int):
    """Every table 0 = T[0] < T[1] < ... < T[2^b - 1] = g: the inner values are a subset of
    {1, ..., g - 1} in increasing order.  (Appendix B counts them as g - 2^b + 1 balls in
    2^b - 1 bins, the balls being the grid points skipped between neighbours.)"""
    for inner in combinations(range(1, g), (1 << bits) - 2):
        yield (0,) + inner + (g,)


def brute_force_table(bits: int, g: int, p: float):
    """Exhaustive search over all strictly increasing tables (small cases only)."""
    tp = tables.t_p(p)
    best = None
    for table in increasing_tables(bits, g):
        key = (round(tables.table_cost(table, g, tp), 13), table)
        if best is None or key < best:
            best = key
    return best[1], best[0]


def test_enumeration_counts_match_appendix_b():
    """The number of candidate tables is C(g - 1, 2^b - 2), which is Appendix B's stars-and-bars
    count C(n + k - 1, k - 1) with n = g - 2^b + 1 balls and k = 2^b - 1 bins; for b = 4, g = 51 the
    paper quotes about 4.8e11 candidates, and 100947 after its symmetry reduction for the
    example it works out."""
    for bits, g in ((1, 5), (2, 4), (2, 9), (3, 12)):
        levels = 1 << bits
        tabs = list(increasing_tables(bits, g))
        n, k = g - levels + 1, levels - 1
        assert len(tabs) == len(set(tabs)) == math.comb(n + k - 1, k - 1) == math.comb(g - 1, levels - 2)
        assert all(t[0] == 0 and t[-1] == g and all(a < b for a, b in zip(t, t[1:])) for t in tabs)
    assert abs(math.comb(48, 14) / 4.8e11 - 1) < 0.01
    assert math.comb(23, 6) == 100947


@pytest.mark.parametrize("bits,g", [(1, 1), (1, 5), (2, 3), (2, 4), (2, 9), (3, 7), (3, 12), (3, 14)])
def test_dp_equals_brute_force(bits, g):
    for p in (1 / 32, 1 / 1024):
        t_dp, c_dp = tables.optimal_table(bits, g, p)
        t_bf, c_bf = brute_force_table(bits, g, p)
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
