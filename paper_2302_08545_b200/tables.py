"""Offline construction of THC's lookup table T_{b,g,p} (Section 5.2 and Appendix B of the
THC paper): the table 0 = T[0] < ... < T[2^b - 1] = g on the grid <g+1> that minimises the
expected squared error of unbiased stochastic quantisation of a standard normal variable
truncated to [-t_p, t_p], t_p = Phi^-1(1 - p/2).

Host-only and offline: the hot path takes T as an input.  The paper enumerates all monotone
tables; because the objective is a sum over the intervals between consecutive table values
(for a in [l, h] the variance of unbiased SQ is (a - l)(h - a), Appendix B's worked integral),
an exact dynamic programme over interval end points finds the same minimiser in O(2^b g^2).
"""
from __future__ import annotations

import math
from statistics import NormalDist


def t_p(p: float) -> float:
    """Truncation threshold Phi^-1(1 - p/2) (Section 5.2)."""
    return NormalDist().inv_cdf(1.0 - p / 2.0)


def _phi(x: float) -> float:
    return math.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)


def _Phi(x: float) -> float:
    return 0.5 * (1.0 + math.erf(x / math.sqrt(2.0)))


def interval_cost(l: float, h: float) -> float:
    """integral over [l, h] of (a - l)(h - a) phi(a) da, in closed form."""
    i0 = _Phi(h) - _Phi(l)
    i1 = _phi(l) - _phi(h)                       # integral of a phi(a)
    i2 = (l * _phi(l) - h * _phi(h)) + i0        # integral of a^2 phi(a)
    return -i2 + (l + h) * i1 - l * h * i0


def table_cost(table, g: int, tp: float) -> float:
    pos = [-tp + 2.0 * tp * t / g for t in table]
    return sum(interval_cost(pos[i], pos[i + 1]) for i in range(len(table) - 1))


def optimal_table(bits: int, g: int, p: float):
    """The minimiser (ties broken towards the lexicographically smallest table, which
    matters for even g where a table and its mirror image g - T tie) and its cost."""
    levels = 1 << bits
    if g < levels - 1:
        raise ValueError("granularity must be at least 2^b - 1")
    tp = t_p(p)
    pos = [-tp + 2.0 * tp * i / g for i in range(g + 1)]
    cost = [[interval_cost(pos[i], pos[j]) if j > i else math.inf for j in range(g + 1)]
            for i in range(g + 1)]
    inf = math.inf
    # best[m][j]: cheapest way to place m intervals ending at grid point j, starting at 0
    best = [[inf] * (g + 1) for _ in range(levels)]
    prev = [[-1] * (g + 1) for _ in range(levels)]
    best[0][0] = 0.0
    eps = 1e-15
    for m in range(1, levels):
        for j in range(m, g + 1):
            for i in range(m - 1, j):
                if best[m - 1][i] == inf:
                    continue
                c = best[m - 1][i] + cost[i][j]
                # larger i later in the scan: accept only a real improvement, so the earliest
                # (smallest) predecessor wins ties -> lexicographically smallest suffix is NOT
                # implied; the final tie-break below compares whole tables
                if c < best[m][j] - eps:
                    best[m][j] = c
                    prev[m][j] = i
    table = [g]
    j = g
    for m in range(levels - 1, 0, -1):
        j = prev[m][j]
        table.append(j)
    table = tuple(reversed(table))
    mirror = tuple(g - t for t in reversed(table))
    if abs(table_cost(mirror, g, tp) - table_cost(table, g, tp)) <= 1e-13 and mirror < table:
        table = mirror
    return table, table_cost(table, g, tp)
