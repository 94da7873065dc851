"""Pins for the oracle's selection (the integer program of Sec. 2.1), CPU only.

The enumeration is the definition; it is pinned by hand examples, by an
itertools re-enumeration written against the problem statement, and by the
properties the paper states (invariance to scale and bias of c, one
configuration per group, the budget inequality).  The branch and bound is then
pinned to the enumeration.
"""
import itertools

import numpy as np
import pytest


def _enumerate(c_tabs, d_tabs, budget):
    best = None
    for p in itertools.product(*[range(len(t)) for t in c_tabs]):
        c = d = 0.0
        for j, pj in enumerate(p):
            d += d_tabs[j][pj]
            c += c_tabs[j][pj]
        if d <= budget:
            key = (-c, d, p)
            if best is None or key < best[0]:
                best = (key, p, c, d)
    return None if best is None else (list(best[1]), best[2], best[3])


def _rand_tables(rng, J, Pmax, integer=False):
    c_tabs, d_tabs = [], []
    for _ in range(J):
        P = int(rng.integers(1, Pmax + 1))
        if integer:
            c = rng.integers(0, 4, P).astype(float)
            d = rng.integers(0, 4, P).astype(float)
        else:
            c = rng.uniform(0, 2, P)
            d = rng.uniform(0, 1, P) ** 3
        if rng.random() < 0.7:
            c[0], d[0] = 0.0, 0.0  # an all-high-precision column
        c_tabs.append(c)
        d_tabs.append(d)
    return c_tabs, d_tabs


def test_hand_examples(orc):
    # two groups, columns (BASE, FP8): gains 3 and 2, costs 5 and 1
    c = [[0.0, 3.0], [0.0, 2.0]]
    d = [[0.0, 5.0], [0.0, 1.0]]
    assert orc.select_bruteforce(c, d, 0.0)[0].tolist() == [0, 0]
    assert orc.select_bruteforce(c, d, 1.0)[0].tolist() == [0, 1]
    assert orc.select_bruteforce(c, d, 4.999)[0].tolist() == [0, 1]
    assert orc.select_bruteforce(c, d, 5.0)[0].tolist() == [1, 0]     # the budget is "<="
    p, cc, dd = orc.select_bruteforce(c, d, 6.0)
    assert p.tolist() == [1, 1] and cc == 5.0 and dd == 6.0
    assert orc.select_bruteforce([[1.0]], [[2.0]], 1.0) is None       # infeasible
    # ties: equal gain -> smaller d; equal both -> lexicographically smaller p
    assert orc.select_bruteforce([[1.0, 1.0]], [[2.0, 1.0]], 5.0)[0].tolist() == [1]
    assert orc.select_bruteforce([[1.0, 1.0], [0.0, 0.0]], [[1.0, 1.0], [0.0, 0.0]], 5.0)[0].tolist() == [0, 0]


@pytest.mark.parametrize("integer", [False, True])
def test_enumeration_matches_problem_statement(orc, integer):
    rng = np.random.default_rng(20 + integer)
    for _ in range(60):
        c, d = _rand_tables(rng, int(rng.integers(1, 7)), 4, integer)
        hi = sum(max(t) for t in d)
        for budget in (0.0, 0.1 * hi, 0.5 * hi, hi, 2 * hi):
            ref = _enumerate(c, d, budget)
            got = orc.select_bruteforce(c, d, budget)
            if ref is None:
                assert got is None
                continue
            assert got[0].tolist() == ref[0] and got[1] == ref[1] and got[2] == ref[2]


def test_properties(orc):
    rng = np.random.default_rng(22)
    for _ in range(30):
        c, d = _rand_tables(rng, 6, 3)
        for t in range(len(c)):
            c[t][0], d[t][0] = 0.0, 0.0
        hi = sum(max(t) for t in d)
        prev = -np.inf
        for budget in np.linspace(0, hi, 7):
            p, cc, dd = orc.select_bruteforce(c, d, budget)
            assert dd <= budget and cc >= prev         # feasible, monotone in the budget
            prev = cc
            # invariance to a positive scale and a bias of the metric (Sec. 2.3.2)
            c2 = [3.0 * t + 0.25 for t in c]
            assert orc.select_bruteforce(c2, d, budget)[0].tolist() == p.tolist()
        assert orc.select_bruteforce(c, d, 0.0)[0].tolist() == [0] * 6          # budget 0 -> all high precision
        big = orc.select_bruteforce(c, d, 10 * hi)[0].tolist()
        for j in range(6):                                                      # unconstrained -> per-group best gain
            assert c[j][big[j]] == max(c[j])


@pytest.mark.parametrize("integer", [False, True])
def test_branch_and_bound_matches_enumeration(orc, integer):
    rng = np.random.default_rng(23 + integer)
    for it in range(120):
        J = int(rng.integers(1, 11))
        c, d = _rand_tables(rng, J, 4, integer)
        hi = sum(max(t) for t in d)
        for budget in (0.0, 0.03 * hi, 0.2 * hi, 0.6 * hi, hi):
            ref = orc.select_bruteforce(c, d, budget)
            got = orc.select_bnb(c, d, budget)
            if ref is None:
                assert got is None
                continue
            assert got[0].tolist() == ref[0].tolist() and got[1] == ref[1] and got[2] == ref[2], (it, budget)


def test_branch_and_bound_large_and_absorbing(orc):
    """J = 20 binary groups (2^20 assignments) with values spread over many
    orders of magnitude, so that small terms are absorbed by rounding."""
    rng = np.random.default_rng(25)
    J = 20
    c = [np.array([0.0, float(x)]) for x in rng.uniform(0.5, 2, J)]
    d = [np.array([0.0, float(x)]) for x in 10.0 ** rng.uniform(-18, 0, J)]
    hi = sum(t[1] for t in d)
    for frac in (0.01, 0.2, 0.5):
        ref = orc.select_bruteforce(c, d, frac * hi)
        got = orc.select_bnb(c, d, frac * hi)
        assert got[0].tolist() == ref[0].tolist() and got[1:] == ref[1:]


def _fold(c_tabs, d_tabs, p):
    c = d = 0.0
    for j, pj in enumerate(p):
        d += d_tabs[j][pj]
        c += c_tabs[j][pj]
    return c, d


def test_integer_dynamic_program_matches_enumeration(orc):
    """The integer-d dynamic program against the enumeration: same (c, d), and
    its assignment is feasible and attains them (which of several equal
    assignments it returns is not specified)."""
    rng = np.random.default_rng(27)
    for it in range(200):
        J = int(rng.integers(1, 10))
        c_tabs, d_tabs = [], []
        for _ in range(J):
            P = int(rng.integers(1, 5))
            c = rng.uniform(0, 2, P) if it % 2 else rng.integers(0, 4, P).astype(float)
            d = rng.integers(0, 30, P)
            if rng.random() < 0.6:
                c[0], d[0] = 0.0, 0
            c_tabs.append(c)
            d_tabs.append(d)
        hi = int(sum(max(t) for t in d_tabs))
        for budget in (0, hi // 20, hi // 3, (2 * hi) // 3, hi, 2 * hi + 1):
            ref = orc.select_bruteforce(c_tabs, [t.astype(float) for t in d_tabs], float(budget))
            got = orc.select_dp_integer(c_tabs, d_tabs, budget)
            if ref is None:
                assert got is None
                continue
            assert got[1] == ref[1] and got[2] == ref[2], (it, budget)
            assert _fold(c_tabs, d_tabs, got[0]) == (ref[1], float(ref[2]))


def test_integer_dynamic_program_absorbing_gains(orc):
    """Gains spread over many orders of magnitude (small ones absorbed by
    rounding): the dynamic program still holds the enumeration's left-fold maximum."""
    rng = np.random.default_rng(28)
    for _ in range(10):
        J = 14
        c = [np.array([0.0, float(x)]) for x in 10.0 ** rng.uniform(-17, 1, J)]
        d = [np.array([0, int(x)]) for x in rng.integers(1, 50, J)]
        hi = int(sum(t[1] for t in d))
        for budget in (hi // 50, hi // 5, hi // 2):
            ref = orc.select_bruteforce(c, [t.astype(float) for t in d], float(budget))
            got = orc.select_dp_integer(c, d, budget)
            assert got[1] == ref[1] and got[2] == ref[2]


def test_branch_and_bound_moderate_sizes_against_dynamic_program(orc):
    """Two independent exact methods beyond the reach of the enumeration: the
    plain depth-first search and the integer dynamic program agree on (c, d) at
    J = 40 binary groups with tight budgets."""
    rng = np.random.default_rng(29)
    J = 40
    c = [np.array([0.0, float(x)]) for x in rng.uniform(0.5, 2.0, J)]
    d = [np.array([0, int(x)]) for x in rng.integers(1, 1000, J)]
    hi = int(sum(t[1] for t in d))
    for budget in (hi // 100, hi // 30):
        a = orc.select_bnb(c, [t.astype(float) for t in d], float(budget), 200_000_000)
        b = orc.select_dp_integer(c, d, budget)
        assert a[1] == b[1] and a[2] == b[2]
        assert _fold(c, d, b[0]) == (a[1], a[2])
