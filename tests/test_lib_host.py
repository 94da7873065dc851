"""Host-side checks of the C-ABI library that need no GPU: the shared object
loads and exports every symbol the header declares, argument errors are
reported as status codes, and the exact selection agrees with the oracle's
enumeration and branch and bound."""
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ampq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ampq_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(ampq):
    names = _declared_symbols()
    assert len(names) >= 20 and set(names) == set(ampq.EXPORTS)
    L = ampq.lib()
    for n in names:
        assert getattr(L, n) is not None, n


def test_status_strings_and_contextless_calls(ampq):
    L = ampq.lib()
    assert L.ampq_strerror(0) == b"ok"
    for code in range(-8, 0):
        assert L.ampq_strerror(code) not in (b"ok", b"unknown status")
    assert ampq.budget_from_tau(0.1, [1.0, 2.0, 3.0]) == pytest.approx(0.01 * 14 / 3, rel=1e-15)
    with pytest.raises(ampq.AmpqError):
        ampq.budget_from_tau(-1.0, [1.0])
    assert L.ampq_destroy(None) == 0
    assert L.ampq_score(None) == ampq.ERR_INVALID


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
            c[0], d[0] = 0.0, 0.0
        c_tabs.append(c)
        d_tabs.append(d)
    return c_tabs, d_tabs


@pytest.mark.parametrize("integer", [False, True])
def test_select_matches_enumeration(ampq, orc, integer):
    rng = np.random.default_rng(40 + integer)
    for it in range(150):
        c, d = _rand_tables(rng, int(rng.integers(1, 9)), 5, integer)
        hi = sum(max(t) for t in d)
        for budget in (0.0, 0.05 * hi, 0.3 * hi, 0.7 * hi, hi, 2 * hi + 1):
            ref = orc.select_bruteforce(c, d, budget)
            got = ampq.select_tables(c, d, budget)
            if ref is None:
                assert got is None
                continue
            assert got[0].tolist() == ref[0].tolist() and got[1] == ref[1] and got[2] == ref[2], (it, budget)


def test_select_absorbing_magnitudes(ampq, orc):
    """Terms spread over 18 orders of magnitude: partial sums absorb small
    terms, so dominated prefixes can tie after rounding; the result must still
    be the enumeration's."""
    rng = np.random.default_rng(42)
    for _ in range(20):
        J = 12
        c = [np.array([0.0, float(x)]) for x in 10.0 ** rng.uniform(-17, 1, J)]
        d = [np.array([0.0, float(x)]) for x in 10.0 ** rng.uniform(-18, 0, J)]
        hi = sum(t[1] for t in d)
        for frac in (1e-6, 0.01, 0.3, 1.0):
            ref = orc.select_bruteforce(c, d, frac * hi)
            got = ampq.select_tables(c, d, frac * hi)
            assert got[0].tolist() == ref[0].tolist() and got[1:] == ref[1:]


@pytest.mark.parametrize("J,P", [(64, 2), (80, 2), (32, 16)])
def test_select_large_matches_integer_dynamic_program(ampq, orc, J, P):
    """Sizes of the format/budget sweep (64 sub-graphs), of the 70B-shaped model
    (80) and of many-column groups: loss MSEs on an integer grid, so that the
    oracle's textbook dynamic program over the budget -- a method that shares
    nothing with the library's solver -- gives the exact optimum.  (c, d) must
    match; the library's assignment must attain them within the budget."""
    rng = np.random.default_rng(43)
    c = [np.concatenate([[0.0], np.sort(rng.uniform(0.5, 2.0, P - 1))]) for _ in range(J)]
    d = [np.concatenate([[0], np.sort((rng.uniform(0, 1, P - 1) ** 2 * 2000).astype(np.int64))]) for _ in range(J)]
    df = [t.astype(float) for t in d]
    hi = int(sum(t[-1] for t in d))
    prev = -1.0
    for frac in (0.01, 0.05, 0.2, 0.5):
        budget = int(frac * hi)
        ref = orc.select_dp_integer(c, d, budget)
        got = ampq.select_tables(c, df, float(budget))
        assert got[1] == ref[1] and got[2] == float(ref[2]), (frac, got[1:], ref[1:])
        cs = ds = 0.0
        for j, pj in enumerate(got[0]):
            ds += df[j][pj]
            cs += c[j][pj]
        assert (cs, ds) == (got[1], got[2]) and ds <= budget and got[1] >= prev
        prev = got[1]


@pytest.mark.parametrize("J,P,fracs", [(40, 2, (0.012, 0.06, 0.15)), (24, 4, (0.01, 0.03)), (64, 2, (0.0015, 0.01, 0.03)), (80, 2, (0.01,))])
def test_select_matches_plain_branch_and_bound(ampq, orc, J, P, fracs):
    """Real-valued loss MSEs beyond the reach of the enumeration, at budgets tight
    enough for the oracle's plain depth-first search: the assignment itself,
    tie-break included, must match."""
    rng = np.random.default_rng(45)
    c = [np.concatenate([[0.0], np.sort(rng.uniform(0.5, 2.0, P - 1))]) for _ in range(J)]
    d = [np.concatenate([[0.0], np.sort(rng.uniform(0, 1, P - 1) ** 2)]) for _ in range(J)]
    hi = sum(t[-1] for t in d)
    for frac in fracs:
        ref = orc.select_bnb(c, d, frac * hi, 400_000_000)
        got = ampq.select_tables(c, d, frac * hi)
        assert got[0].tolist() == ref[0].tolist() and got[1] == ref[1] and got[2] == ref[2]


def test_select_ties_at_large_J_resolve_lexicographically(ampq):
    """A case whose answer is known in closed form at a size no enumeration
    reaches: 72 identical groups with columns (0, 0), (c, d), (c, d).  Every
    choice of k groups in low precision gains the same, so the ordering rules
    decide: smaller d cannot separate them either, and the lexicographically
    smallest assignment puts column 1 (never its twin, column 2) in the LAST k
    groups.  Dyadic values keep every sum exact."""
    J, c, d = 72, 1.25, 0.5
    c_tabs = [np.array([0.0, c, c])] * J
    d_tabs = [np.array([0.0, d, d])] * J
    for k in (0, 1, 7, 36, 71, 72):
        p, ct, dt = ampq.select_tables(c_tabs, d_tabs, k * d + 0.25)
        assert p.tolist() == [0] * (J - k) + [1] * k and ct == k * c and dt == k * d
    # one group made slightly cheaper must be taken first; one made slightly more gainful too
    d2 = [t.copy() for t in d_tabs]
    d2[10] = np.array([0.0, d - 0.125, d])
    p, ct, dt = ampq.select_tables(c_tabs, d2, 3 * d)
    assert p.tolist() == [0] * 10 + [1] + [0] * (J - 13) + [1, 1] and dt == 3 * d - 0.125
    c2 = [t.copy() for t in c_tabs]
    c2[20] = np.array([0.0, c, c + 0.5])
    p, ct, dt = ampq.select_tables(c2, d_tabs, 2 * d)
    assert p.tolist() == [0] * 20 + [2] + [0] * (J - 22) + [1] and ct == 2 * c + 0.5


def test_select_edge_cases(ampq):
    assert ampq.select_tables([[1.0]], [[2.0]], 1.0) is None
    p, c, d = ampq.select_tables([], [], 0.0)
    assert len(p) == 0 and c == 0.0 and d == 0.0
    with pytest.raises(ampq.AmpqError):
        ampq.select_tables([[1.0]], [[-1.0]], 1.0)       # negative loss MSE
    with pytest.raises(ampq.AmpqError):
        ampq.select_tables([[float("nan")]], [[0.0]], 1.0)
    # invariance to scale and bias of the metric
    rng = np.random.default_rng(44)
    c, d = _rand_tables(rng, 10, 4)
    hi = sum(max(t) for t in d)
    a = ampq.select_tables(c, d, 0.4 * hi)
    b = ampq.select_tables([2.5 * t + 1.0 for t in c], d, 0.4 * hi)
    assert a[0].tolist() == b[0].tolist()


def test_header_is_plain_c(tmp_path):
    """include/ampq.h compiles as C99 and as C++ on its own (no CUDA, no torch
    types), and a C program can name every declared entry point."""
    import subprocess

    hdr = os.path.join(ROOT, "include", "ampq.h")
    names = _declared_symbols()
    src = tmp_path / "use.c"
    src.write_text('#include "%s"\nvoid *table[] = {%s};\nint main(void) { return AMPQ_OK; }\n'
                   % (hdr, ", ".join("(void *)%s" % n for n in names)))
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-c", str(src), "-o", str(tmp_path / "use.o")])
    subprocess.check_call(["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr])
