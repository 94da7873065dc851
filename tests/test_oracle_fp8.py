"""Pins for the oracle's FP8 grid and cast (CPU only).

The grid is pinned to the constants in tests/golden/format_constants.txt and
to torch's own float8 dtypes (an independent library decode); the cast is
pinned to a brute-force nearest-grid-point search over the decoded grid and to
torch's round-to-nearest-even cast inside the finite range.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from conftest import read_golden

FMTS = {"e4m3": 1, "e5m2": 2}
TORCH_DT = {1: torch.float8_e4m3fn, 2: torch.float8_e5m2}


def _pow(s):
    s = s.strip()
    if s.startswith("2^"):
        return Fraction(2) ** int(s[2:])
    return Fraction(s)


def test_alpha_matches_paper_closed_form(orc):
    g = read_golden("format_constants.txt")
    for m in (3, 2, 7):
        assert orc.alpha(m) == float(Fraction(g["alpha.m%d" % m]))  # 1/(12*4^m) rounds once
    assert orc.mantissa_bits(orc.FMT_E4M3) == int(g["e4m3.mantissa_bits"])
    assert orc.mantissa_bits(orc.FMT_E5M2) == int(g["e5m2.mantissa_bits"])
    assert orc.mantissa_bits(orc.FMT_BASE) == int(g["bf16.mantissa_bits"])


@pytest.mark.parametrize("name", ["e4m3", "e5m2"])
def test_grid_constants(orc, name):
    g = read_golden("format_constants.txt")
    f = FMTS[name]
    assert Fraction(orc.fmax(f)) == _pow(g[name + ".max"])
    assert Fraction(orc.fp8_decode(f, int(g[name + ".max_code"], 16))) == _pow(g[name + ".max"])
    assert Fraction(orc.fp8_decode(f, int(g[name + ".min_normal_code"], 16))) == _pow(g[name + ".min_normal"])
    assert Fraction(orc.fp8_decode(f, int(g[name + ".min_subnormal_code"], 16))) == _pow(g[name + ".min_subnormal"])
    vals = [orc.fp8_decode(f, c) for c in range(256)]
    finite = [v for v in vals if np.isfinite(v)]
    assert len(finite) == int(g[name + ".finite_codes"])
    assert max(finite) == float(_pow(g[name + ".max"]))
    if name == "e4m3":
        assert np.isnan(vals[int(g["e4m3.nan_code"], 16)]) and np.isnan(vals[0xFF])
    else:
        assert vals[int(g["e5m2.inf_code"], 16)] == float("inf") and vals[0xFC] == float("-inf")
        assert all(np.isnan(vals[c]) for c in (0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF))


@pytest.mark.parametrize("f", [1, 2])
def test_decode_matches_torch_float8(orc, f):
    ref = torch.arange(256, dtype=torch.uint8).view(TORCH_DT[f]).to(torch.float64).numpy()
    got = np.array([orc.fp8_decode(f, c) for c in range(256)])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    # the sign of zero survives
    assert np.signbit(got[0x80]) and got[0x80] == 0.0 and not np.signbit(got[0])


@pytest.mark.parametrize("f", [1, 2])
def test_grid_structure(orc, f):
    """Monotone in the code, symmetric, 2^m steps per binade, spacing doubles."""
    m = orc.mantissa_bits(f)
    pos = [orc.fp8_decode(f, c) for c in range(128)]
    pos = [v for v in pos if np.isfinite(v)]
    assert all(b > a for a, b in zip(pos, pos[1:]))
    for c in range(128):
        v = orc.fp8_decode(f, c)
        if np.isfinite(v):
            assert orc.fp8_decode(f, c | 0x80) == -v
    # spacing inside each binade is constant and doubles from one to the next
    steps = np.diff(pos)
    n = 1 << m
    assert np.all(steps[: 2 * n] == steps[0])              # subnormals + first binade
    for b in range(2, (len(steps) + n - 1) // n):
        blk = steps[b * n: (b + 1) * n]
        assert np.all(blk == blk[0]) and blk[0] == 2 * steps[(b - 1) * n]


def _nearest_code_bruteforce(orc, f, y, grid):
    """Definition of the cast: the finite grid point nearest to y, ties to the
    even code, beyond the largest finite value -> that value; sign kept."""
    sign = 0x80 if np.signbit(y) else 0
    a = Fraction(abs(float(y))) if np.isfinite(y) else None
    codes = [c for c in range(128) if np.isfinite(grid[c])]
    if a is None or a >= Fraction(grid[codes[-1]]):
        return sign | codes[-1]
    best, bd = None, None
    for c in codes:
        d = abs(Fraction(grid[c]) - a)
        if bd is None or d < bd or (d == bd and c % 2 == 0 and best % 2 == 1):
            best, bd = c, d
    return sign | best


@pytest.mark.parametrize("f", [1, 2])
def test_encode_roundtrip_and_bruteforce(orc, f):
    grid = [orc.fp8_decode(f, c) for c in range(256)]
    for c in range(256):
        if np.isfinite(grid[c]):
            assert orc.fp8_encode(f, grid[c]) == c, hex(c)
    rng = np.random.default_rng(0)
    fm = orc.fmax(f)
    ys = []
    # every midpoint between neighbours, and its two fp32 neighbours
    pos = sorted(v for v in grid[:128] if np.isfinite(v))
    for a, b in zip(pos, pos[1:]):
        mid = np.float32((a + b) / 2)
        ys += [mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(np.inf))]
    ys += [np.float32(fm), np.nextafter(np.float32(fm), np.float32(np.inf)), np.float32(fm * 1.5),
           np.float32(np.inf), np.float32(3e38), np.float32(1e-45), np.float32(pos[1] / 2),
           np.nextafter(np.float32(pos[1] / 2), np.float32(1)), np.float32(0.0)]
    ys += list(np.exp(rng.uniform(np.log(pos[1] / 8), np.log(fm * 2), 3000)).astype(np.float32))
    ys += list(rng.standard_normal(2000).astype(np.float32) * 50)
    for y in ys:
        for s in (1.0, -1.0):
            yy = np.float32(s * y)
            assert orc.fp8_encode(f, float(yy)) == _nearest_code_bruteforce(orc, f, yy, grid), float(yy)
    assert orc.fp8_encode(f, -0.0) == 0x80
    # half the smallest subnormal ties to zero (even), anything above goes up
    assert orc.fp8_encode(f, pos[1] / 2) == 0
    assert orc.fp8_encode(f, float(np.nextafter(np.float32(pos[1] / 2), np.float32(1)))) == 1


@pytest.mark.parametrize("f", [1, 2])
def test_encode_matches_torch_cast_in_range(orc, f):
    """torch's float8 cast is round-to-nearest-even; inside the finite range it
    must agree with the oracle code for code."""
    rng = np.random.default_rng(1)
    fm = orc.fmax(f)
    y = np.concatenate([
        rng.uniform(-fm, fm, 20000), rng.standard_normal(20000) * fm / 100,
        np.exp(rng.uniform(np.log(1e-8), np.log(fm), 20000))]).astype(np.float32)
    ref = torch.from_numpy(y).to(TORCH_DT[f]).view(torch.uint8).numpy()
    got = np.array([orc.fp8_encode(f, float(v)) for v in y], dtype=np.uint8)
    assert np.array_equal(ref, got)
    # and the vectorised entry point is the same function with scale 1
    assert np.array_equal(orc.codes(y, f, 1.0), got)


def test_scales(orc):
    """scale = fl32(amax/fmax), inv = fl32(fmax/amax): IEEE fp32 divisions."""
    rng = np.random.default_rng(2)
    for f in (1, 2):
        fm = np.float32(orc.fmax(f))
        for a in list(rng.uniform(1e-3, 1e3, 200).astype(np.float32)) + [np.float32(448), np.float32(57344)]:
            s, i = orc.scales(f, a)
            assert s == np.float32(a) / fm and i == fm / np.float32(a)
        assert orc.scales(f, 0.0) == (np.float32(1), np.float32(1))
        assert orc.scales(f, 1e-42) == (np.float32(1), np.float32(1))  # fmax/amax overflows
    assert orc.scales(1, 448.0 * 4) == (np.float32(4), np.float32(0.25))
