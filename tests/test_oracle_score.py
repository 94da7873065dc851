"""Pins for the oracle's amax / cast / error / weighting / reduction (CPU only).

Each test fixes the oracle to something it does not compute itself: exact
rational arithmetic on tiny inputs (with a brute-force nearest-grid search for
the cast), closed forms (zero error on the grid, ulp^2/12 rounding variance,
the Gaussian expectation of the sensitivity), and exact scaling laws.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from conftest import read_golden

TORCH_DT = {1: torch.float8_e4m3fn, 2: torch.float8_e5m2}


def _grid(f):
    """(code, value) of every finite non-negative grid point, from torch's float8."""
    v = torch.arange(128, dtype=torch.uint8).view(TORCH_DT[f]).to(torch.float64).numpy()
    return [(c, Fraction(float(x))) for c, x in enumerate(v) if np.isfinite(x)]


def _quantise_exact(y, grid):
    """Nearest grid value to the fp32 number y (ties -> even code, saturating)."""
    a = Fraction(abs(float(y)))
    top = grid[-1][1]
    if a >= top:
        q = top
    else:
        best = None
        for c, v in grid:
            d = abs(v - a)
            if best is None or d < best[0] or (d == best[0] and c % 2 == 0 and best[1] % 2 == 1):
                best = (d, c, v)
        q = best[2]
    return -q if np.signbit(y) else q


def _bf16_round(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)


def _as_oracle_array(t):
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("f", [1, 2])
def test_tiny_against_rational_arithmetic(orc, dtype, f):
    rng = np.random.default_rng(10 + f)
    n = 97
    z = torch.from_numpy((rng.standard_normal(n) * np.exp(rng.uniform(-6, 3, n))).astype(np.float32)).to(dtype)
    g = torch.from_numpy((rng.standard_normal(n) * 1e-2).astype(np.float32)).to(dtype)
    z[5] = 0.0
    z[6] = -0.0
    zf = z.to(torch.float32).numpy()
    gf = g.to(torch.float32).numpy()
    amax = np.float32(np.max(np.abs(zf)))
    fm = np.float32(read_golden("format_constants.txt")["e4m3.max" if f == 1 else "e5m2.max"])
    scale, inv = np.float32(amax / fm), np.float32(fm / amax)
    grid = _grid(f)
    S = Fraction(0)
    D = Fraction(0)
    for zk, gk in zip(zf, gf):
        y = np.float32(zk) * inv  # fp32 multiply
        e = _quantise_exact(y, grid) * Fraction(float(scale)) - Fraction(float(zk))
        S += (Fraction(float(zk)) * Fraction(float(gk))) ** 2
        D += (Fraction(float(gk)) * e) ** 2
    a, sc, iv, seg = orc.score_operand(_as_oracle_array(z), _as_oracle_array(g), 1, False, [f])
    assert a == amax and sc[0] == scale and iv[0] == inv
    assert abs(seg[0, 0] - float(S)) <= 1e-13 * float(S)
    assert abs(seg[0, 1] - float(D)) <= 1e-12 * float(D)


@pytest.mark.parametrize("f", [1, 2])
@pytest.mark.parametrize("k", [-5, 0, 7])
def test_zero_error_on_grid(orc, f, k):
    """A tensor of grid values times 2^k that contains +-fmax*2^k has scale 2^k
    exactly, so every element is reproduced and D = 0 while S > 0."""
    rng = np.random.default_rng(3)
    grid = np.array([float(v) for _, v in _grid(f)])
    vals = rng.choice(grid, 4096) * rng.choice([-1.0, 1.0], 4096) * 2.0 ** k
    vals[0], vals[1] = grid[-1] * 2.0 ** k, -grid[-1] * 2.0 ** k
    v = vals.astype(np.float32)
    g = rng.standard_normal(4096).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(v, g, 1, False, [f])
    assert sc[0] == np.float32(2.0 ** k) and iv[0] == np.float32(2.0 ** -k)
    assert seg[0, 1] == 0.0 and seg[0, 0] > 0.0
    # and the codes are the grid codes
    assert np.array_equal(orc.codes(v, f, iv[0]) & 0x7F,
                          np.array([orc.fp8_encode(f, float(abs(x) / 2.0 ** k)) for x in v], np.uint8))


@pytest.mark.parametrize("f", [1, 2])
def test_uniform_binade_gives_closed_form_noise_variance(orc, f):
    """Values on a fine uniform lattice over [1,2) plus one element equal to
    fmax (so scale = 1): the rounding error is the textbook sawtooth, whose
    mean square over one grid cell of width u = 2^-m and lattice step h is
    h^2 (2 sum_{j<c/2} j^2 + (c/2)^2) / c with c = u/h, i.e. u^2/12 (1 + 2 h^2/u^2).
    With g = 1 this is the noise model's alpha_f at |z| = 1, and D / (alpha_f S)
    tends to 1 / E[y^2] = 3/7."""
    gold = read_golden("format_constants.txt")
    m = orc.mantissa_bits(f)
    alpha = float(Fraction(gold["alpha.m%d" % m]))
    hbits = 12
    n = 1 << hbits
    y = (1.0 + np.arange(n) / n).astype(np.float32)
    v = np.concatenate([y, np.array([orc.fmax(f)], np.float32)])
    g = np.ones_like(v)
    g[-1] = 0.0  # the pinning element carries no weight
    a, sc, iv, seg = orc.score_operand(v, g, 1, False, [f])
    assert sc[0] == 1.0 and iv[0] == 1.0
    c = n >> m                      # lattice points per grid cell
    h = Fraction(1, n)
    cell = h * h * (2 * sum(j * j for j in range(1, c // 2)) + (c // 2) ** 2)
    expect = cell * (1 << m)        # 2^m cells in [1,2)
    assert Fraction(seg[0, 1]) == expect          # exact: every term is a dyadic rational
    assert abs(seg[0, 1] / n - alpha) < 1e-4 * alpha
    assert abs(seg[0, 1] / (alpha * seg[0, 0]) - 3.0 / 7.0) < 2e-3


def test_gaussian_expectation_of_sensitivity(orc):
    """iid z ~ N(0, s^2), g ~ N(0, t^2): E[S] = N s^2 t^2 with relative standard
    deviation sqrt(8/N); and the measured term sits inside the band the noise
    model allows, (1/4) alpha S < D < alpha S, near alpha S / E[(1+u)^2]."""
    rng = np.random.default_rng(4)
    N, s, t = 1 << 20, 0.7, 3e-3
    z = (rng.standard_normal(N) * s).astype(np.float32)
    g = (rng.standard_normal(N) * t).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(z, g, 1, False, [1, 2])
    expect = N * s * s * t * t
    assert abs(seg[0, 0] - expect) < 5 * np.sqrt(8.0 / N) * expect
    for col, m in ((1, 3), (2, 2)):
        ratio = seg[0, col] / (orc.alpha(m) * seg[0, 0])
        assert 0.25 < ratio < 1.0
        assert 0.38 < ratio < 0.62


def test_measured_error_against_quadrature(orc):
    """Expected D for Gaussian data from a 1-D quadrature of the deterministic
    rounding-error function (computed here with torch's float8 cast, not the
    oracle) against the Gaussian density."""
    rng = np.random.default_rng(5)
    N, t = 1 << 21, 1e-3
    z = rng.standard_normal(N).astype(np.float32)
    z[0] = 5.0  # pins amax
    z = np.clip(z, -5, 5)
    g = (rng.standard_normal(N) * t).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(z, g, 1, False, [1])
    x = np.linspace(-5, 5, 2_000_001)
    y = torch.from_numpy((x.astype(np.float32) * iv[0]))
    q = y.to(torch.float8_e4m3fn).to(torch.float64).numpy() * float(sc[0])
    err2 = (q - x) ** 2
    pdf = np.exp(-x * x / 2) / np.sqrt(2 * np.pi)
    expect = N * t * t * np.trapezoid(err2 * pdf, x)
    assert abs(seg[0, 1] - expect) < 0.02 * expect


def test_power_of_two_scaling_laws(orc):
    rng = np.random.default_rng(6)
    z = rng.standard_normal(5000).astype(np.float32)
    g = (rng.standard_normal(5000) * 1e-3).astype(np.float32)
    _, _, iv0, s0 = orc.score_operand(z, g, 1, False, [1, 2])
    for a, b in ((3, -2), (-7, 5)):
        z2 = (z * np.float32(2.0 ** a)).astype(np.float32)
        g2 = (g * np.float32(2.0 ** b)).astype(np.float32)
        _, _, iv1, s1 = orc.score_operand(z2, g2, 1, False, [1, 2])
        assert np.array_equal(s1, s0 * 2.0 ** (2 * (a + b)))       # exact
        for f, i0, i1 in ((1, iv0[0], iv1[0]), (2, iv0[1], iv1[1])):
            assert np.array_equal(orc.codes(z, f, i0), orc.codes(z2, f, i1))
    # sign flips change nothing; a permutation only changes the summation order
    _, _, _, s2 = orc.score_operand(-z, g, 1, False, [1, 2])
    assert np.array_equal(s2, s0)
    p = rng.permutation(5000)
    _, _, _, s3 = orc.score_operand(z[p], g[p], 1, False, [1, 2])
    assert np.allclose(s3, s0, rtol=1e-12, atol=0)


def test_segments_samples_and_shared_values(orc):
    """Per-sample operands: sample r owns row r and one amax covers all rows.
    Shared operands: the same values weighted by each sample's gradient.  Both
    are additive over a split of the element range."""
    rng = np.random.default_rng(7)
    R, n = 3, 1000
    x = rng.standard_normal((R, n)).astype(np.float32)
    gx = (rng.standard_normal((R, n)) * 1e-3).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(x, gx, R, True, [1])
    assert a == np.max(np.abs(x))
    for r in range(R):
        one = orc.score_segment(x[r], gx[r], [1], sc, iv)
        assert np.array_equal(one, seg[r])
        left = orc.score_segment(x[r, :400], gx[r, :400], [1], sc, iv)
        right = orc.score_segment(x[r, 400:], gx[r, 400:], [1], sc, iv)
        assert np.allclose(left + right, seg[r], rtol=1e-13, atol=0)
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    gw = (rng.standard_normal((R, n)) * 1e-3).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(w, gw, R, False, [1])
    for r in range(R):
        assert np.array_equal(orc.score_segment(w, gw[r], [1], sc, iv), seg[r])
    # a preset amax (static scale) below the data saturates instead of wrapping
    a2, sc2, iv2, seg2 = orc.score_operand(w, gw, R, False, [1], amax_preset=float(a) / 4)
    assert a2 == np.float32(float(a) / 4)
    assert np.all(np.abs(torch.from_numpy(orc.codes(w, 1, iv2[0]) & 0x7F).numpy()) <= 0x7E)
    assert seg2[0, 1] > seg[0, 1]


def test_layer_combine_hand_example(orc):
    """s^r = S(op0,r) + S(op1,r); s = mean_r; d_model = alpha_f s; d_meas = mean
    of the summed measured terms; the high-precision format costs 0."""
    gold = read_golden("format_constants.txt")
    seg0 = np.array([[1.0, 2.0, 0.5], [3.0, 4.0, 1.5]])
    seg1 = np.array([[10.0, 20.0, 5.0], [30.0, 40.0, 15.0]])
    out = orc.layer_combine(seg0, seg1, [orc.FMT_BASE, orc.FMT_E4M3, orc.FMT_E5M2])
    assert list(out["s_per_sample"]) == [11.0, 33.0]
    assert out["s_mean"] == 22.0
    assert out["d_model"][0] == 0.0
    assert out["d_model"][1] == 22.0 * float(Fraction(gold["alpha.m3"]))
    assert out["d_model"][2] == 22.0 * float(Fraction(gold["alpha.m2"]))
    assert out["d_meas_per_sample"].tolist() == [[0.0, 22.0, 5.5], [0.0, 44.0, 16.5]]
    assert out["d_meas"].tolist() == [0.0, 33.0, 11.0]


def test_group_costs_and_budget_hand_examples(orc):
    d_layer = np.array([[0.0, 1.0], [0.0, 10.0], [0.0, 100.0]])
    # group of layers (2, 0) with all four configurations, column p = (f of layer 2, f of layer 0)
    Q = np.array([[0, 1, 0, 1], [0, 0, 1, 1]], dtype=np.uint8)
    assert orc.group_costs([2, 0], Q, d_layer).tolist() == [0.0, 100.0, 1.0, 101.0]
    # J = L special case: single-layer groups
    for l in range(3):
        assert orc.group_costs([l], np.array([[0, 1]], np.uint8), d_layer).tolist() == [0.0, d_layer[l, 1]]
    assert orc.budget_from_tau(0.1, [1.0, 2.0, 3.0]) == pytest.approx(0.01 * 14.0 / 3.0, rel=1e-15)
    assert orc.budget_from_tau(0.0, [1.0, 2.0]) == 0.0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("f", [1, 2])
def test_fake_quant_pins(orc, dtype, f):
    """The quantised operand z^: equals the rational nearest-grid value times the
    scale (rounded once to fp32, then to the storage type by torch's own cast),
    reproduces tensors already on the grid, is idempotent, and its error squares
    to the oracle's own D."""
    rng = np.random.default_rng(21)
    grid = _grid(f)
    x = (rng.standard_normal(300) * np.exp(rng.uniform(-6, 3, 300))).astype(np.float32)
    t = torch.from_numpy(x).to(dtype)
    v = _as_oracle_array(t)
    a = orc.amax(v)
    sc, iv = orc.scales(f, a)
    zh = orc.fake_quant(v, f, sc, iv)
    z64 = t.to(torch.float64).numpy()
    for k in range(300):   # rational arithmetic, independent of the C code
        y = np.float32(Fraction(float(z64[k])) * Fraction(float(iv)))
        want = np.float32(_quantise_exact(y, grid) * Fraction(float(sc)))
        want = torch.tensor([want]).to(dtype)
        assert _as_oracle_array(want)[0] == zh[k], k
    # error of z^ squares to D (fp32 storage: only the one rounding of the product differs)
    if dtype == torch.float32:
        g = rng.standard_normal(300).astype(np.float32)
        seg = orc.score_segment(v, g, [f], [sc], [iv])
        d = float(np.sum((g.astype(np.float64) * (zh.astype(np.float64) - z64)) ** 2))
        assert d == pytest.approx(seg[1], rel=1e-5)
    # idempotent under the same scale
    assert np.array_equal(orc.fake_quant(zh, f, sc, iv), zh)
    # a tensor on the grid (scale a power of two) comes back unchanged
    gv = np.array([float(q) for _, q in grid])
    on = (rng.choice(gv, 512) * rng.choice([-1.0, 1.0], 512) * 0.25).astype(np.float32)
    on[0] = gv[-1] * 0.25
    ton = torch.from_numpy(on).to(dtype)
    von = _as_oracle_array(ton)   # every FP8 value fits the 8 significant bits of bf16
    s2, i2 = orc.scales(f, orc.amax(von))
    assert s2 == np.float32(0.25)
    assert np.array_equal(orc.fake_quant(von, f, s2, i2), von)


@pytest.mark.parametrize("f", [1, 2])
def test_power_of_two_scale_pins(orc, f):
    """The power-of-two scale: a power of two, just large enough that amax does
    not saturate (fmax*p >= amax > fmax*p/2, checked in rational arithmetic),
    equal to the amax scale when amax is fmax times a power of two, neutral for 0
    and for magnitudes whose scale is not a normal fp32."""
    fmax = Fraction(orc.fmax(f))
    rng = np.random.default_rng(8)
    for a in list(np.exp(rng.uniform(-60, 60, 200)).astype(np.float32)) + [np.float32(1.0), np.float32(448.0)]:
        sc, iv = orc.scales(f, a, pow2=True)
        m, e = np.frexp(float(sc))
        assert m == 0.5 and float(sc) * float(iv) == 1.0
        assert fmax * Fraction(float(sc)) >= Fraction(float(a)) > fmax * Fraction(float(sc)) / 2
    for k in (-20, 0, 13):
        a = np.float32(float(fmax) * 2.0 ** k)
        assert orc.scales(f, a, pow2=True) == orc.scales(f, a) == (np.float32(2.0 ** k), np.float32(2.0 ** -k))
        up = np.nextafter(a, np.float32(np.inf))
        assert orc.scales(f, up, pow2=True)[0] == np.float32(2.0 ** (k + 1))
    assert orc.scales(f, 0.0, pow2=True) == (1.0, 1.0)
    assert orc.scales(f, np.float32(1e-44), pow2=True) == (1.0, 1.0)
    # with a power-of-two scale the scaled value is exact, so the codes of z and of 4z agree
    v = (rng.standard_normal(1000) * 3).astype(np.float32)
    a, sc, iv, seg = orc.score_operand(v, np.ones(1000, np.float32), 1, False, [f], pow2=True)
    a4, sc4, iv4, seg4 = orc.score_operand(4 * v, np.ones(1000, np.float32), 1, False, [f], pow2=True)
    assert sc4[0] == 4 * sc[0] and seg4[0, 1] == 16 * seg[0, 1]
    assert np.array_equal(orc.codes(v, f, iv[0]), orc.codes(4 * v, f, iv4[0]))
