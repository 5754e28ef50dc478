"""Pins for the NSD quantizer oracle: published generator vectors, closed forms of the
paper's error statistics (Eqs. (unbiased), (bounded variance)) and sparsity model
(Section 3.2), exact rational arithmetic on small inputs."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield line.split()


def test_splitmix64_known_answers():
    n = 0
    for seed, idx, val in _rows("splitmix64_kat.txt"):
        assert oracle.splitmix64_at(int(seed), int(idx)) == int(val, 0)
        n += 1
    assert n == 9


def test_splitmix64_python_twin_agrees():
    from oracle.nsd import _splitmix64_py
    for seed in (0, 1, 2 ** 63, 2 ** 64 - 1, 1234567):
        for c in (0, 1, 5, 2 ** 40 + 3):
            assert _splitmix64_py(seed, c) == oracle.splitmix64_at(seed, c)


def _u(seed, n, base=0):
    return np.array([oracle.dither_u(seed, base + i) for i in range(n)], dtype=np.float64)


def test_dither_grid_open_interval_and_pairing():
    u = _u(7, 4096)
    k = u * 2 ** 24
    assert np.all(k == np.round(k)) and np.all(k.astype(np.int64) % 2 == 1)
    assert u.min() > 0.0 and u.max() < 1.0
    # element 2c uses the low, 2c+1 the high 32 bits of output c; top 23 bits of each
    for i in (0, 1, 10, 11, 2 ** 33 + 1):
        r = oracle.splitmix64_at(7, i >> 1)
        h = (r >> 32) if (i & 1) else (r & 0xFFFFFFFF)
        assert oracle.dither_u(7, i) == (2 * (h >> 9) + 1) / 2 ** 24


def test_dither_uniformity_moments_chi2_serial():
    n = 1 << 18
    u = _u(0, n)
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 4 * math.sqrt(1 / 180 / n)
    counts = np.bincount((u * 256).astype(int), minlength=256)
    chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 255 + 5 * math.sqrt(2 * 255)
    c = u - 0.5
    for lag in range(1, 33):
        r = (c[:-lag] * c[lag:]).mean() * 12
        assert abs(r) < 5 / math.sqrt(n), (lag, r)


def test_dither_independent_across_seeds_and_symmetric():
    n = 1 << 16
    a, b = _u(0, n) - 0.5, _u(1, n) - 0.5
    assert abs((a * b).mean() * 12) < 5 / math.sqrt(n)
    g = _u(oracle.derive_layer_seed(0, 0), n) - 0.5
    h = _u(oracle.derive_layer_seed(0, 1), n) - 0.5
    assert abs((g * h).mean() * 12) < 5 / math.sqrt(n)
    # the grid is symmetric about 1/2: u and 1-u are both grid points
    assert np.all(((1 - _u(3, 64)) * 2 ** 24) % 2 == 1)


def test_mean_std_closed_forms():
    m, s = oracle.mean_std(np.array([1, -1, 3, -3], dtype=np.float32))
    assert m == 0.0 and s == math.sqrt(5.0)          # population: sqrt(20/4)
    m, s = oracle.mean_std(np.array([2, 4, 4, 4, 5, 5, 7, 9], dtype=np.float32))
    assert m == 5.0 and s == 2.0                     # textbook example, population std
    x = np.arange(1, 101, dtype=np.float32)          # 1..100: var = (n^2-1)/12
    m, s = oracle.mean_std(x)
    assert m == 50.5 and abs(s - math.sqrt((100 ** 2 - 1) / 12)) < 1e-12
    # mean is removed: a constant offset does not change sigma
    y = wl.laplace(5, 1, 10000, 1e-3).astype(np.float32)
    _, s0 = oracle.mean_std(y)
    _, s1 = oracle.mean_std((y.astype(np.float64) + 0.25).astype(np.float32))
    assert abs(s1 - s0) / s0 < 1e-4
    assert abs(s0 - np.std(y.astype(np.float64))) < 1e-15
    assert oracle.mean_std(np.zeros(5, np.float32)) == (0.0, 0.0)


def test_step_size_is_s_times_sigma():
    L = wl.config1()
    _, sd = oracle.mean_std(L.delta)
    assert oracle.step_size(L.delta, 2.0) == np.float32(2.0 * sd)
    # Laplace(0,b) kept with probability p: sigma -> b sqrt(2p) = 1e-3
    assert abs(sd - 1e-3) / 1e-3 < 0.02


def test_codes_match_exact_rational_arithmetic():
    rng = np.random.default_rng(11)
    D = np.float32(0.37)
    x = np.concatenate([
        rng.normal(0, 0.5, 300), [0.0, -0.0, 0.37, -0.37, 0.185, -0.185, 1e-30, -1e-30],
        rng.normal(0, 40.0, 40), [46.9, -46.9, 47.2, -47.2, 1e6, -1e6]]).astype(np.float32)
    for seed, base in ((0, 0), (99, 7), (2 ** 64 - 1, 2 ** 33 + 5)):
        c, nnz, nsat = oracle.nsd_codes(x, seed, D, base)
        e = oracle.nsd_codes_exact_python(x, seed, D, base)
        assert np.array_equal(c, e)
        assert nnz == int((e != 0).sum())
        assert nsat >= 2 and c.max() == 127 and c.min() == -127


def test_exact_helper_rounds_like_ieee():
    from oracle.nsd import _round_to_f32
    rng = np.random.default_rng(3)
    for v in rng.normal(0, 1, 200):
        assert _round_to_f32(Fraction(float(v))) == Fraction(float(np.float32(v)))
    # ties to even at 1 + 2^-24 (between 1 and 1+2^-23) and 1 + 3*2^-24
    assert _round_to_f32(1 + Fraction(1, 2 ** 24)) == 1
    assert _round_to_f32(1 + Fraction(3, 2 ** 24)) == 1 + Fraction(2, 2 ** 23)


def test_literal_fp64_formula_is_the_same_quantizer():
    L = wl.config1()
    D = oracle.step_size(L.delta, 2.0)
    c, _, _ = oracle.nsd_codes(L.delta, 0, D)
    lit = oracle.nsd_codes_literal_f64(L.delta, 0, D)
    assert (c.astype(np.int32) != lit).mean() < 1e-5


def test_unbiased_and_variance_per_element():
    """E[eps] = 0 and E[eps^2] = Delta^2 f (1-f) <= Delta^2/4, f = frac(x/Delta)."""
    D = np.float32(1.0)
    x = np.array([0.0, 0.1, 0.25, 0.5, 0.75, 0.9, -0.3, -1.5, 2.2, 7.49], dtype=np.float32)
    M = 20000
    q = np.stack([oracle.nsd_codes(x, s, D)[0] for s in range(M)]).astype(np.float64)
    err = q * float(D) - x.astype(np.float64)
    f = x.astype(np.float64) - np.floor(x.astype(np.float64))
    var = f * (1 - f)
    assert np.all(np.abs(err.mean(axis=0)) <= 4.5 * np.sqrt(var / M) + 1e-12)
    assert np.all(np.abs(err.var(axis=0) - var) <= 6 * np.sqrt(var / M) * 0.5 + 1e-12)
    assert np.all(err.var(axis=0) <= 0.25 + 1e-12)
    assert np.all(q[:, 0] == 0)                      # x = 0 is never moved off zero
    assert np.all(q[:, 3].mean() - 0.5 < 0.02)       # x = Delta/2 -> code 1 half the time


def _laplace_zero(r):
    return 1 - (1 - math.exp(-r)) / r


def _laplace_k(r, k):
    return math.exp(-k * r) * (math.cosh(r) - 1) / r


def _gauss_zero(r):
    return math.erf(r / math.sqrt(2)) - 2 / (r * math.sqrt(2 * math.pi)) * (1 - math.exp(-r * r / 2))


def test_closed_form_table_matches_formulas():
    for dist, p, s, what, val in _rows("nsd_closed_forms.txt"):
        p, s, val = float(p), float(s), float(val)
        if dist == "gauss":
            f = _gauss_zero(s)
        else:
            r = s * math.sqrt(2 * p)
            f = (1 - p) + p * _laplace_zero(r) if what == "zero_fraction" else 2 * p * _laplace_k(r, 1)
        assert abs(f - val) < 6e-6, (dist, p, s, what, f)


@pytest.mark.parametrize("s", [1.0, 2.0, 3.0, 4.0])
def test_zero_fraction_gaussian(s):
    n = 1 << 21
    x = wl.normal(42, 1, n, 3e-3).astype(np.float32)
    D = np.float32(s * 3e-3)                         # Delta = s sigma with the true sigma
    c, nnz, _ = oracle.nsd_codes(x, 5, D)
    p0 = _gauss_zero(float(D) / 3e-3)
    assert abs((1 - nnz / n) - p0) < 5 * math.sqrt(p0 * (1 - p0) / n)


@pytest.mark.parametrize("s,keep", [(2.0, 0.5), (5.0, 0.5), (2.0, 1.0)])
def test_zero_fraction_and_code_histogram_laplace(s, keep):
    n = 1 << 21
    b = 1e-3
    x = (wl.laplace(43, 1, n, b) * wl.bernoulli(43, 2, n, keep)).astype(np.float32)
    D = np.float32(s * b * math.sqrt(2 * keep))
    c, nnz, nsat = oracle.nsd_codes(x, 9, D)
    r = float(D) / b
    p0 = (1 - keep) + keep * _laplace_zero(r)
    assert abs((1 - nnz / n) - p0) < 5 * math.sqrt(p0 * (1 - p0) / n)
    for k in (1, 2, 3):
        pk = keep * _laplace_k(r, k)
        for sign in (1, -1):
            got = (c == sign * k).mean()
            assert abs(got - pk) < 5 * math.sqrt(pk / n) + 1e-6
    assert nsat == 0 and np.abs(c).max() <= 127
    assert (c == 0).sum() >= (x == 0).sum()          # masked zeros stay zero


def test_scale_equivariance_and_step_override():
    L = wl.config1()
    D = oracle.step_size(L.delta, 2.0)
    c0, _, _ = oracle.nsd_codes(L.delta, 0, D)
    for a in (2.0 ** -7, 2.0 ** 5):
        d2 = (L.delta * np.float32(a)).astype(np.float32)
        D2 = oracle.step_size(d2, 2.0)
        assert D2 == np.float32(float(D) * a)
        assert np.array_equal(oracle.nsd_codes(d2, 0, D2)[0], c0)


def test_degenerate_steps_and_slicing():
    x = wl.laplace(1, 1, 1000, 1.0).astype(np.float32)
    for D in (0.0, -1.0, float("nan"), float("inf")):
        c, nnz, nsat = oracle.nsd_codes(x, 0, D)
        assert nnz == 0 and not c.any()
    c, _, _ = oracle.nsd_codes(x, 3, 0.5)
    part, _, _ = oracle.nsd_codes(x[101:400], 3, 0.5, index_base=101)
    assert np.array_equal(part, c[101:400])
    assert not np.array_equal(oracle.nsd_codes(x, 4, 0.5)[0], c)   # seed matters
    # larger step -> sparser (Figure 2, right)
    nz = [oracle.nsd_codes(x, 0, D)[1] for D in (0.5, 1.0, 2.0, 4.0)]
    assert nz == sorted(nz, reverse=True)
