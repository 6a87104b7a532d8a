"""Pins for the oracle's building blocks: each is checked against a textbook or
library routine, a closed form, or a convention the paper states -- never
against a retyped copy of the oracle's own formula."""
from fractions import Fraction

import numpy as np
import pytest
import scipy.special as sps

pytestmark = pytest.mark.filterwarnings("ignore::RuntimeWarning")


# ---- schedules (Eq. sdar, UniformRSD, linear variant) -------------------------
@pytest.mark.parametrize("L", [1, 2, 4, 8, 16, 32])
@pytest.mark.parametrize("delta,nu", [(1.1, 0.7), (2.0, 0.7), (1.0, 0.05), (4.0, 1.5)])
def test_exp_schedule_constraints(oracle, L, delta, nu):
    w = oracle.make_schedule(1, delta, nu, L)
    # the normaliser mu is defined by sum_i exp(-nu i - mu) = L  =>  sum omega_i = delta L
    assert np.isclose(w.sum(), delta * L, rtol=1e-13)
    # geometric decay with ratio exp(-nu), strictly decreasing (annealing)
    if L > 1:
        assert np.allclose(w[1:] / w[:-1], np.exp(-nu), rtol=1e-12)
        assert np.all(np.diff(w) < 0)
    assert np.all(w > 0)


def test_exp_schedule_limits(oracle):
    # nu -> 0 recovers the uniform schedule omega_i = delta
    w = oracle.make_schedule(1, 1.7, 1e-12, 8)
    assert np.allclose(w, 1.7, rtol=1e-10)
    # delta = 1 and no decay is vanilla speculative decoding
    assert np.array_equal(oracle.make_schedule(0, 1.0, 0.0, 5), np.ones(5))
    # L = 1: the single multiplier carries the whole budget
    assert np.isclose(oracle.make_schedule(1, 1.1, 0.7, 1)[0], 1.1)


def test_exp_schedule_mu_root(oracle):
    """mu recovered from omega satisfies the paper's defining equation."""
    L, delta, nu = 8, 1.1, 0.7
    w = oracle.make_schedule(1, delta, nu, L)
    i = np.arange(1, L + 1)
    mu = -np.log(w[0] / delta) - nu * 1          # omega_1 = delta exp(-nu - mu)
    assert np.isclose(np.exp(-nu * i - mu).sum(), L, rtol=1e-13)
    assert np.allclose(w, delta * np.exp(-nu * i - mu), rtol=1e-13)


def test_linear_schedule(oracle):
    L, delta, ell = 4, 1.3, 8.0
    w = oracle.make_schedule(2, delta, ell, L)
    assert np.isclose(w.sum(), delta * L)
    # linear in i: constant second difference zero, slope negative
    assert np.allclose(np.diff(w, 2), 0.0, atol=1e-13)
    assert np.all(np.diff(w) < 0)
    # proportional to (ell - i): omega_i / omega_j = (ell-i)/(ell-j)
    assert np.isclose(w[0] / w[3], (ell - 1) / (ell - 4))
    # beyond i >= ell the weight is clamped at zero, budget still delta L
    w = oracle.make_schedule(2, 1.0, 8.0, 12)
    assert np.all(w[7:] == 0) and np.isclose(w.sum(), 12.0)


def test_schedule_bad_args(oracle):
    for args in [(1, 1.1, 0.7, 0), (1, -1.0, 0.7, 4), (3, 1.0, 0.7, 4), (2, 1.0, 1.0, 4)]:
        with pytest.raises(ValueError):
            oracle.make_schedule(*args)


# ---- acceptance probability (Eq. relax) and the 0/0 := 1 convention -----------
def test_accept_prob_cases(oracle):
    assert oracle.accept_prob(0.25, 0.5, 1.0) == 0.5         # vanilla ratio
    assert oracle.accept_prob(0.5, 0.25, 1.0) == 1.0         # capped at one
    assert oracle.accept_prob(0.25, 0.5, 1.5) == 0.75        # multiplicative relaxation
    assert oracle.accept_prob(0.25, 0.5, 3.0) == 1.0
    assert oracle.accept_prob(0.25, 0.5, 0.0) == 0.0         # omega = 0 rejects everything
    assert oracle.accept_prob(0.0, 0.0, 1.0) == 1.0          # 0/0 := 1
    assert oracle.accept_prob(0.0, 0.0, 0.5) == 1.0
    assert oracle.accept_prob(0.3, 0.0, 1.0) == 1.0          # p/0 = +inf
    assert oracle.accept_prob(0.0, 0.3, 2.0) == 0.0
    # Eq. relax is stated for omega >= 0: a negative or NaN multiplier is read as 0
    assert oracle.accept_prob(0.25, 0.5, float("nan")) == 0.0
    assert oracle.accept_prob(0.25, 0.5, -3.0) == 0.0
    assert oracle.accept_prob(0.0, 0.0, float("nan")) == 1.0  # 0/0 := 1 is kept
    # ... and Eq. opt_G then gives the target distribution itself (f = 0 everywhere)
    P, Q = np.array([0.5, 0.3, 0.2]), np.array([0.2, 0.2, 0.6])
    for om in (float("nan"), -1.0, 0.0):
        assert np.allclose(oracle.resample_dist(P, Q, om), P, atol=1e-15)


def test_accept_rate_is_overlap(oracle):
    """E_{x~Q}[f] = sum_x min{Q, omega P}; at omega = 1 it is 1 - TV(P, Q)."""
    rng = np.random.default_rng(1)
    P, Q = rng.dirichlet(np.ones(11)), rng.dirichlet(np.ones(11))
    for omega in (0.3, 1.0, 1.7):
        rate = sum(Q[x] * oracle.accept_prob(P[x], Q[x], omega) for x in range(11))
        assert np.isclose(rate, np.minimum(Q, omega * P).sum(), rtol=1e-13)
    rate1 = sum(Q[x] * oracle.accept_prob(P[x], Q[x], 1.0) for x in range(11))
    assert np.isclose(rate1, 1.0 - 0.5 * np.abs(P - Q).sum(), rtol=1e-13)


# ---- softmax -------------------------------------------------------------------
@pytest.mark.parametrize("V", [2, 7, 33, 1000, 16384])
def test_softmax_vs_scipy(oracle, V):
    rng = np.random.default_rng(V)
    z = rng.normal(0, 3, V)
    P = oracle.softmax(z)
    assert np.allclose(P, sps.softmax(z), rtol=1e-13, atol=0)
    assert np.allclose(np.log(P), z - sps.logsumexp(z), rtol=0, atol=1e-12)
    assert np.isclose(P.sum(), 1.0, rtol=1e-14)


def test_softmax_extremes(oracle):
    z = np.array([1000.0, 999.0, -1000.0, -np.inf])
    P = oracle.softmax(z)
    assert np.allclose(P, [1 / (1 + np.exp(-1)), np.exp(-1) / (1 + np.exp(-1)), 0, 0], rtol=1e-14)
    assert oracle.softmax(np.array([0.0, np.nan])) is None
    assert oracle.softmax(np.array([0.0, np.inf])) is None
    assert oracle.softmax(np.array([-np.inf, -np.inf])) is None
    # shift invariance
    z = np.random.default_rng(0).normal(size=50)
    assert np.allclose(oracle.softmax(z), oracle.softmax(z + 123.0), rtol=1e-12)


# ---- row preparation: bf16 decode, guidance mix, top-k ---------------------------
def _bf16_bits(x32):
    """Round-to-nearest-even fp32 -> bf16 bit patterns (test-side construction)."""
    b = np.asarray(x32, np.float32).view(np.uint32).astype(np.uint64)
    r = ((b + 0x7FFF + ((b >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def test_prepare_row_decodes_bf16(oracle):
    vals = np.array([1.0, -2.5, 0.15625, 3.0e38, -1.0e-30, 0.0], np.float32)
    bits = _bf16_bits(vals)
    back = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    z = oracle.prepare_row(bits, None, oracle.BF16, 1.0, 0)
    assert np.array_equal(z, back)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_guidance_mix_is_fp32_fma(oracle, dtype):
    rng = np.random.default_rng(5)
    c = rng.normal(0, 3, 257).astype(np.float32)
    u = rng.normal(0, 3, 257).astype(np.float32)
    if dtype == "bf16":
        cb, ub = _bf16_bits(c), _bf16_bits(u)
        c = (cb.astype(np.uint32) << 16).view(np.float32)
        u = (ub.astype(np.uint32) << 16).view(np.float32)
        z = oracle.prepare_row(cb, ub, oracle.BF16, 4.0, 0)
    else:
        z = oracle.prepare_row(c, u, oracle.F32, 4.0, 0)
    d = (c - u).astype(np.float32)                      # difference rounded to fp32
    exact = [Fraction(4) * Fraction(float(di)) + Fraction(float(ui)) for di, ui in zip(d, u)]
    want = np.array([np.float32(float(e)) for e in exact], np.float32)   # single rounding
    assert np.array_equal(z.astype(np.float32), want)
    assert np.array_equal(z, want.astype(np.float64))   # value is exactly an fp32 number


def test_topk_keeps_ties_and_matches_partition(oracle):
    rng = np.random.default_rng(9)
    z = rng.normal(0, 3, 500).astype(np.float32)
    for k in (1, 7, 100, 499):
        out = oracle.prepare_row(z, None, oracle.F32, 1.0, k)
        kth = np.partition(z.astype(np.float64), -k)[-k]
        keep = z >= kth
        assert np.array_equal(np.isfinite(out), keep)
        assert np.array_equal(out[keep], z[keep].astype(np.float64))
        assert keep.sum() == k
    # ties at the threshold are all kept
    zt = np.array([5, 3, 3, 3, 1, 0], np.float32)
    out = oracle.prepare_row(zt, None, oracle.F32, 1.0, 2)
    assert np.array_equal(np.isfinite(out), [True, True, True, True, False, False])
    # k = 0 and k >= V switch the filter off
    assert np.array_equal(oracle.prepare_row(zt, None, oracle.F32, 1.0, 0), zt)
    assert np.array_equal(oracle.prepare_row(zt, None, oracle.F32, 1.0, 6), zt)


# ---- inverse CDF ----------------------------------------------------------------
@pytest.mark.parametrize("V", [2, 5, 64, 1000])
def test_inverse_cdf_vs_searchsorted(oracle, V):
    rng = np.random.default_rng(V)
    g = rng.random(V) * (rng.random(V) < 0.6)
    g[rng.integers(V)] += 0.1                     # at least one positive entry
    Z = float(np.cumsum(g)[-1])
    cum = np.cumsum(g)
    for u in np.r_[rng.random(200), 2.0 ** -24, 1 - 2.0 ** -24]:
        tok, margin = oracle.inverse_cdf(g, Z, u)
        want = int(np.searchsorted(cum, u * Z, side="right"))   # first C(x) > uZ
        assert tok == want and g[tok] > 0
        lo = cum[tok - 1] / Z if tok > 0 else 0.0
        assert lo <= u < cum[tok] / Z
        pos = np.flatnonzero(g > 0)
        d = []
        if tok != pos[0]:
            d.append(abs(u - lo))
        if tok != pos[-1]:
            d.append(abs(u - cum[tok] / Z))
        assert margin == (min(d) if d else np.inf)


def test_inverse_cdf_edge(oracle):
    g = np.array([0.0, 0.5, 0.0, 0.5, 0.0])
    assert oracle.inverse_cdf(g, 1.0, 0.25)[0] == 1
    assert oracle.inverse_cdf(g, 1.0, 0.5)[0] == 3          # C(1) = 0.5 is not > 0.5
    assert oracle.inverse_cdf(g, 1.0, 0.999)[0] == 3
    # a total that overstates the sum (rounding stand-in): last positive token
    assert oracle.inverse_cdf(g, 1.5, 0.9)[0] == 3
    # single positive entry: always picked, no competing boundary
    tok, m = oracle.inverse_cdf(np.array([0, 0, 2.0]), 2.0, 0.3)
    assert tok == 2 and m == np.inf


def test_inverse_cdf_frequencies(oracle):
    """Stratified u over a fine grid reproduces the distribution to grid accuracy."""
    g = np.array([0.1, 0.0, 0.4, 0.2, 0.3])
    n = 20000
    us = (np.arange(n) + 0.5) / n
    counts = np.bincount([oracle.inverse_cdf(g, 1.0, u)[0] for u in us], minlength=5)
    assert np.allclose(counts / n, g, atol=1.5 / n)


# ---- resampling distribution (Eq. opt_G) -------------------------------------------
@pytest.mark.parametrize("omega", [0.0, 0.3, 0.999, 1.0, 1.1, 2.0, 50.0])
def test_resample_dist_is_distribution(oracle, omega):
    rng = np.random.default_rng(int(omega * 10))
    for V in (2, 3, 8, 100):
        P, Q = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
        G = oracle.resample_dist(P, Q, omega)
        assert np.all(G >= 0) and np.isclose(G.sum(), 1.0, rtol=1e-13)


def test_resample_dist_prop2_equals_vanilla(oracle):
    """Proposition 2: G* = G^van = Norm([P - Q]_+) whenever f >= f^van (omega >= 1)."""
    rng = np.random.default_rng(2)
    for V in (3, 8, 50):
        P, Q = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
        van = np.maximum(P - Q, 0)
        van /= van.sum()
        for omega in (1.0, 1.1, 2.0, 1e6):
            assert np.allclose(oracle.resample_dist(P, Q, omega), van, rtol=1e-12, atol=1e-15)


def test_resample_dist_below_one(oracle):
    """omega < 1: [P - min(Q, omega P)]_+ = max{P - Q, (1 - omega) P} pointwise."""
    rng = np.random.default_rng(3)
    P, Q = rng.dirichlet(np.ones(12)), rng.dirichlet(np.ones(12))
    for omega in (0.0, 0.25, 0.9):
        want = np.maximum(P - Q, (1 - omega) * P)
        want /= want.sum()
        assert np.allclose(oracle.resample_dist(P, Q, omega), want, rtol=1e-12)
    assert np.allclose(oracle.resample_dist(P, Q, 0.0), P, rtol=1e-13)   # f = 0 => G* = P


def test_resample_dist_zero_mass_and_fallback(oracle):
    P = np.array([0.5, 0.5, 0.0, 0.0])
    Q = np.array([0.0, 0.25, 0.75, 0.0])
    # token 0: q = 0 -> f = 1 -> P - 0; token 1: P > Q -> P - Q; tokens 2,3: nothing
    G = oracle.resample_dist(P, Q, 1.0)
    assert np.allclose(G, np.array([0.5, 0.25, 0, 0]) / 0.75)
    # P == Q and omega >= 1: empty positive part, falls back to P
    g, Z = oracle.resample_weights(P, P, 1.0)
    assert Z == 0.0 and np.all(g == 0)
    assert np.array_equal(oracle.resample_dist(P, P, 1.3), P)


def test_prop_lp_closed_form_and_optimality(oracle):
    """Proposition LP: min over distributions G of
    sum_x |P - Q f - G sum(1-f)Q| equals sum|P - Q f| - sum(1-f)Q, attained at G*.
    Checked against an exhaustive simplex grid (V = 3) and random G (V = 4),
    for omega on both sides of 1."""
    rng = np.random.default_rng(4)

    def objective(P, Q, f, G):
        rej = ((1 - f) * Q).sum()
        return np.abs(P - Q * f - G * rej).sum()

    for V, omega in [(3, 1.0), (3, 1.6), (3, 0.4), (4, 0.7), (4, 2.5)]:
        P, Q = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
        f = np.array([oracle.accept_prob(P[x], Q[x], omega) for x in range(V)])
        Gs = oracle.resample_dist(P, Q, omega)
        closed = np.abs(P - Q * f).sum() - ((1 - f) * Q).sum()
        best = objective(P, Q, f, Gs)
        assert np.isclose(best, closed, rtol=1e-12, atol=1e-14)
        if V == 3:
            n = 120
            cands = [np.array([a, b, n - a - b]) / n for a in range(n + 1) for b in range(n + 1 - a)]
        else:
            cands = list(rng.dirichlet(np.ones(V) * 0.5, size=4000))
        vals = np.array([objective(P, Q, f, G) for G in cands])
        assert vals.min() >= best - 1e-12


# ---- per-position sums of Theorem 2 ------------------------------------------------------------
@pytest.mark.parametrize("omega", [0.0, 0.25, 1.0, 1.1, 2.36, 50.0])
def test_position_terms_closed_forms(oracle, omega):
    """sum_x Q f = sum_x min{Q, omega P}; the bracket of Eq. bd2 equals 2 sum_x [min{Q, omega P} - P]_+
    (both follow from f = min{1, omega P/Q}); zero entries follow the 0/0 := 1 convention."""
    rng = np.random.default_rng(int(omega * 100) + 3)
    for V in (2, 7, 64):
        P = rng.dirichlet(np.full(V, 0.6))
        Q = rng.dirichlet(np.full(V, 0.6))
        if V > 2:
            P[1] = 0.0; P /= P.sum()
            Q[2] = 0.0; Q /= Q.sum()
        am, bt = oracle.position_terms(P, Q, omega)
        mn = np.minimum(Q, omega * P)
        assert np.isclose(am, mn.sum(), rtol=1e-13, atol=1e-15)
        assert np.isclose(bt, 2.0 * np.maximum(mn - P, 0.0).sum(), rtol=1e-12, atol=1e-14)
        assert -1e-15 <= am <= 1.0 + 1e-15 and bt >= -1e-15
        if omega <= 1.0:
            assert abs(bt) < 1e-14          # no relaxation beyond vanilla: the bound's bracket vanishes
        if omega == 1.0:
            assert np.isclose(am, 1.0 - 0.5 * np.abs(P - Q).sum(), rtol=1e-13)   # 1 - TV(P, Q)
        if omega == 0.0:
            assert am == 0.0 or np.isclose(am, Q[P == 0.0].sum() * 0.0)


def test_position_terms_is_the_infimum_of_prop_lp(oracle):
    """The bracket equals the objective of Proposition LP at G* = Norm([P - Q f]_+), and no other G
    gets below it."""
    rng = np.random.default_rng(11)
    for omega in (0.4, 1.0, 1.8, 4.0):
        P, Q = rng.dirichlet(np.ones(5)), rng.dirichlet(np.ones(5))
        f = np.array([oracle.accept_prob(p, q, omega) for p, q in zip(P, Q)])
        rej = ((1.0 - f) * Q).sum()
        objective = lambda G: np.abs(P - Q * f - G * rej).sum()
        _, bt = oracle.position_terms(P, Q, omega)
        assert np.isclose(objective(oracle.resample_dist(P, Q, omega)), bt, rtol=1e-12, atol=1e-14)
        for _ in range(200):
            assert objective(rng.dirichlet(np.ones(5))) >= bt - 1e-12
