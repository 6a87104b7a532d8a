"""Pins of the extended-precision statement of Eq. opt_G and the inverse-CDF draw (oracle/exact.py),
and through it of the fp64 oracle's resolution: where the fp64 oracle has the digits the two agree,
and where both models put all but 1e-16 of their mass on one token the fp64 oracle is shown to lose
the largest weight while the extended-precision statement keeps it."""
from decimal import Decimal, localcontext
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import exact


def _frac_to_dec(fr: Fraction, prec=exact.PREC) -> Decimal:
    with localcontext() as ctx:
        ctx.prec = prec
        return Decimal(fr.numerator) / Decimal(fr.denominator)


def _ln(fr: Fraction, prec=exact.PREC) -> Decimal:
    with localcontext() as ctx:
        ctx.prec = prec
        return _frac_to_dec(fr, prec).ln()


def _exact_fraction_case(P, Q, omega):
    """Eq. relax and Eq. opt_G in rational arithmetic, written from the equations."""
    g = []
    for p, q in zip(P, Q):
        if q == 0:
            f = Fraction(1)
        elif p == 0:
            f = Fraction(0)
        else:
            f = min(Fraction(1), omega * p / q)
        g.append(max(Fraction(0), p - q * f))
    return g, sum(g)


RATIONAL_CASES = [
    ([Fraction(1, 2), Fraction(1, 4), Fraction(1, 8), Fraction(1, 16), Fraction(1, 16)],
     [Fraction(1, 5), Fraction(2, 5), Fraction(1, 10), Fraction(1, 5), Fraction(1, 10)]),
    ([Fraction(3, 7), Fraction(2, 7), Fraction(1, 7), Fraction(1, 7)],
     [Fraction(1, 3), Fraction(1, 3), Fraction(1, 6), Fraction(1, 6)]),
    ([Fraction(999999, 1000000), Fraction(1, 3000000), Fraction(2, 3000000)],
     [Fraction(999998, 1000000), Fraction(1, 1000000), Fraction(1, 1000000)]),
]


@pytest.mark.parametrize("P,Q", RATIONAL_CASES)
@pytest.mark.parametrize("omega", [Fraction(0), Fraction(3, 10), Fraction(1), Fraction(11, 10), Fraction(5, 2)])
def test_rational_distributions_against_fraction_arithmetic(P, Q, omega):
    """Logits are the logarithms of rational probabilities, so the softmax must give those rationals
    back and Eq. opt_G must match rational arithmetic to the working precision."""
    with localcontext() as ctx:
        ctx.prec = exact.PREC
        zt = [_ln(p) + Decimal(7) for p in P]       # a common shift does not change the softmax
        zd = [_ln(q) - Decimal(3) for q in Q]
    Pd, Qd = exact.softmax(zt), exact.softmax(zd)
    tol = Decimal(10) ** -(exact.PREC - 8)
    for got, want in zip(Pd, P):
        assert abs(got - _frac_to_dec(want)) < tol
    for got, want in zip(Qd, Q):
        assert abs(got - _frac_to_dec(want)) < tol
    g, Z = exact.resample_weights(Pd, Qd, _frac_to_dec(omega))
    g_fr, Z_fr = _exact_fraction_case(P, Q, omega)
    for got, want in zip(g, g_fr):
        assert abs(got - _frac_to_dec(want)) < tol
    assert abs(Z - _frac_to_dec(Z_fr)) < tol
    if Z_fr > 0:
        # the draw: every uniform on a grid must land on the token rational arithmetic gives
        cum = np.cumsum([float(x / Z_fr) for x in g_fr])
        for u in [0.0009765625 * k + 0.00048828125 for k in range(0, 1024, 37)]:
            c, want_tok = Fraction(0), None
            for x, w in enumerate(g_fr):
                c += w
                if want_tok is None and c > Fraction(u) * Z_fr:
                    want_tok = x
            tok, margin = exact.inverse_cdf(g, Z, u)
            if margin > tol:
                assert tok == want_tok, (u, tok, want_tok, cum)


def test_inverse_cdf_conventions():
    g = [Decimal(0), Decimal("0.25"), Decimal(0), Decimal("0.5"), Decimal("0.25"), Decimal(0)]
    Z = Decimal(1)
    assert exact.inverse_cdf(g, Z, 0.1)[0] == 1
    assert exact.inverse_cdf(g, Z, 0.25)[0] == 3          # strict: C(1) = 0.25 is not > 0.25
    assert exact.inverse_cdf(g, Z, 0.74)[0] == 3
    assert exact.inverse_cdf(g, Z, 0.75)[0] == 4
    assert exact.inverse_cdf(g, Z, 1.0)[0] == 4           # no crossing: the last token with weight
    assert exact.inverse_cdf(g, Z, float("nan"))[0] == 4
    assert exact.inverse_cdf(g, Z, 0.0)[0] == 1           # zero-weight tokens are never drawn
    tok, margin = exact.inverse_cdf(g, Z, 0.3)
    assert tok == 3 and abs(margin - Decimal("0.05")) < Decimal("1e-15")
    # the same conventions as the fp64 oracle's
    gf = np.array([float(x) for x in g])
    for u in (0.1, 0.25, 0.74, 0.75, 1.0, 0.0, 0.3):
        assert oracle.inverse_cdf(gf, 1.0, u)[0] == exact.inverse_cdf(g, Z, u)[0]


@pytest.mark.parametrize("seed", range(6))
def test_agrees_with_fp64_oracle_where_that_has_the_digits(seed):
    r = np.random.default_rng(seed)
    V = 257
    zt = (3.0 * r.standard_normal(V)).astype(np.float32).astype(np.float64)
    zd = (0.9 * zt + 1.3 * r.standard_normal(V)).astype(np.float32).astype(np.float64)
    if seed % 2:
        zt[r.integers(V, size=40)] = -np.inf       # masked entries (a top-k filter leaves such rows)
        zd[r.integers(V, size=40)] = -np.inf
    P64, Q64 = oracle.softmax(zt), oracle.softmax(zd)
    for omega in (0.0, 0.4, 1.0, 1.1, 3.0):
        g64, Z64 = oracle.resample_weights(P64, Q64, omega)
        Pd, Qd = exact.softmax(zt), exact.softmax(zd)
        g, Z = exact.resample_weights(Pd, Qd, omega)
        assert abs(float(Z) - Z64) < 1e-13
        assert np.abs(np.array([float(x) for x in g]) - g64).max() < 1e-14
        for u in (0.001, 0.37, 0.5, 0.93, 0.9999):
            tok64, m64 = oracle.inverse_cdf(g64, Z64, u)
            res = exact.draw(zt, zd, omega, u)
            if m64 > 1e-9 and float(res["margin"]) > 1e-9:
                assert res["token"] == tok64


def test_fp64_oracle_loses_the_top_weight_when_both_models_peak_and_the_exact_statement_keeps_it():
    """Both models put all but exp(-gap) of their mass on token 0.  Summing P(x) - Q(x) over x gives 0,
    so the weight at token 0 equals the mass the drafter has elsewhere in excess of the target's: a
    closed form.  The fp64 oracle, which forms P(0) - Q(0) from two numbers next to 1, keeps it while the
    tails exceed its rounding (gap 20) and loses it beyond (gap 45); the extended-precision statement
    follows the closed form throughout."""
    tail_t = np.array([0.0, -0.5, -1.5, -0.25])      # target logits of the other tokens, before the gap
    tail_d = np.array([1.0, 0.5, -0.5, 0.75])        # drafter's: more mass on every one of them
    for gap, oracle_keeps in ((20.0, True), (45.0, False), (60.0, False)):
        zt = np.concatenate([[gap], tail_t])
        zd = np.concatenate([[gap], tail_d])
        # closed form in extended precision: with omega = 1, g(0) = P(0) - Q(0) = sum_{x>0} (Q(x) - P(x))
        with localcontext() as ctx:
            ctx.prec = exact.PREC
            et = [Decimal(float(v) - gap).exp() for v in tail_t]
            ed = [Decimal(float(v) - gap).exp() for v in tail_d]
            St, Sd = 1 + sum(et), 1 + sum(ed)
            want_g0 = sum(d / Sd - t / St for t, d in zip(et, ed))
        res = exact.draw(zt, zd, 1.0, 0.5)
        g = res["weights"]
        assert want_g0 > 0 and abs(g[0] - want_g0) < want_g0 * Decimal("1e-40")   # (80 digits, weights down to 1e-26)
        assert all(w == 0 for w in g[1:])             # P(x) < Q(x) on every other token
        assert res["token"] == 0 and not res["fallback"]
        P64, Q64 = oracle.softmax(zt), oracle.softmax(zd)
        g64, Z64 = oracle.resample_weights(P64, Q64, 1.0)
        if oracle_keeps:
            assert abs(g64[0] - float(want_g0)) < 1e-3 * float(want_g0)
        else:
            assert g64[0] == 0.0 and Z64 == 0.0       # the difference of two values next to 1 is gone


def test_draw_conventions_for_unusable_rows_and_fallback():
    z = np.array([0.0, 1.0, 2.0])
    assert exact.draw(np.array([0.0, np.nan, 1.0]), z, 1.0, 0.5)["token"] == -1
    assert exact.draw(np.array([-np.inf] * 3), z, 1.0, 0.5)["token"] == -1
    same = exact.draw(z, z, 1.0, 0.5)                 # P == Q, omega >= 1: empty positive part -> P
    assert same["fallback"] and same["token"] == oracle.inverse_cdf(oracle.softmax(z), 1.0, 0.5)[0]
    bonus = exact.draw(z, None, 1.0, 0.2)
    assert not bonus["fallback"] and bonus["token"] == oracle.inverse_cdf(oracle.softmax(z), 1.0, 0.2)[0]
    nan_omega = exact.draw(z, z[::-1].copy(), float("nan"), 0.9)   # f = 0 everywhere: the target distribution
    assert nan_omega["token"] == oracle.inverse_cdf(oracle.softmax(z), 1.0, 0.9)[0]
