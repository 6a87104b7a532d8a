"""Extended-precision statement of Eq. opt_G and of the inverse-CDF draw -- TEST INFRASTRUCTURE.

The fp64 oracle (``csd_oracle.c``) forms Eq. opt_G as the paper writes it, from probabilities that
each carry an absolute rounding of about 1e-16.  Where both models put all but 1e-16 or less of
their mass on one token, the weight ``P(x) - Q(x) f(x)`` at that token -- a difference of two values
next to 1 -- is lost in fp64 although it can be the largest weight of all.  This module writes the
same definitions out in decimal arithmetic of ``PREC`` significant digits (Python's ``decimal``:
``exp`` is correctly rounded at the context's precision), so that such draws can be adjudicated:

  softmax            P(x) = exp(z_x - m) / sum_y exp(z_y - m)       (Algorithm 1, "calculate P ...")
  accept_prob        f = min{1, omega p / q}, 0/0 := 1              (Eq. relax; Notations)
  resample_weights   g(x) = [P(x) - Q(x) f(x)]_+ , Z = sum_x g(x)   (Eq. opt_G, Theorem 2)
  inverse_cdf        smallest x with C(x) > u Z, else the last x with g(x) > 0
  draw               the four in sequence for one position

Inputs are the prepared logits of a row (after the guidance mix and the top-k mask, e.g. from
``oracle.prepare_row``): finite floats or ``-inf``; a float converts to ``Decimal`` exactly.  Nothing
here is shared with, or imported by, the CUDA library.  Pins: ``tests/test_oracle_exact.py`` (rational
distributions evaluated with ``fractions.Fraction``, agreement with the fp64 oracle where that one has
the digits, and the regime where it has not).
"""
from __future__ import annotations

from decimal import Decimal, localcontext
from typing import Iterable, List, Optional, Sequence, Tuple

PREC = 80
_NEG_INF = Decimal("-Infinity")


def _dec(x) -> Decimal:
    return x if isinstance(x, Decimal) else Decimal(float(x))


def softmax(z: Iterable, prec: int = PREC) -> Optional[List[Decimal]]:
    """Softmax of prepared logits; ``None`` for an unusable row (NaN, +inf, or no finite entry)."""
    zs = [_dec(v) for v in z]
    if any(v.is_nan() or v == Decimal("Infinity") for v in zs):
        return None
    finite = [v for v in zs if v != _NEG_INF]
    if not finite:
        return None
    with localcontext() as ctx:
        ctx.prec = prec
        m = max(finite)
        e = [Decimal(0) if v == _NEG_INF else (v - m).exp() for v in zs]
        S = sum(e, Decimal(0))
        return [v / S for v in e]


def accept_prob(p: Decimal, q: Decimal, omega, prec: int = PREC) -> Decimal:
    """Eq. relax at one token; a negative or NaN multiplier counts as 0."""
    om = _dec(omega)
    if om.is_nan() or om < 0:
        om = Decimal(0)
    with localcontext() as ctx:
        ctx.prec = prec
        if q == 0:
            return Decimal(1)      # p/q = +inf for p > 0, and 0/0 := 1
        if p == 0:
            return Decimal(0)
        r = om * p / q
        return r if r < 1 else Decimal(1)


def resample_weights(P: Sequence[Decimal], Q: Sequence[Decimal], omega, prec: int = PREC) -> Tuple[List[Decimal], Decimal]:
    """Unnormalised Eq. opt_G, g(x) = [P(x) - Q(x) f(x)]_+ with f from Eq. relax at candidate x, and Z."""
    with localcontext() as ctx:
        ctx.prec = prec
        g = []
        for p, q in zip(P, Q):
            v = p - q * accept_prob(p, q, omega, prec)
            g.append(v if v > 0 else Decimal(0))
        return g, sum(g, Decimal(0))


def inverse_cdf(g: Sequence[Decimal], Z: Decimal, u, prec: int = PREC) -> Tuple[int, Decimal]:
    """Token = smallest x with C(x) > u Z in token-id order, else the last x with g(x) > 0; and the
    distance, in probability units, from u to the nearest boundary of the picked token's CDF interval
    that separates it from another token of positive weight (0 when rounding alone decided)."""
    with localcontext() as ctx:
        ctx.prec = prec
        ud = _dec(u)
        target = ud * Z
        c = Decimal(0)
        tok, c_lo, c_hi = -1, Decimal(0), Decimal(0)
        first_pos = last_pos = -1
        for x, w in enumerate(g):
            c_prev = c
            c = c + w
            if w > 0:
                last_pos = x
                if first_pos < 0:
                    first_pos = x
            if tok < 0 and not ud.is_nan() and c > target:
                tok, c_lo, c_hi = x, c_prev, c
        if tok < 0:
            return last_pos, Decimal(0)
        margin = Decimal("Infinity")
        if tok != first_pos:
            margin = abs(ud - c_lo / Z)
        if tok != last_pos:
            margin = min(margin, abs(ud - c_hi / Z))
        return tok, margin


def draw(z_target: Iterable, z_draft: Optional[Iterable], omega, u, prec: int = PREC) -> dict:
    """One draw at a rejected position (``z_draft`` given: from Eq. opt_G, falling back to the target
    distribution when its positive part is empty) or the bonus draw (``z_draft`` None: from P).
    Returns token (-1 if the target row is unusable), Z, margin, and whether the fallback was taken."""
    P = softmax(z_target, prec)
    if P is None:
        return dict(token=-1, Z=Decimal(0), margin=Decimal(0), fallback=False, weights=None)
    Q = softmax(z_draft, prec) if z_draft is not None else None
    fallback = False
    if Q is not None:
        g, Z = resample_weights(P, Q, omega, prec)
        if not Z > 0:
            fallback = True
            g, Z = list(P), sum(P, Decimal(0))
    else:
        g, Z = list(P), sum(P, Decimal(0))   # bonus draw, or an unusable drafter row: f = 0 everywhere
    tok, margin = inverse_cdf(g, Z, u, prec)
    return dict(token=tok, Z=Z, margin=margin, fallback=fallback, weights=g)
