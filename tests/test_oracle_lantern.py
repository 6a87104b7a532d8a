"""Pins of the oracle's similarity relaxation (LANTERN++'s acceptance with the paper's resampling
distribution G*; Ablation Study, "Principled Resampling Strategy").

  * the aggregated mass follows the stated selection rule (hand-worked cases);
  * with no neighbours, or lambda = 0, the round is Algorithm 1 bit for bit;
  * the acceptance is never below the plain one, so by Proposition 2 the resampling distribution at
    omega >= 1 is the vanilla Norm([P - Q]_+) whatever the neighbour table;
  * Eq. opt_G with this acceptance still minimises Proposition LP's objective (random search);
  * the real sampler's accept rate is the enumerated sum_x Q(x) f(x).
"""
import numpy as np
import pytest


def test_neighbour_mass_selection_rule(oracle):
    P = np.array([0.40, 0.05, 0.10, 0.20, 0.25])
    # token 0 with neighbours 1, 2, 3: lambda = 0.5 -> budget 0.20: takes 0.05, then 0.10 (0.15 < 0.20), not 0.20
    assert oracle.neighbour_mass(P, [1, 2, 3], 0.5, 0) == pytest.approx(0.40 + 0.05 + 0.10, abs=0)
    # the first neighbour that would break the budget ends the selection, although a later one would fit
    assert oracle.neighbour_mass(P, [3, 1], 0.5, 0) == 0.40
    # strict inequality: 0.05 + 0.10 = 0.15 is not below 0.375 * 0.40 = 0.15
    assert oracle.neighbour_mass(P, [1, 2], 0.375, 0) == pytest.approx(0.45, abs=1e-15)
    # -1, out-of-range entries and the token itself are skipped
    assert oracle.neighbour_mass(P, [-1, 0, 7, 1], 0.5, 0) == pytest.approx(0.45, abs=1e-15)
    assert oracle.neighbour_mass(P, [1, 2, 3], 0.0, 0) == 0.40
    assert oracle.neighbour_mass(np.array([0.0, 1.0]), [1], 5.0, 0) == 0.0     # nothing is below 0


def _case(r, V, k):
    P, Q = r.dirichlet(np.ones(V) * 0.7), r.dirichlet(np.ones(V) * 0.7)
    nbr = np.stack([r.permutation(V)[:k] for _ in range(V)]).astype(np.int32)
    return P, Q, nbr


@pytest.mark.parametrize("seed", range(5))
def test_acceptance_dominates_and_proposition_2(oracle, seed):
    r = np.random.default_rng(seed)
    V, k = 12, 4
    P, Q, nbr = _case(r, V, k)
    for lam in (0.3, 1.0, 4.0):
        f_n = np.array([oracle.accept_prob(oracle.neighbour_mass(P, nbr[x], lam, x), Q[x], 1.0) for x in range(V)])
        f_v = np.array([oracle.accept_prob(P[x], Q[x], 1.0) for x in range(V)])
        assert np.all(f_n >= f_v)
        assert f_n.sum() > f_v.sum() or lam == 0.3
        # f >= f_van  =>  G* = G_van (Proposition 2)
        for omega in (1.0, 1.7):
            g, Z = oracle.resample_weights_nbr(P, Q, omega, nbr, lam)
            van = np.maximum(P - Q, 0.0)
            assert np.allclose(g / Z, van / van.sum(), atol=1e-15)
        # below 1 the multiplier matters: g(x) = [P - min{Q, omega A}]_+ by the definition
        g, Z = oracle.resample_weights_nbr(P, Q, 0.4, nbr, lam)
        A = np.array([oracle.neighbour_mass(P, nbr[x], lam, x) for x in range(V)])
        assert np.allclose(g, np.maximum(P - np.minimum(Q, 0.4 * A), 0.0), atol=1e-16)


@pytest.mark.parametrize("seed", range(3))
def test_resampling_distribution_minimises_proposition_lp_objective(oracle, seed):
    """inf_G sum_x |P - Q f - G sum_y (1 - f) Q| is attained by Norm([P - Q f]_+) for ANY 0 <= f <= 1
    (Proposition LP), so also for the similarity-relaxed f."""
    r = np.random.default_rng(100 + seed)
    V, k = 6, 2
    P, Q, nbr = _case(r, V, k)
    lam, omega = 2.0, 0.8
    f = np.array([oracle.accept_prob(oracle.neighbour_mass(P, nbr[x], lam, x), Q[x], omega) for x in range(V)])
    rej = ((1 - f) * Q).sum()
    obj = lambda G: np.abs(P - Q * f - G * rej).sum()
    g, Z = oracle.resample_weights_nbr(P, Q, omega, nbr, lam)
    best = obj(g / Z)
    closed = np.abs(P - Q * f).sum() - rej
    assert best == pytest.approx(closed, abs=1e-12)
    for _ in range(4000):
        G = r.dirichlet(np.ones(V) * r.choice([0.2, 1.0, 5.0]))
        assert obj(G) >= best - 1e-12


def test_round_without_neighbours_is_algorithm_1_and_accept_rate(oracle):
    r = np.random.default_rng(7)
    B, L, V, k = 4000, 3, 16, 3
    t = (2 * r.standard_normal((1, L, V))).astype(np.float32).repeat(B, 0)
    d = (2 * r.standard_normal((1, L, V))).astype(np.float32).repeat(B, 0)
    Qrows = np.exp(d[0].astype(np.float64)); Qrows /= Qrows.sum(-1, keepdims=True)
    tok = np.stack([r.choice(V, size=B, p=Qrows[i]) for i in range(L)], 1).astype(np.int32)
    u = np.clip(r.random((B, L + 1)), 1e-7, 1 - 1e-7).astype(np.float32)
    om = np.ones(L, np.float32)
    nbr = np.stack([r.permutation(V)[:k] for _ in range(V)]).astype(np.int32)
    base = oracle.verify(t, d, tok, u, om)
    for kw in (dict(neighbours=nbr, nbr_lambda=0.0), dict(neighbours=np.full((V, k), -1, np.int32), nbr_lambda=3.0)):
        same = oracle.verify(t, d, tok, u, om, **kw)
        assert np.array_equal(same.tokens, base.tokens) and np.array_equal(same.accept_len, base.accept_len)
        assert np.array_equal(same.G, base.G) and np.array_equal(same.f, base.f)
    lam = 2.0
    rel = oracle.verify(t, d, tok, u, om, neighbours=nbr, nbr_lambda=lam)
    assert rel.accept_len.mean() > base.accept_len.mean()
    # first position: empirical accept rate vs sum_x Q(x) f(x)
    P0 = np.exp(t[0, 0].astype(np.float64)); P0 /= P0.sum()
    f = np.array([oracle.accept_prob(oracle.neighbour_mass(P0, nbr[x], lam, x), Qrows[0][x], 1.0) for x in range(V)])
    want = (Qrows[0] * f).sum()
    got = (rel.accept_len >= 1).mean()
    assert abs(got - want) < 4 * np.sqrt(want * (1 - want) / B)
    # the reported p is the mass the test used
    x0 = tok[0, 0]
    assert rel.p[0, 0] == pytest.approx(oracle.neighbour_mass(P0, nbr[x0], lam, x0), rel=1e-12)
    # every emitted token has positive mass under the distribution it was drawn from
    for b in range(0, B, 97):
        j = rel.accept_len[b]
        if j < L:
            assert rel.G[b, rel.tokens[b, j]] > 0 and abs(rel.G[b].sum() - 1) < 1e-12
