"""Pins for the oracle's whole procedure against what the paper proves.

A tiny "model" is a pair of conditional tables P(.|prefix), Q(.|prefix) over an
alphabet of V symbols for every prefix shorter than L+1.  From Algorithm 1's
description the law P_hat of the (virtually extended) output over X^{L+1} can be
enumerated exactly, using only the oracle's acceptance probability and
resampling distribution.  That law must
  * equal P for the vanilla choice (Theorem 1),
  * agree with the paper's closed form (Eq. joint),
  * have TV(P_hat, P) below the bound of Theorem 2 (Eq. tv_token), which at G*
    takes the value of Eq. bd2 and is zero for the vanilla choice,
  * give E[tau + 1] of Eq. token_exp,
and the oracle's real sampler (orc_verify, driven by supplied uniforms) must
reproduce P_hat empirically (chi-square over >= 10^6 rounds at V = 8).
"""
import itertools

import numpy as np
import pytest
import scipy.stats as st


# ----------------------------------------------------------------------------------
class TinyModel:
    def __init__(self, V, L, rng, conc=1.0, share=0.0):
        self.V, self.L = V, L
        self.P, self.Q = {}, {}
        for n in range(L + 1):
            for pre in itertools.product(range(V), repeat=n):
                p = rng.dirichlet(np.ones(V) * conc)
                q = rng.dirichlet(np.ones(V) * conc)
                self.P[pre] = p
                self.Q[pre] = share * p + (1 - share) * q

    def joint_P(self):
        V, L = self.V, self.L
        out = np.zeros((V,) * (L + 1))
        for xs in itertools.product(range(V), repeat=L + 1):
            pr = 1.0
            for i in range(L + 1):
                pr *= self.P[xs[:i]][xs[i]]
            out[xs] = pr
        return out


def f_table(oracle, model, omegas):
    """f_i(x_{1:i}) for every prefix (Eq. relax), from the oracle."""
    f = {}
    for n in range(1, model.L + 1):
        for xs in itertools.product(range(model.V), repeat=n):
            pre = xs[:-1]
            f[xs] = oracle.accept_prob(model.P[pre][xs[-1]], model.Q[pre][xs[-1]], omegas[n - 1])
    return f


def g_table(oracle, model, omegas, kind="star"):
    G = {}
    rng = np.random.default_rng(99)
    for n in range(model.L):
        for pre in itertools.product(range(model.V), repeat=n):
            if kind == "star":
                G[pre] = oracle.resample_dist(model.P[pre], model.Q[pre], omegas[n])
            elif kind == "random":
                G[pre] = rng.dirichlet(np.ones(model.V))
    return G


def enumerate_output_law(model, f, G):
    """P_hat over X^{L+1} straight from Algorithm 1 plus the virtual extension."""
    V, L = model.V, model.L
    out = np.zeros((V,) * (L + 1))

    def extend(prefix, weight):
        """append target samples until length L+1"""
        if len(prefix) == L + 1:
            out[prefix] += weight
            return
        for x in range(V):
            extend(prefix + (x,), weight * model.P[prefix][x])

    for draft in itertools.product(range(V), repeat=L):
        wq = 1.0
        for i in range(L):
            wq *= model.Q[draft[:i]][draft[i]]
        acc = 1.0   # probability that positions 1..j were all accepted
        for j in range(L):
            fj = f[draft[:j + 1]]
            rej = acc * (1.0 - fj)
            if rej > 0:
                for x in range(V):
                    extend(draft[:j] + (x,), wq * rej * G[draft[:j]][x])
            acc *= fj
        extend(draft, wq * acc)     # all accepted, bonus token from P
    return out


def closed_form_law(model, f, G):
    """Eq. joint at i = L, times P(x_{L+1} | x_{1:L}) (Eq. condp)."""
    V, L = model.V, model.L

    def Qseq(xs):
        pr = 1.0
        for i in range(len(xs)):
            pr *= model.Q[xs[:i]][xs[i]]
        return pr

    def Pcont(xs, start):
        """P(x_{start+1:len} | x_{1:start})"""
        pr = 1.0
        for i in range(start, len(xs)):
            pr *= model.P[xs[:i]][xs[i]]
        return pr

    out = np.zeros((V,) * (L + 1))
    for xs in itertools.product(range(V), repeat=L):
        val = Qseq(xs) * np.prod([f[xs[:k]] for k in range(1, L + 1)])
        for j in range(L):
            p_bar = Qseq(xs[:j]) * G[xs[:j]][xs[j]] * Pcont(xs, j + 1)
            r_bar = sum(model.Q[xs[:j]][t] * (1 - f[xs[:j] + (t,)]) for t in range(V))
            r_bar *= np.prod([f[xs[:k]] for k in range(1, j + 1)])
            val += p_bar * r_bar
        for x in range(V):
            out[xs + (x,)] = val * model.P[xs][x]
    return out


def tv_bound(model, f, G):
    """Right-hand side of Eq. tv_token."""
    V, L = model.V, model.L
    total = 0.0
    for i in range(L):
        for pre in itertools.product(range(V), repeat=i):
            w = 1.0
            for k in range(i):
                w *= model.Q[pre[:k]][pre[k]] * f[pre[:k + 1]]
            rej = sum((1 - f[pre + (t,)]) * model.Q[pre][t] for t in range(V))
            for x in range(V):
                total += w * abs(model.Q[pre][x] * f[pre + (x,)] - model.P[pre][x] + G[pre][x] * rej)
    return 0.5 * total


def tv_bound_at_gstar(model, f):
    """Eq. bd2."""
    V, L = model.V, model.L
    total = 0.0
    for i in range(L):
        for pre in itertools.product(range(V), repeat=i):
            w = 1.0
            for k in range(i):
                w *= model.Q[pre[:k]][pre[k]] * f[pre[:k + 1]]
            a = sum(abs(model.P[pre][x] - model.Q[pre][x] * f[pre + (x,)]) for x in range(V))
            b = sum((1 - f[pre + (x,)]) * model.Q[pre][x] for x in range(V))
            total += w * (a - b)
    return 0.5 * total


def bound_and_length_through_position_terms(oracle, model, f, omegas):
    """Eq. bd2 and Eq. token_exp assembled from the oracle's per-position sums: every prefix
    x_{1:i} contributes, with weight Q(x_{1:i}) prod f, its bracket / its acceptance mass."""
    V, L = model.V, model.L
    bound, e_len = 0.0, 1.0
    for i in range(L):
        for pre in itertools.product(range(V), repeat=i):
            w = 1.0
            for k in range(i):
                w *= model.Q[pre[:k]][pre[k]] * f[pre[:k + 1]]
            am, bt = oracle.position_terms(model.P[pre], model.Q[pre], omegas[i])
            bound += w * bt
            e_len += w * am
    return 0.5 * bound, e_len


def expected_len_formula(model, f):
    """Eq. token_exp."""
    V, L = model.V, model.L
    tot = 1.0
    for i in range(1, L + 1):
        for xs in itertools.product(range(V), repeat=i):
            w = 1.0
            for k in range(i):
                w *= model.Q[xs[:k]][xs[k]] * f[xs[:k + 1]]
            tot += w
    return tot


# ----------------------------------------------------------------------------------
@pytest.mark.parametrize("V,L", [(2, 1), (2, 3), (3, 2), (4, 2), (5, 1), (8, 1), (8, 2)])
def test_theorem1_vanilla_is_exact(oracle, V, L):
    model = TinyModel(V, L, np.random.default_rng(V * 10 + L))
    om = np.ones(L)
    f, G = f_table(oracle, model, om), g_table(oracle, model, om)
    phat = enumerate_output_law(model, f, G)
    assert np.isclose(phat.sum(), 1.0, rtol=1e-12)
    assert np.abs(phat - model.joint_P()).max() < 1e-12
    assert tv_bound(model, f, G) < 1e-12            # bound collapses to zero (vanilla)
    assert abs(tv_bound_at_gstar(model, f)) < 1e-12


@pytest.mark.parametrize("V,L,omegas", [
    (3, 2, (1.6, 0.8)), (3, 3, (2.36, 1.17, 0.58)), (4, 2, (0.5, 0.2)), (2, 3, (3.0, 3.0, 3.0)),
    (5, 2, (1.1, 1.1)), (3, 2, (0.0, 0.0))])
@pytest.mark.parametrize("gkind", ["star", "random"])
def test_theorem2_law_bound_and_length(oracle, V, L, omegas, gkind):
    model = TinyModel(V, L, np.random.default_rng(7 + V + L), conc=0.8)
    f, G = f_table(oracle, model, omegas), g_table(oracle, model, omegas, gkind)
    phat = enumerate_output_law(model, f, G)
    assert np.isclose(phat.sum(), 1.0, rtol=1e-12)
    # the paper's closed form of the same law
    assert np.abs(phat - closed_form_law(model, f, G)).max() < 1e-12
    tv = 0.5 * np.abs(phat - model.joint_P()).sum()
    bound = tv_bound(model, f, G)
    assert tv <= bound + 1e-12
    if gkind == "star":
        assert np.isclose(bound, tv_bound_at_gstar(model, f), rtol=1e-10, atol=1e-13)
    else:   # no G does better than G* on the bound
        assert bound >= tv_bound_at_gstar(model, f) - 1e-12
    # expected emitted length: enumerate tau's law directly
    e_len = 1.0
    for i in range(1, L + 1):
        for xs in itertools.product(range(V), repeat=i):
            w = 1.0
            for k in range(i):
                w *= model.Q[xs[:k]][xs[k]] * f[xs[:k + 1]]
            e_len += w
    assert np.isclose(e_len, expected_len_formula(model, f))
    # the per-position sums (what the library can report per drafted prefix) give the same two numbers
    b_terms, len_terms = bound_and_length_through_position_terms(oracle, model, f, omegas)
    assert np.isclose(b_terms, tv_bound_at_gstar(model, f), rtol=1e-10, atol=1e-13)
    assert np.isclose(len_terms, e_len, rtol=1e-12)
    if all(o == 0.0 for o in omegas):
        # omega = 0: everything is rejected, G* = P, the output is a pure target sample
        assert np.abs(phat - model.joint_P()).max() < 1e-12 or gkind == "random"
        assert np.isclose(e_len, 1.0)


def test_relaxation_increases_length_and_annealing_budget(oracle):
    """omega > 1 accepts more than vanilla; omega < 1 accepts less (Eq. token_exp)."""
    model = TinyModel(4, 2, np.random.default_rng(0))
    lens = [expected_len_formula(model, f_table(oracle, model, (w, w))) for w in (0.5, 1.0, 1.5, 3.0)]
    assert lens == sorted(lens) and lens[0] < lens[1] < lens[2]


# ---- the real sampler -----------------------------------------------------------------
def _run_sampler(oracle, model, omegas, n, seed, bonus=True):
    """Drive orc_verify as a decoder would: draft with Q, hand it the rows that
    belong to the drafted prefix, then extend virtually with P."""
    V, L = model.V, model.L
    rng = np.random.default_rng(seed)
    drafts = np.zeros((n, L), np.int64)
    T = L + 1 if bonus else L
    tl = np.zeros((n, T, V))
    dl = np.zeros((n, L, V))
    # group trials by drafted prefix so table lookups stay vectorised
    for i in range(L + 1):
        keys = [tuple(r) for r in drafts[:, :i]] if i else [()] * n
        uniq = set(keys)
        keys_arr = np.array([hash(k) for k in keys])
        for pre in uniq:
            sel = np.flatnonzero(keys_arr == hash(pre))
            if i < T:
                with np.errstate(divide="ignore"):
                    tl[sel, i, :] = np.log(model.P[pre])
            if i < L:
                with np.errstate(divide="ignore"):
                    dl[sel, i, :] = np.log(model.Q[pre])
                drafts[sel, i] = rng.choice(V, size=sel.size, p=model.Q[pre])
    uni = (rng.integers(0, 2 ** 23, size=(n, L + 1)) * 2 + 1).astype(np.float64) * 2.0 ** -24
    res = oracle.verify(tl, dl, drafts.astype(np.int32), uni.astype(np.float32),
                        np.asarray(omegas, np.float32), dtype=oracle.F64, want_G=False,
                        want_pqf=False)
    return res, drafts, rng


def _extend(model, res, rng, n):
    V, L = model.V, model.L
    full = np.array(res.tokens[:, :L + 1], dtype=np.int64)
    for i in range(L + 1):
        need = np.flatnonzero(full[:, i] < 0)
        if need.size == 0:
            continue
        keys = [tuple(r) for r in full[need, :i]]
        for pre in set(keys):
            sel = need[[k == pre for k in keys]]
            full[sel, i] = rng.choice(V, size=sel.size, p=model.P[pre])
    return full


@pytest.mark.parametrize("omegas", [(1.0, 1.0), (2.2, 0.6)])
def test_sampler_chi_square_v8(oracle, omegas):
    """>= 10^6 rounds at V = 8, L = 2: the sampler's output law is the enumerated
    one, which for omega = 1 is the target itself (Theorem 1)."""
    V, L, n = 8, 2, 1_200_000
    model = TinyModel(V, L, np.random.default_rng(11), conc=4.0, share=0.5)
    f, G = f_table(oracle, model, omegas), g_table(oracle, model, omegas)
    phat = enumerate_output_law(model, f, G)
    if omegas == (1.0, 1.0):
        assert np.abs(phat - model.joint_P()).max() < 1e-12
    res, drafts, rng = _run_sampler(oracle, model, omegas, n, seed=5)
    # structure of the output: accepted prefix equals the draft, then one new token, then -1
    tau = res.accept_len
    assert tau.min() >= 0 and tau.max() <= L
    for i in range(L):
        acc = tau > i
        assert np.array_equal(res.tokens[acc, i], drafts[acc, i].astype(np.int32))
    assert np.all(res.tokens[np.arange(n), tau] >= 0)
    for i in range(1, L + 1):
        assert np.all(res.tokens[tau < i, i] == -1)
    full = _extend(model, res, rng, n)
    idx = np.ravel_multi_index(tuple(full.T), (V,) * (L + 1))
    counts = np.bincount(idx, minlength=V ** (L + 1)).astype(np.float64)
    expected = phat.ravel() * n
    assert expected.min() > 20      # chi-square validity
    chi2, pval = st.chisquare(counts, expected)
    assert pval > 1e-4, (chi2, pval)
    # mean emitted length against Eq. token_exp
    want = expected_len_formula(model, f)
    se = (tau + 1).std() / np.sqrt(n)
    assert abs((tau + 1).mean() - want) < 5 * se
    # and the law is NOT the target when relaxed (the test can tell the difference)
    if omegas != (1.0, 1.0):
        _, p_wrong = st.chisquare(counts, model.joint_P().ravel() * n)
        assert p_wrong < 1e-6


def test_sampler_omega_zero_is_target_sample(oracle):
    V, L, n = 8, 2, 300_000
    model = TinyModel(V, L, np.random.default_rng(21), conc=2.0)
    res, _, _ = _run_sampler(oracle, model, (0.0, 0.0), n, seed=8)
    assert np.all(res.accept_len == 0)
    counts = np.bincount(res.tokens[:, 0], minlength=V).astype(np.float64)
    _, pval = st.chisquare(counts, model.P[()] * n)
    assert pval > 1e-4


def test_sampler_without_bonus_row(oracle):
    V, L, n = 4, 2, 20000
    model = TinyModel(V, L, np.random.default_rng(3), conc=2.0, share=0.8)
    res, drafts, _ = _run_sampler(oracle, model, (1.2, 1.2), n, seed=2, bonus=False)
    full = res.accept_len == L
    assert full.any() and (~full).any()
    assert np.all(res.tokens[full, L] == -1)
    assert np.array_equal(res.tokens[full, :L], drafts[full].astype(np.int32))


def test_planted_mistakes_are_caught(oracle):
    """The enumeration can tell right from wrong: a resampling distribution with a
    dropped positive part, or a swapped P/Q ratio, breaks Theorem 1."""
    model = TinyModel(3, 2, np.random.default_rng(5))
    om = np.ones(2)
    f, G = f_table(oracle, model, om), g_table(oracle, model, om)
    bad_G = {k: oracle.resample_dist(model.Q[k], model.P[k], 1.0) for k in G}   # transposed
    assert np.abs(enumerate_output_law(model, f, bad_G) - model.joint_P()).max() > 1e-3
    bad_f = {xs: oracle.accept_prob(model.Q[xs[:-1]][xs[-1]], model.P[xs[:-1]][xs[-1]], 1.0)
             for xs in f}
    assert np.abs(enumerate_output_law(model, bad_f, G) - model.joint_P()).max() > 1e-3
