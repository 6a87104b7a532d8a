"""Pins of the oracle's tree-structured verification (orc_verify_tree).

The paper's experiments draft a static tree; the rule for several candidates of one node under the
relaxed test is the build's reading (stated in csd_oracle.c).  It is pinned here by what must hold
whatever the reading:
  * a chain-shaped tree IS Algorithm 1: identical to orc_verify bit for bit;
  * with omega == 1 the output law equals the target's (Theorem 1), by exact enumeration of the rule
    on tiny conditional tables, and empirically through the real sampler (chi-square);
  * with a relaxed schedule the real sampler follows the enumerated law of the rule (chi-square),
    and accepts more than the lossless one;
  * bad data (NaN rows, tokens out of range) is reported, not trapped.
"""
import itertools

import numpy as np
import pytest
import scipy.stats as st

# a small static tree: two candidates at the root, two below the first, one below the second,
# and a third level below the very first path
PARENT = np.array([-1, -1, 0, 0, 1, 2], dtype=np.int32)


def children_of(parent, ctx_node):
    return [n for n, p in enumerate(parent) if p == ctx_node]


class Tables:
    """P(.|prefix), Q(.|prefix) for every prefix up to the tree's depth."""
    def __init__(self, V, D, rng, share=0.3):
        self.V, self.D = V, D
        self.P, self.Q = {}, {}
        for n in range(D + 1):
            for pre in itertools.product(range(V), repeat=n):
                p, q = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
                self.P[pre] = p
                self.Q[pre] = share * p + (1 - share) * q


def emitted_law(oracle, tab, parent, omegas):
    """Exact law of the emitted block (variable length) under the rule: candidates i.i.d. from Q in
    their parent's context, tried in order, the residual updated by Eq. opt_G after every rejection."""
    law = {}

    def emit(seq, w):
        law[seq] = law.get(seq, 0.0) + w

    def walk(prefix, ctx_node, level, w):
        kids = children_of(parent, ctx_node)
        if not kids:
            for x in range(tab.V):
                emit(prefix + (x,), w * tab.P[prefix][x])
            return
        R, Q, om = tab.P[prefix].copy(), tab.Q[prefix], omegas[level]
        for n in kids:
            rej = 0.0
            for x in range(tab.V):
                f = oracle.accept_prob(R[x], Q[x], om)
                if Q[x] * f > 0:
                    walk(prefix + (x,), n, level + 1, w * Q[x] * f)
                rej += Q[x] * (1.0 - f)
            w *= rej
            R = oracle.resample_dist(R, Q, om)
        for x in range(tab.V):
            emit(prefix + (x,), w * R[x])

    walk((), -1, 0, 1.0)
    return law


def extended_law(tab, law, length):
    """The emitted block padded with target samples to a fixed length (the virtual extension)."""
    out = np.zeros((tab.V,) * length)

    def extend(seq, w):
        if len(seq) == length:
            out[seq] += w
            return
        for x in range(tab.V):
            extend(seq + (x,), w * tab.P[seq][x])

    for seq, w in law.items():
        extend(seq, w)
    return out


def target_joint(tab, length):
    out = np.zeros((tab.V,) * length)
    for xs in itertools.product(range(tab.V), repeat=length):
        pr = 1.0
        for i in range(length):
            pr *= tab.P[xs[:i]][xs[i]]
        out[xs] = pr
    return out


@pytest.mark.parametrize("seed,V", [(0, 2), (1, 3), (2, 4)])
def test_rule_is_lossless_at_omega_one_by_exact_enumeration(oracle, seed, V):
    D = oracle.tree_depth(PARENT)
    tab = Tables(V, D, np.random.default_rng(seed))
    law = emitted_law(oracle, tab, PARENT, np.ones(D))
    assert abs(sum(law.values()) - 1.0) < 1e-12
    assert np.abs(extended_law(tab, law, D + 1) - target_joint(tab, D + 1)).max() < 1e-12
    # ... and a relaxed schedule moves it away from the target while still being a distribution
    relaxed = emitted_law(oracle, tab, PARENT, np.array([2.5, 1.5, 0.6])[:D])
    assert abs(sum(relaxed.values()) - 1.0) < 1e-12
    assert np.abs(extended_law(tab, relaxed, D + 1) - target_joint(tab, D + 1)).max() > 1e-4


def sample_rounds(oracle, tab, parent, omegas, B, seed):
    """B rounds through the real sampler: candidates drawn as the rule says, rows = logs of the tables."""
    rng = np.random.default_rng(seed)
    N, V = len(parent), tab.V
    tok = np.zeros((B, N), np.int32)
    t = np.zeros((B, N + 1, V))
    d = np.zeros((B, N + 1, V))
    prefixes = [[()] * B]                      # context 0: the root
    t[:, 0], d[:, 0] = np.log(tab.P[()]), np.log(tab.Q[()])
    for n in range(N):
        ctx = parent[n] + 1
        pre = prefixes[ctx]
        q = np.stack([tab.Q[p] for p in pre])
        cum = np.cumsum(q, axis=1)
        tok[:, n] = np.minimum((rng.random(B)[:, None] > cum).sum(1), V - 1)
        mine = [p + (int(x),) for p, x in zip(pre, tok[:, n])]
        prefixes.append(mine)
        if len(mine[0]) <= tab.D:
            t[:, n + 1] = np.log(np.stack([tab.P[p] for p in mine]))
            d[:, n + 1] = np.log(np.stack([tab.Q[p] for p in mine]))
    uni = rng.random((B, N + 1)).astype(np.float32)
    uni = np.clip(uni, 2.0 ** -24, 1 - 2.0 ** -24)
    res = oracle.verify_tree(t, d, parent, tok, uni, np.asarray(omegas, np.float32), dtype=oracle.F64, want_G=False)
    return res, tok


@pytest.mark.parametrize("omegas,name", [((1.0, 1.0, 1.0), "lossless"), ((2.5, 1.5, 0.6), "relaxed")])
def test_real_sampler_follows_the_enumerated_law(oracle, omegas, name):
    V, B = 3, 400_000
    D = oracle.tree_depth(PARENT)
    tab = Tables(V, D, np.random.default_rng(5))
    law = emitted_law(oracle, tab, PARENT, np.asarray(omegas, np.float32).astype(np.float64))
    res, tok = sample_rounds(oracle, tab, PARENT, omegas, B, seed=11)
    assert np.all(res.status == 0)
    counts = {}
    for b in range(B):
        seq = tuple(int(x) for x in res.tokens[b, :res.accept_len[b] + 1])
        counts[seq] = counts.get(seq, 0) + 1
    keys = [k for k, w in law.items() if w * B >= 5]
    obs = np.array([counts.get(k, 0) for k in keys], float)
    exp = np.array([law[k] for k in keys]) * B
    rest_o, rest_e = B - obs.sum(), B - exp.sum()
    if rest_e >= 5:
        obs, exp = np.append(obs, rest_o), np.append(exp, rest_e)
    chi2 = ((obs - exp) ** 2 / exp).sum()
    p = st.chi2.sf(chi2, len(obs) - 1)
    assert p > 1e-4, (name, chi2, len(obs), p)
    assert set(counts) <= set(law)            # nothing outside the law's support is ever emitted
    # structure: the accepted path is a root-to-node path of the tree carrying the drafted tokens
    for b in range(0, B, 997):
        prev = -1
        for lvl in range(res.accept_len[b]):
            n = res.nodes[b, lvl]
            assert PARENT[n] == prev and res.tokens[b, lvl] == tok[b, n]
            prev = n
    if name == "relaxed":
        lossless = emitted_law(oracle, tab, PARENT, np.ones(D))
        mean_len = lambda L: sum(w * len(k) for k, w in L.items())
        assert mean_len(law) > mean_len(lossless)                      # relaxation accepts more
        assert abs(res.accept_len.mean() + 1 - mean_len(law)) < 0.01


def test_chain_shaped_tree_is_algorithm_1_bit_for_bit(oracle):
    r = np.random.default_rng(0)
    for dtype, V, top_k, cfg in ((oracle.F32, 257, 0, False), (oracle.F32, 1000, 50, True), (oracle.BF16, 512, 0, False)):
        B, L = 40, 5

        def rows(n):
            a = (3 * r.standard_normal((B, n, V))).astype(np.float32)
            if dtype == oracle.BF16:
                return (a.view(np.uint32) >> 16).astype(np.uint16)
            return a

        t, d = rows(L + 1), rows(L + 1)
        tu, du = (rows(L + 1), rows(L + 1)) if cfg else (None, None)
        tok = r.integers(0, V, (B, L)).astype(np.int32)
        tok[3, 2] = V + 5                                  # a token out of range rejects on both sides
        u = np.clip(r.random((B, L + 1)), 1e-6, 1 - 1e-6).astype(np.float32)
        om = oracle.make_schedule(1, 1.3, 0.4, L).astype(np.float32)
        kw = dict(dtype=dtype, cfg_scale=1.5, top_k=top_k)
        chain = oracle.verify(t, np.ascontiguousarray(d[:, :L]), tok, u, om, target_uncond=tu,
                              draft_uncond=None if du is None else np.ascontiguousarray(du[:, :L]), **kw)
        tree = oracle.verify_tree(t, d, np.arange(-1, L - 1), tok, u, om, target_uncond=tu, draft_uncond=du, **kw)
        assert np.array_equal(chain.tokens, tree.tokens) and np.array_equal(chain.accept_len, tree.accept_len)
        assert np.array_equal(chain.status, tree.status) and np.array_equal(chain.G, tree.G)
        assert np.array_equal(chain.margin_accept, tree.margin_accept)
        assert np.array_equal(chain.margin_cdf, tree.margin_cdf)
        assert chain.accept_len.min() < L and chain.accept_len.max() >= 1


def test_tree_bad_data_and_shapes(oracle):
    r = np.random.default_rng(3)
    B, V = 6, 40
    N = len(PARENT)
    t = (2 * r.standard_normal((B, N + 1, V))).astype(np.float32)
    d = (2 * r.standard_normal((B, N + 1, V))).astype(np.float32)
    tok = r.integers(0, V, (B, N)).astype(np.int32)
    u = np.full((B, N + 1), 0.5, np.float32)
    om = np.full(3, 1e6, np.float32)                # everything usable accepts
    t[1, 0, 3] = np.nan                             # root target row unusable: nothing accepted, token -1
    d[2, 0, 5] = np.inf                             # root drafter row unusable: rejects, draws from P
    tok[3, 0] = -1                                  # first candidate unusable, the second one accepts
    res = oracle.verify_tree(t, d, PARENT, tok, u, om)
    assert res.accept_len[0] == 3 and res.status[0] == 0 and res.nodes[0].tolist() == [0, 2, 5]
    assert res.accept_len[1] == 0 and res.tokens[1, 0] == -1 and res.status[1] & 1
    assert res.accept_len[2] == 0 and res.tokens[2, 0] >= 0 and res.status[2] & 1
    assert res.status[3] & 2 and res.nodes[3, 0] == 1 and res.accept_len[3] == 2
    with pytest.raises(ValueError):
        oracle.tree_depth([0, -1])                  # a parent must be an earlier node
