"""orc_verify on realistic rows: structure of the result, agreement with library
routines (scipy softmax, cumsum/searchsorted), and the defined behaviour on bad data."""
import numpy as np
import pytest
import scipy.special as sps

from paper_2601_09212_b200 import workloads as W


def _call(oracle, w, **kw):
    h = w.host_arrays()
    return h, oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                            h["relax_schedule"], dtype=w.dtype, target_uncond=h["target_uncond"],
                            draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k, **kw)


def _decode(a, dtype):
    if dtype == W.BF16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


@pytest.mark.parametrize("bonus", [False, True])
@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
def test_verify_against_library_routines(oracle, dtype, bonus):
    B, L, V = 12, 5, 777
    sched = oracle.make_schedule(1, 1.1, 0.7, L)
    w = W.make("t", B=B, gamma=L, V=V, dtype=dtype, rho=0.8, bonus_row=bonus, schedule=sched, seed=3)
    h, r = _call(oracle, w)
    zt, zd = _decode(h["target_logits"], dtype), _decode(h["draft_logits"], dtype)
    P, Q = sps.softmax(zt, axis=-1), sps.softmax(zd, axis=-1)
    om = h["relax_schedule"].astype(np.float64)
    uni = h["uniforms"].astype(np.float64)
    tok = h["draft_tokens"]
    seen_reject = seen_full = False
    for b in range(B):
        p = P[b, np.arange(L), tok[b]]
        q = Q[b, np.arange(L), tok[b]]
        f = np.minimum(1.0, om * p / q)
        assert np.allclose(r.p[b], p, rtol=1e-12) and np.allclose(r.q[b], q, rtol=1e-12)
        assert np.allclose(r.f[b], f, rtol=1e-12)
        acc = uni[b, :L] <= f
        tau = L if acc.all() else int(np.argmin(acc))
        assert r.accept_len[b] == tau
        assert np.array_equal(r.tokens[b, :tau], tok[b, :tau])
        assert np.all(r.tokens[b, tau + 1:] == -1)
        if tau < L:
            seen_reject = True
            g = np.maximum(P[b, tau] - np.minimum(Q[b, tau], om[tau] * P[b, tau]), 0.0)
            G = g / g.sum()
            assert np.allclose(r.G[b], G, rtol=1e-10, atol=1e-16)
            cum = np.cumsum(r.G[b])
            want = int(np.searchsorted(cum, uni[b, L] * cum[-1], side="right"))
            assert r.tokens[b, tau] == want and r.G[b, want] > 0
            assert np.isclose(r.margin_accept[b, tau], abs(uni[b, tau] - f[tau]))
        else:
            seen_full = True
            if bonus:
                assert np.allclose(r.G[b], P[b, L], rtol=1e-10)
                cum = np.cumsum(P[b, L])
                assert r.tokens[b, L] == int(np.searchsorted(cum, uni[b, L] * cum[-1], side="right"))
            else:
                assert r.tokens[b, L] == -1 and np.all(r.G[b] == 0)
        assert np.all(np.isinf(r.margin_accept[b, tau + 1:]))
    assert seen_reject
    assert r.status.max() == 0


def test_verify_vanilla_schedule_equals_plain_sd(oracle):
    """omega == 1: acceptance min{1, P/Q}, resampling Norm([P - Q]_+) (vanilla SD)."""
    w = W.make("t", B=40, gamma=4, V=300, rho=0.7, seed=1)
    h, r = _call(oracle, w)
    P = sps.softmax(h["target_logits"].astype(np.float64), axis=-1)
    Q = sps.softmax(h["draft_logits"].astype(np.float64), axis=-1)
    for b in np.flatnonzero(r.accept_len < 4):
        j = r.accept_len[b]
        van = np.maximum(P[b, j] - Q[b, j], 0)
        assert np.allclose(r.G[b], van / van.sum(), rtol=1e-10, atol=1e-16)
    tok = h["draft_tokens"][..., None].astype(np.int64)
    fvan = np.minimum(1.0, np.take_along_axis(P, tok, -1)[..., 0] /
                      np.take_along_axis(Q, tok, -1)[..., 0])
    assert np.allclose(r.f, fvan, rtol=1e-12)


def test_verify_cfg_topk_path(oracle):
    B, L, V, k = 6, 3, 512, 40
    sched = oracle.make_schedule(1, 1.1, 0.7, L)
    w = W.make("t", B=B, gamma=L, V=V, dtype=W.BF16, cfg=True, cfg_scale=4.0, top_k=k, rho=0.9,
               bonus_row=True, schedule=sched, seed=4)
    h, r = _call(oracle, w)
    # rows as the oracle's own (separately pinned) preparation step builds them
    for b in range(B):
        tau = r.accept_len[b]
        zt = oracle.prepare_row(h["target_logits"][b, tau], h["target_uncond"][b, tau], W.BF16, 4.0, k)
        assert np.isfinite(zt).sum() == k or np.isfinite(zt).sum() > k   # ties may add
        assert np.all(r.G[b][~np.isfinite(zt)] == 0)                       # support inside top-k of P
        assert np.isclose(r.G[b].sum(), 1.0)
        assert np.isfinite(zt[r.tokens[b, tau]])
    # draft tokens were drawn from the filtered drafter row: q > 0 everywhere
    assert np.all(r.q > 0)


def test_verify_bad_data_semantics(oracle):
    B, L, V = 5, 3, 64
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=np.full(L, 1e6), seed=2)
    h = w.host_arrays()
    t, d, tok = h["target_logits"], h["draft_logits"], h["draft_tokens"]
    d[0, 1, 5] = np.nan          # drafter row invalid at position 2 of sequence 0
    t[1, 0, 7] = np.inf          # target row invalid at position 1 of sequence 1
    tok[2, 2] = V                # out-of-range draft token at position 3 of sequence 2
    tok[3, 0] = -1
    r = oracle.verify(t, d, tok, h["uniforms"], h["relax_schedule"])
    # omega = 1e6 accepts every healthy position
    assert r.accept_len.tolist() == [1, 0, 2, 0, 3]
    assert r.status.tolist() == [oracle.STATUS_BADROW, oracle.STATUS_BADROW,
                                 oracle.STATUS_BADTOKEN, oracle.STATUS_BADTOKEN, 0]
    P01 = sps.softmax(t[0, 1].astype(np.float64))
    assert np.allclose(r.G[0], P01, rtol=1e-10)          # invalid drafter row: G = P
    assert r.tokens[1, 0] == -1 and np.all(r.G[1] == 0)   # invalid target row: nothing to draw
    assert r.tokens[2, 2] >= 0 and r.tokens[3, 0] >= 0
    assert r.tokens[4, 3] >= 0                            # bonus token


def test_verify_identical_models_fallback(oracle):
    """P == Q with omega >= 1 never rejects (f = 1 >= r); with omega < 1 it can, and then
    G* = Norm((1 - omega) P) = P."""
    w = W.make("t", B=30, gamma=2, V=50, rho=1.0, seed=6, schedule=np.array([1.0, 0.3]))
    h = w.host_arrays()
    r = oracle.verify(h["target_logits"], h["target_logits"][:, :2].copy(), h["draft_tokens"],
                      h["uniforms"], h["relax_schedule"])
    assert np.all(r.accept_len >= 1)
    rej = np.flatnonzero(r.accept_len == 1)
    assert rej.size > 0
    for b in rej:
        assert np.allclose(r.G[b], sps.softmax(h["target_logits"][b, 1].astype(np.float64)), rtol=1e-10)
    assert r.status.max() == 0


def test_verify_reports_position_terms(oracle):
    """The optional per-position sums of Theorem 2 against scipy's softmax and their closed forms, at
    every position (also those after the first rejection), with and without guidance mix + top-k."""
    B, L, V = 6, 4, 500
    sched = oracle.make_schedule(1, 1.1, 0.7, L)
    for extra in ({}, dict(cfg=True, cfg_scale=2.5, top_k=40)):
        w = W.make("t", B=B, gamma=L, V=V, dtype=W.F32, rho=0.8, schedule=sched, seed=9, **extra)
        h = w.host_arrays()
        r = oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                          h["relax_schedule"], dtype=W.F32, target_uncond=h["target_uncond"],
                          draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k, want_terms=True)
        om = h["relax_schedule"].astype(np.float64)
        for b in range(B):
            for i in range(L):
                zt = oracle.prepare_row(h["target_logits"][b, i], None if h["target_uncond"] is None else h["target_uncond"][b, i],
                                        W.F32, w.cfg_scale, w.top_k)
                zd = oracle.prepare_row(h["draft_logits"][b, i], None if h["draft_uncond"] is None else h["draft_uncond"][b, i],
                                        W.F32, w.cfg_scale, w.top_k)
                P, Q = sps.softmax(zt), sps.softmax(zd)
                mn = np.minimum(Q, om[i] * P)
                assert np.isclose(r.accept_mass[b, i], mn.sum(), rtol=1e-11)
                assert np.isclose(r.bound_term[b, i], 2.0 * np.maximum(mn - P, 0.0).sum(), rtol=1e-9, atol=1e-13)


@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
def test_sample_rows_against_library_routines(oracle, dtype):
    """Drafting-stage draws: scipy softmax + cumsum/searchsorted on the prepared rows; chi-square of the
    drawn tokens against the row's distribution; an unusable row gives -1 and the status bit."""
    rng = np.random.default_rng(4)
    R, V = 40, 300
    w = W.make("t", B=R, gamma=1, V=V, dtype=dtype, rho=0.8, schedule=np.ones(1, np.float32), seed=12,
               cfg=True, cfg_scale=3.0, top_k=25)
    h = w.host_arrays()
    logits, unc = h["draft_logits"][:, 0], h["draft_uncond"][:, 0]
    uni = ((rng.integers(0, 2 ** 23, size=R) * 2 + 1) * 2.0 ** -24).astype(np.float32)
    tok, st, mg = oracle.sample_rows(logits, uni, dtype=dtype, uncond=unc, cfg_scale=3.0, top_k=25)
    for r in range(R):
        z = oracle.prepare_row(logits[r], unc[r], dtype, 3.0, 25)
        P = sps.softmax(z)
        cum = np.cumsum(P)
        assert tok[r] == int(np.searchsorted(cum, float(uni[r]) * cum[-1], side="right")) and P[tok[r]] > 0
        assert (np.isfinite(z)).sum() >= 25 and st[r] == 0
    # the law of the draw: many uniforms on one row
    n = 20000
    row = np.repeat(logits[:1], n, axis=0)
    us = ((rng.integers(0, 2 ** 23, size=n) * 2 + 1) * 2.0 ** -24).astype(np.float32)
    toks, _, _ = oracle.sample_rows(row, us, dtype=dtype, uncond=np.repeat(unc[:1], n, axis=0), cfg_scale=3.0, top_k=25)
    P = sps.softmax(oracle.prepare_row(logits[0], unc[0], dtype, 3.0, 25))
    keep = P > 0
    obs = np.bincount(toks, minlength=V)[keep]
    assert obs.sum() == n
    chi2 = ((obs - n * P[keep]) ** 2 / (n * P[keep])).sum()
    assert chi2 < 25 + 6 * np.sqrt(2 * 25)          # about 6 sigma for keep.sum() - 1 degrees of freedom
    bad = np.array(logits[:2], copy=True)
    bad_f = _decode(bad, dtype)
    if dtype == W.F32:
        bad[1, 3] = np.nan
        tok2, st2, _ = oracle.sample_rows(bad, uni[:2], dtype=dtype, uncond=unc[:2], cfg_scale=3.0, top_k=25)
        assert tok2[1] == -1 and st2[1] == oracle.STATUS_BADROW and tok2[0] == tok[0]
