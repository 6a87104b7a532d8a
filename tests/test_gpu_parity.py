"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs and the same supplied uniforms.  Accepted lengths and tokens must be identical
except for decisions the oracle flags as within 1e-6 of a threshold (counted); probabilities and
the resampling distribution within 1e-5 (fp32 logits) / 2e-3 (bf16 logits) absolute."""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import oracle
import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W
from gpu_util import check, run_gpu, run_oracle

DEV = "cuda"


def sched(L, kind="exp"):
    if kind == "vanilla":
        return np.ones(L, np.float32)
    return csd.csd_make_schedule(1, 1.1, 0.7, L)


def assert_ok(rep, max_near_frac=0.02):
    assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:5])
    assert rep.tau_mismatch_near + rep.token_mismatch_near <= max(2, max_near_frac * rep.n_seq), rep.summary()


@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("V", [2, 8, 33, 1000, 1024, 4100, 16384, 20000])
@pytest.mark.parametrize("bonus", [False, True])
def test_shapes_small(dtype, V, bonus):
    L = 5
    w = W.make("t", B=7, gamma=L, V=V, dtype=dtype, rho=0.8, bonus_row=bonus, schedule=sched(L),
               seed=V, device=DEV)
    rep, got, ref = check(w)
    assert_ok(rep)


@pytest.mark.parametrize("L", [1, 2, 16, 31, 32])
def test_gamma_range(L):
    w = W.make("t", B=5, gamma=L, V=2048, rho=0.95, bonus_row=True,
               schedule=csd.csd_make_schedule(0, 1.5, 0.0, L), seed=L, device=DEV)
    rep, got, ref = check(w)
    assert_ok(rep)
    assert got["accept_len"].max() > 2 or L <= 2


@pytest.mark.parametrize("name,rho,kind", [("C1", 0.9, "exp"), ("C2", 0.7, "vanilla"), ("C2", 0.9, "exp"),
                                           ("C2", 0.97, "vanilla"), ("C2", 0.97, "exp")])
def test_config_c1_c2(name, rho, kind):
    L = W.CONFIGS[name]["gamma"]
    reps = []
    for step in range(3):
        w = W.config(name, step=step, rho=rho, schedule=sched(L, kind), device=DEV)
        rep, got, ref = check(w)
        assert_ok(rep)
        reps.append(rep)
    print(name, rho, kind, reps[0].summary())


def test_vanilla_schedule_matches_plain_sd_on_gpu():
    """omega == 1: the distribution drawn from is Norm([P - Q]_+) (Proposition 2)."""
    w = W.make("t", B=32, gamma=4, V=4096, rho=0.8, schedule=sched(4, "vanilla"), seed=5, device=DEV)
    got = run_gpu(w)
    P = torch.softmax(w.target_logits.double(), -1).cpu().numpy()
    Q = torch.softmax(w.draft_logits.double(), -1).cpu().numpy()
    n = 0
    for b in range(32):
        j = got["accept_len"][b]
        if j < 4:
            van = np.maximum(P[b, j] - Q[b, j], 0)
            assert np.abs(got["G"][b] - van / van.sum()).max() < 1e-5
            n += 1
    assert n > 0
    assert abs(got["G"].sum(-1)[got["accept_len"] < 4] - 1).max() < 1e-4


def test_bf16_large_batch_c4_sampled():
    """Full-size heavy-tailed config: oracle on a sample of sequences."""
    L = W.CONFIGS["C4"]["gamma"]
    w = W.config("C4", step=0, schedule=sched(L), device=DEV)
    rows = np.arange(0, 256, 8)
    rep, got, ref = check(w, rows=rows, want_dbg=True)
    assert_ok(rep)
    # properties that hold for every sequence
    tau = got["accept_len"]
    assert tau.min() >= 0 and tau.max() <= L
    tok = w.draft_tokens.cpu().numpy()
    for b in range(256):
        assert np.array_equal(got["tokens"][b, :tau[b]], tok[b, :tau[b]])
        assert np.all(got["tokens"][b, tau[b] + 1:] == -1)
        if tau[b] < L:
            assert 0 <= got["tokens"][b, tau[b]] < w.V
            assert abs(got["G"][b].sum() - 1) < 1e-3 and got["G"][b].min() >= 0
            assert got["G"][b, got["tokens"][b, tau[b]]] > 0


@pytest.mark.parametrize("kw", [
    dict(B=256, gamma=16, V=65536, dtype=W.BF16),
    dict(B=256, gamma=4, V=65536, dtype=W.F32),
    dict(B=64, gamma=16, V=32768, dtype=W.F32),
    dict(B=16, gamma=8, V=4096, dtype=W.BF16),
    dict(B=1, gamma=16, V=65536, dtype=W.F32),
])
def test_sweep_grid_corners_sampled(kw):
    """Corners of the V x gamma x B x dtype sweep at full size, in the partition used for timing
    (calls enqueued back to back): the oracle on a sample of sequences, structure on all of them."""
    L, B = kw["gamma"], kw["B"]
    w = W.make("t", rho=0.9, schedule=sched(L), seed=55, device=DEV, **kw)
    rows = np.unique(np.linspace(0, B - 1, 8).astype(int))
    rep, got, ref = check(w, rows=rows, want_dbg=True, back_to_back=True)
    assert_ok(rep)
    tau, tok = got["accept_len"], w.draft_tokens.cpu().numpy()
    assert tau.min() >= 0 and tau.max() <= L and np.all(got["status"] == 0)
    for b in range(B):
        assert np.array_equal(got["tokens"][b, :tau[b]], tok[b, :tau[b]])
        assert np.all(got["tokens"][b, tau[b] + 1:] == -1)
        if tau[b] < L:
            assert 0 <= got["tokens"][b, tau[b]] < w.V and got["G"][b, got["tokens"][b, tau[b]]] > 0
    base = run_gpu(w, want_dbg=False)
    assert np.array_equal(base["tokens"], got["tokens"]) and np.array_equal(base["accept_len"], got["accept_len"])


@pytest.mark.parametrize("i", range(16))
def test_seeded_sweep_of_tied_topk_rows(i):
    """Logits rounded to a coarse grid: the k-th largest value is shared by many tokens (all of them are
    kept), histogram bins are crowded, candidate lists overflow -- the streaming selection has to hand
    such rows to the exact one, and both must agree with the oracle's threshold rule."""
    r = np.random.default_rng(4000 + i)
    V = int(r.choice([1000, 4096, 16384, 20000]))
    kw = dict(B=int(r.choice([2, 9, 40])), gamma=int(r.choice([2, 5, 8])), V=V,
              dtype=[W.F32, W.BF16][int(r.integers(2))], bonus_row=bool(r.integers(2)), cfg=bool(r.integers(2)),
              top_k=int(r.integers(1, max(2, V // 4))), rho=0.9)
    L = kw["gamma"]
    w = W.make("t", schedule=sched(L), seed=4100 + i, device=DEV, **kw)
    q = float(r.choice([0.125, 0.5, 2.0]))
    for t in (w.target_logits, w.draft_logits, w.target_uncond, w.draft_uncond):
        if t is not None:
            t.copy_((t.float() / q).round() * q)
    b2b = bool(r.integers(2))
    rep, got, ref = check(w, back_to_back=b2b, want_dbg=kw["B"] * V <= 4e6)
    assert_ok(rep)
    other = run_gpu(w, want_dbg=False, back_to_back=not b2b)
    for key in ("tokens", "accept_len", "status"):
        assert np.array_equal(got[key], other[key]), (key, kw, b2b)


def test_cfg_mix_fused():
    L = 6
    for dtype in (W.F32, W.BF16):
        w = W.make("t", B=9, gamma=L, V=3000 if dtype == W.F32 else 4096, dtype=dtype, cfg=True,
                   cfg_scale=4.0, rho=0.9, bonus_row=True, schedule=sched(L), seed=11, device=DEV)
        rep, got, ref = check(w)
        assert_ok(rep)


@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("V,k", [(64, 1), (64, 63), (1000, 10), (4096, 1000), (5000, 4999), (16384, 1000),
                                 (20000, 50), (70000, 1000)])
def test_topk_filter(dtype, V, k):
    """Top-k before the softmax (keep every logit >= the k-th largest of its row), with and
    without the guidance mix; bf16 rows hold many tied values, which the tie rule must keep."""
    L = 4
    for cfg in (False, True):
        w = W.make("t", B=5, gamma=L, V=V, dtype=dtype, rho=0.9, bonus_row=True, cfg=cfg, top_k=k,
                   schedule=sched(L), seed=V + k, device=DEV)
        rep, got, ref = check(w)
        assert_ok(rep)
        live = got["accept_len"] < L
        # the distribution drawn from has at most the kept tokens in its support
        assert ((got["G"] > 0).sum(-1) >= 1).all()
        if dtype == W.F32 and not cfg:
            assert ((got["G"] > 0).sum(-1) <= k).all()


def test_topk_with_masked_and_tied_rows():
    """Rows with fewer than k finite entries (threshold -inf: nothing more is removed) and rows
    where the k-th largest value is shared by many tokens."""
    B, L, V, k = 4, 3, 512, 100
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, top_k=k, schedule=sched(L), seed=1, device=DEV)
    w.target_logits[0, 0, 50:] = float("-inf")
    w.draft_logits[0, 0, 50:] = float("-inf")
    w.draft_tokens[0, 0] = 7
    w.target_logits[1, :, :] = torch.round(w.target_logits[1, :, :])       # heavy ties
    w.draft_logits[1, :, :] = torch.round(w.draft_logits[1, :, :])
    w.target_logits[2, 1, :] = 0.0                                         # all equal: everything kept
    w.target_logits[3, 0, 5] = -0.0
    w.target_logits[3, 0, 6] = 0.0
    rep, got, ref = check(w)
    assert_ok(rep)


@pytest.mark.parametrize("kw", [dict(V=65536, dtype=W.BF16, cfg=True, cfg_scale=3.0, top_k=2000),
                                dict(V=32768, dtype=W.F32, top_k=2400),
                                dict(V=50000, dtype=W.BF16, cfg=True, top_k=1800),
                                dict(V=65536, dtype=W.BF16, top_k=2000, law="student3"),
                                dict(V=20000, dtype=W.F32, cfg=True, top_k=1400)])
@pytest.mark.parametrize("b2b", [False, True])
def test_topk_beyond_the_small_lists(kw, b2b):
    """k between about 1200 and 2400 (a 65536-token vocabulary filtered to its 2000 best, say): the
    streaming selection runs on the instance of the kernel with the larger candidate lists; whole and
    ragged rows, Gaussian and heavy-tailed logits."""
    L = 4
    w = W.make("t", B=10, gamma=L, rho=0.9, bonus_row=True, schedule=sched(L), seed=kw["V"] % 97, device=DEV, **kw)
    w.target_logits[1, 0, :] = torch.round(w.target_logits[1, 0, :])     # heavy ties around the threshold
    rep, got, ref = check(w, back_to_back=b2b, want_dbg=False)
    assert_ok(rep)
    rep, got, ref = check(w, back_to_back=b2b)                            # with G: the full selection, exact thresholds
    assert_ok(rep)


@pytest.mark.parametrize("kw", [
    dict(B=64, gamma=8, V=16384, dtype=W.F32),
    dict(B=64, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000),
    dict(B=40, gamma=16, V=8192, dtype=W.BF16, bonus_row=True),
    dict(B=3, gamma=7, V=32768, dtype=W.F32, bonus_row=True, top_k=50),
    dict(B=24, gamma=5, V=4100, dtype=W.BF16),
])
def test_back_to_back_partition(kw):
    """The partition for calls enqueued back to back (one block per sequence, programmatic launch)
    against the oracle, and against the default partition (sequences split over the blocks of a
    cluster): identical integer outputs."""
    L = kw["gamma"]
    w = W.make("t", rho=0.9, schedule=sched(L), seed=77, device=DEV, **kw)
    rep, got, ref = check(w, back_to_back=True)
    assert_ok(rep)
    base = run_gpu(w, want_dbg=False)
    assert np.array_equal(got["tokens"], base["tokens"])
    assert np.array_equal(got["accept_len"], base["accept_len"])
    assert np.array_equal(got["status"], base["status"])


@pytest.mark.parametrize("kw", [
    dict(B=4, gamma=3, V=65536, dtype=W.BF16, bonus_row=True),
    dict(B=2, gamma=2, V=131072, dtype=W.F32),                      # the last size of the single-launch path (fp32)
    dict(B=2, gamma=2, V=131076, dtype=W.F32),                      # one tile more: multi-launch path
    dict(B=2, gamma=3, V=262144, dtype=W.BF16, top_k=1000),
    dict(B=1, gamma=2, V=2 ** 20, dtype=W.F32, bonus_row=True),     # the largest vocabulary accepted
    dict(B=1, gamma=2, V=2 ** 20, dtype=W.BF16, top_k=50),
    dict(B=1, gamma=16, V=8192, dtype=W.F32, bonus_row=True),       # clusters of 8 by default
])
def test_large_vocabularies_and_limits(kw):
    L = kw["gamma"]
    w = W.make("t", rho=0.9, schedule=sched(L), seed=5, device=DEV, **kw)
    for b2b in (False, True):
        rep, got, ref = check(w, back_to_back=b2b)
        assert_ok(rep)


@pytest.mark.parametrize("B", [147, 148, 149, 295, 296, 297, 1183, 1184, 1185, 2368, 2369])
def test_partition_boundaries(B):
    """Batch sizes on both sides of every point where the launch partition changes (multiples of the 148
    SMs: clusters -> one block per sequence -> several sequences per block), both stream modes."""
    L = 3
    for dtype, V, top_k in ((W.BF16, 1024, 0), (W.F32, 512, 40)):
        w = W.make("t", B=B, gamma=L, V=V, dtype=dtype, rho=0.9, bonus_row=True, top_k=top_k, schedule=sched(L),
                   seed=B, device=DEV)
        rep, got, ref = check(w, want_dbg=False)
        assert_ok(rep)
        other = run_gpu(w, want_dbg=False, back_to_back=True)
        for key in ("tokens", "accept_len", "status"):
            assert np.array_equal(got[key], other[key]), (key, B)


def _random_case(i):
    """Case i of a seeded sweep over the launch partition's inputs: batch sizes on both sides of the
    points where sequences are split over a cluster, kept one per block or merged several per block;
    every draft length class; vocabularies with ragged tails; dtype, guidance mix, top-k, bonus row."""
    r = np.random.default_rng(1000 + i)
    B = int(r.choice([1, 2, 3, 5, 9, 15, 16, 17, 33, 70, 149, 297, 600, 1300]))
    L = int(r.choice([1, 2, 3, 4, 7, 8, 12, 16, 32]))
    V = int(r.choice([16, 250, 1000, 2048, 3001, 4096, 8200, 16384, 40000]))
    while B * L * V > 2.2e7:                       # keep the oracle to a few seconds per case
        if V > 1000: V //= 2
        else: B = max(1, B // 2)
    kw = dict(B=B, gamma=L, V=V, dtype=[W.F32, W.BF16][int(r.integers(2))], bonus_row=bool(r.integers(2)),
              rho=float(r.choice([0.5, 0.9, 0.99])))
    if r.integers(3) == 0:
        kw["cfg"] = True
    if r.integers(3) == 0:
        kw["top_k"] = int(min(V - 1, r.choice([1, 7, 100, 1000])))
    if r.integers(4) == 0:
        kw["law"] = "student3"                     # heavy tails: the selection's guess misses and adapts
    b2b = bool(r.integers(2))
    r2 = np.random.default_rng(7000 + i)           # (a second stream, so that the cases above stay what they were)
    if r2.integers(4) == 0 and V >= 8192:          # k beyond the small candidate lists, and beyond the large ones
        kw["top_k"] = int(min(V - 1, r2.choice([1200, 1500, 2000, 2400, 3000])))
    return kw, b2b


# CSD_SWEEP_CASES=8000 runs the same sweep over that many cases (about six minutes on a B200)
@pytest.mark.parametrize("i", range(int(os.environ.get("CSD_SWEEP_CASES", "96"))))
def test_seeded_sweep_of_partitions(i):
    kw, b2b = _random_case(i)
    L = kw["gamma"]
    w = W.make("t", schedule=sched(L, "exp" if i % 3 else "vanilla"), seed=300 + i, device=DEV, **kw)
    rep, got, ref = check(w, back_to_back=b2b, want_dbg=kw["B"] * kw["V"] <= 4e6)
    assert_ok(rep)
    other = run_gpu(w, want_dbg=False, back_to_back=not b2b)
    for key in ("tokens", "accept_len", "status"):
        assert np.array_equal(got[key], other[key]), (key, kw, b2b)
    if i % 4 == 0:                                  # the per-position monitors on the same inputs
        mon = run_gpu(w, want_dbg=False, want_terms=True, back_to_back=b2b)
        assert np.array_equal(mon["tokens"], got["tokens"])
        _, ref_t = run_oracle(w, want_G=False, want_terms=True)
        tol = 1e-5 if w.dtype == W.F32 else 2e-3
        assert np.abs(mon["accept_mass"] - ref_t.accept_mass).max() < tol
        assert np.abs(mon["bound_term"] - ref_t.bound_term).max() < 2 * tol
    if i % 4 == 1:                                  # the drafting stage's draw on the first draft rows
        logits = w.draft_logits[:, 0].contiguous()
        unc = None if w.draft_uncond is None else w.draft_uncond[:, 0].contiguous()
        uni = w.uniforms[:, 0].contiguous()
        tok = torch.full((w.B,), -7, dtype=torch.int32, device=DEV)
        csd.csd_sample_rows(logits, uni, tok, uncond=unc, cfg_scale=w.cfg_scale, top_k=w.top_k, back_to_back=b2b)
        torch.cuda.synchronize()
        h = w.host_arrays()
        ref_tok, _, margin = oracle.sample_rows(
            h["draft_logits"][:, 0], h["uniforms"][:, 0], dtype=w.dtype,
            uncond=None if h["draft_uncond"] is None else h["draft_uncond"][:, 0], cfg_scale=w.cfg_scale,
            top_k=w.top_k)
        differ = tok.cpu().numpy() != ref_tok
        assert np.all(margin[differ] < 1e-6) and differ.sum() <= max(1, w.B // 50)


@pytest.mark.parametrize("b2b", [False, True])
@pytest.mark.parametrize("kw", [
    dict(B=20, gamma=8, V=16384, dtype=W.F32),
    dict(B=20, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000),
    dict(B=3, gamma=6, V=8192, dtype=W.BF16, bonus_row=True),
    dict(B=5, gamma=4, V=4100, dtype=W.F32, top_k=37),           # multi-launch path
    dict(B=40, gamma=3, V=2048, dtype=W.F32),
])
def test_theorem2_position_terms(kw, b2b):
    """The optional per-position monitors (inner sum of Eq. token_exp, bracket of Eq. bd2) against the
    oracle's, at every position of every sequence; asking for them must not change the round itself."""
    L = kw["gamma"]
    for schedule in (sched(L), csd.csd_make_schedule(0, 1.7, 0.0, L), np.ones(L, np.float32)):
        w = W.make("t", rho=0.85, schedule=schedule, seed=31, device=DEV, **kw)
        got = run_gpu(w, want_dbg=False, want_terms=True, back_to_back=b2b)
        base = run_gpu(w, want_dbg=False, back_to_back=b2b)
        assert np.array_equal(got["tokens"], base["tokens"]) and np.array_equal(got["accept_len"], base["accept_len"])
        h = w.host_arrays()
        ref = oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                            h["relax_schedule"], dtype=w.dtype, target_uncond=h["target_uncond"],
                            draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k,
                            want_G=False, want_terms=True)
        tol = 1e-5 if w.dtype == W.F32 else 2e-3
        assert np.abs(got["accept_mass"] - ref.accept_mass).max() < tol
        assert np.abs(got["bound_term"] - ref.bound_term).max() < 2 * tol
        if np.all(np.asarray(schedule) <= 1.0):
            assert np.abs(got["bound_term"]).max() < 2 * tol     # vanilla: the bound's bracket vanishes


def test_position_terms_on_unusable_rows():
    L = 4
    w = W.make("t", B=6, gamma=L, V=4096, dtype=W.F32, rho=0.9, schedule=sched(L), seed=8, device=DEV)
    w.target_logits[1, 2, 17] = float("nan")
    w.draft_logits[3, 0, :] = float("-inf")
    got = run_gpu(w, want_dbg=False, want_terms=True)
    assert np.isnan(got["accept_mass"][1, 2]) and np.isnan(got["bound_term"][1, 2])
    assert np.isnan(got["accept_mass"][3, 0]) and np.isnan(got["bound_term"][3, 0])
    ok = np.ones((6, L), bool); ok[1, 2] = ok[3, 0] = False
    assert np.all(np.isfinite(got["accept_mass"][ok])) and np.all(got["accept_mass"][ok] <= 1.0 + 1e-5)


@pytest.mark.parametrize("b2b", [False, True])
@pytest.mark.parametrize("kw", [
    dict(R=64, V=16384, dtype=W.F32),
    dict(R=300, V=16384, dtype=W.BF16, cfg=True, top_k=1000),
    dict(R=5, V=65536, dtype=W.BF16),
    dict(R=33, V=4100, dtype=W.F32, top_k=50),            # multi-launch path
    dict(R=1, V=2048, dtype=W.F32, cfg=True),
    dict(R=1500, V=2048, dtype=W.BF16),                   # several rows per block
])
def test_drafting_stage_sampling(kw, b2b):
    """csd_sample_rows (Algorithm 1, drafting stage) against the oracle's draws on the same rows and
    uniforms: identical tokens except where the oracle reports the uniform within 1e-6 of a CDF boundary."""
    kw = dict(kw)
    R = kw.pop("R")
    w = W.make("t", B=R, gamma=1, rho=0.9, schedule=np.ones(1, np.float32), seed=41, device=DEV, **kw)
    logits = w.draft_logits[:, 0].contiguous()
    unc = None if w.draft_uncond is None else w.draft_uncond[:, 0].contiguous()
    uni = w.uniforms[:, 0].contiguous()
    tok = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    st = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    csd.csd_sample_rows(logits, uni, tok, uncond=unc, cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=st,
                        back_to_back=b2b)
    torch.cuda.synchronize()
    h = w.host_arrays()
    ref_tok, ref_st, margin = oracle.sample_rows(
        h["draft_logits"][:, 0], h["uniforms"][:, 0], dtype=w.dtype,
        uncond=None if h["draft_uncond"] is None else h["draft_uncond"][:, 0], cfg_scale=w.cfg_scale, top_k=w.top_k)
    got = tok.cpu().numpy()
    differ = got != ref_tok
    assert np.all(margin[differ] < 1e-6), (np.flatnonzero(differ)[:5], margin[differ][:5])
    assert differ.sum() <= max(1, R // 50)
    assert np.array_equal(st.cpu().numpy(), ref_st)
    assert got.min() >= 0 and got.max() < w.V


@pytest.mark.parametrize("kw", [
    dict(B=40, gamma=3, V=4096, dtype=W.BF16, cfg=True, top_k=200),
    dict(B=7, gamma=2, V=16384, dtype=W.F32),
    dict(B=300, gamma=1, V=1000, dtype=W.BF16, bonus_row=True),
])
def test_drafting_stage_sampling_of_spaced_rows(kw):
    """Rows taken out of a [B, T, V] tensor (the last position of every sequence): the row stride reaches
    the library, and the draws equal those from a packed copy of the same rows."""
    w = W.make("t", rho=0.9, schedule=sched(kw["gamma"]), seed=61, device=DEV, **kw)
    last = w.target_logits.shape[1] - 1
    view = w.target_logits[:, last]
    unc = None if w.target_uncond is None else w.target_uncond[:, last]
    assert not view.is_contiguous() or last == 0
    uni = w.uniforms[:, 0].contiguous()
    toks = []
    for lg, un in ((view, unc), (view.contiguous(), None if unc is None else unc.contiguous())):
        tok = torch.full((w.B,), -7, dtype=torch.int32, device=DEV)
        csd.csd_sample_rows(lg, uni, tok, uncond=un, cfg_scale=w.cfg_scale, top_k=w.top_k)
        torch.cuda.synchronize()
        toks.append(tok.cpu().numpy())
    assert np.array_equal(toks[0], toks[1]) and toks[0].min() >= 0
    h = w.host_arrays()
    ref_tok, _, margin = oracle.sample_rows(
        h["target_logits"][:, last], h["uniforms"][:, 0], dtype=w.dtype,
        uncond=None if h["target_uncond"] is None else h["target_uncond"][:, last], cfg_scale=w.cfg_scale, top_k=w.top_k)
    differ = toks[0] != ref_tok
    assert np.all(margin[differ] < 1e-6) and differ.sum() <= max(1, w.B // 50)


def test_drafting_stage_sampling_bad_row_and_errors():
    R, V = 6, 4096
    logits = torch.randn(R, V, device=DEV)
    logits[2, 7] = float("nan")
    logits[4, :] = float("-inf")
    uni = torch.full((R,), 0.37, device=DEV)
    tok = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    st = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    csd.csd_sample_rows(logits, uni, tok, out_status=st)
    torch.cuda.synchronize()
    t, s_ = tok.cpu().numpy(), st.cpu().numpy()
    assert t[2] == -1 and t[4] == -1 and s_[2] == 1 and s_[4] == 1
    assert np.all(t[[0, 1, 3, 5]] >= 0) and np.all(s_[[0, 1, 3, 5]] == 0)
    lib = csd.library()
    assert lib.csd_sample_rows(None, None, 1.0, 0, 0, R, V, 0, None, None, None, None, 0, 0, None) == -1
    assert csd.csd_sample_workspace_size(0, V, 0) == 0


@pytest.mark.parametrize("b2b", [False, True])
def test_topk_on_heavy_tailed_rows(b2b):
    """Student-t logits: the normal-quantile guess of the streaming selection misses, rows are selected
    exactly or with the adapted guess; the results must not depend on which."""
    L = 8
    w = W.make("t", B=20, gamma=L, V=16384, dtype=W.BF16, rho=0.85, law="student3", top_k=1000,
               schedule=sched(L), seed=13, device=DEV)
    rep, got, ref = check(w, back_to_back=b2b)
    assert_ok(rep)
    w = W.make("t", B=6, gamma=4, V=16384, dtype=W.F32, rho=0.85, law="student3", cfg=True, top_k=300,
               schedule=sched(4), seed=14, device=DEV)
    rep, got, ref = check(w, back_to_back=b2b)
    assert_ok(rep)


def test_config_c3_guidance_and_topk():
    """B=64, gamma=8, V=16384, bf16, guidance mix s=4 fused into the load, top-k 1000."""
    L = W.CONFIGS["C3"]["gamma"]
    for step in range(2):
        w = W.config("C3", step=step, schedule=sched(L), device=DEV)
        rep, got, ref = check(w)
        assert_ok(rep)
        print("C3", rep.summary())


@pytest.mark.parametrize("name,kw,b2b", [
    ("plain, one block per sequence, overlapping", dict(B=16, gamma=8, V=16384, dtype=W.F32), True),
    ("plain, clusters of 8, stream order", dict(B=16, gamma=8, V=16384, dtype=W.F32), False),
    ("plain, clusters of 4, stream order", dict(B=64, gamma=8, V=16384, dtype=W.F32), False),
    ("plain, clusters of 2, overlapping", dict(B=8, gamma=8, V=16384, dtype=W.BF16), True),
    ("top-k with guidance, one block per sequence, overlapping",
     dict(B=64, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000), True),
    ("top-k with guidance, clusters of 4, stream order",
     dict(B=64, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000), False),
    ("top-k with guidance, clusters of 4, overlapping",
     dict(B=4, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000), True),
    ("several sequences per block, overlapping", dict(B=1500, gamma=2, V=2048, dtype=W.BF16), True),
])
def test_back_to_back_calls_on_one_stream(name, kw, b2b):
    """Consecutive calls (with back_to_back they overlap on the device through programmatic dependent
    launch) share ONE workspace and ONE set of output buffers per slot; every call's results must equal those of
    the same call run alone, both when enqueued directly and when replayed as a CUDA graph."""
    L = kw["gamma"]
    n = 6
    ws_shared = csd.new_workspace(kw["B"], L, kw["V"], kw["dtype"], DEV)
    steps = [W.make("t", rho=0.9, schedule=sched(L), seed=100 + i, device=DEV, **kw) for i in range(n)]
    alone = [run_gpu(w, want_dbg=False) for w in steps]
    outs = [dict(tok=torch.full((w.B, L + 1), -7, dtype=torch.int32, device=DEV),
                 tau=torch.full((w.B,), -7, dtype=torch.int32, device=DEV),
                 st=torch.full((w.B,), -7, dtype=torch.int32, device=DEV)) for w in steps]
    stream = torch.cuda.Stream()
    prms = [csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                            o["tok"], o["tau"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                            cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=o["st"], workspace=ws_shared,
                            stream=stream, back_to_back=b2b) for w, o in zip(steps, outs)]

    def check_all(tag):
        for i, (o, ref) in enumerate(zip(outs, alone)):
            assert np.array_equal(o["tok"].cpu().numpy(), ref["tokens"]), (tag, name, i)
            assert np.array_equal(o["tau"].cpu().numpy(), ref["accept_len"]), (tag, name, i)
            assert np.array_equal(o["st"].cpu().numpy(), ref["status"]), (tag, name, i)
            o["tok"].fill_(-7); o["tau"].fill_(-7); o["st"].fill_(-7)

    with torch.cuda.stream(stream):
        for _ in range(3):
            for p in prms:
                csd.csd_verify_ex(p)
    stream.synchronize()
    check_all("direct")
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for p in prms:
            csd.csd_verify_ex(p)
    with torch.cuda.stream(stream):
        for _ in range(5):
            g.replay()
    stream.synchronize()
    check_all("graph")


@pytest.mark.parametrize("b2b", [False, True])
def test_mixed_calls_share_one_stream_and_workspace(b2b):
    """Calls of different shapes and kinds -- both single-launch kernels in every partition, the
    multi-launch path, the drafting-stage draw -- enqueued one after the other on one stream with ONE
    workspace, directly and as a replayed CUDA graph: each must give what it gives alone."""
    kinds = [
        dict(B=16, gamma=8, V=16384, dtype=W.F32),
        dict(B=64, gamma=8, V=16384, dtype=W.BF16, cfg=True, top_k=1000),
        dict(B=5, gamma=4, V=3001, dtype=W.F32, top_k=20),                 # multi-launch path
        dict(B=3, gamma=16, V=8192, dtype=W.BF16, bonus_row=True),         # clusters
        dict(B=9, gamma=3, V=250, dtype=W.BF16, cfg=True),                 # multi-launch path
        dict(B=700, gamma=2, V=2048, dtype=W.BF16, bonus_row=True),
        dict(B=1500, gamma=2, V=1024, dtype=W.F32, top_k=5),               # several sequences per block
    ]
    steps = [W.make("t", rho=0.9, schedule=sched(kw["gamma"]), seed=200 + i, device=DEV, **kw)
             for i, kw in enumerate(kinds)]
    alone = [run_gpu(w, want_dbg=False) for w in steps]
    size = max(csd.csd_workspace_size(w.B, w.gamma, w.V, w.dtype) for w in steps)
    size = max(size, csd.csd_sample_workspace_size(64, 16384, W.BF16))
    ws = torch.zeros(size, dtype=torch.uint8, device=DEV)
    outs = [dict(tok=torch.full((w.B, w.gamma + 1), -7, dtype=torch.int32, device=DEV),
                 tau=torch.full((w.B,), -7, dtype=torch.int32, device=DEV),
                 st=torch.full((w.B,), -7, dtype=torch.int32, device=DEV)) for w in steps]
    stream = torch.cuda.Stream()
    prms = [csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                            o["tok"], o["tau"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                            cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=o["st"], workspace=ws,
                            stream=stream, back_to_back=b2b) for w, o in zip(steps, outs)]
    # the drafting-stage draw between them, on the guided rows of the second workload
    d = steps[1]
    d_logits, d_unc = d.draft_logits[:, 0].contiguous(), d.draft_uncond[:, 0].contiguous()
    d_uni = d.uniforms[:, 0].contiguous()
    d_tok = torch.full((d.B,), -7, dtype=torch.int32, device=DEV)
    csd.csd_sample_rows(d_logits, d_uni, d_tok, uncond=d_unc, cfg_scale=d.cfg_scale, top_k=d.top_k)
    torch.cuda.synchronize()
    d_alone = d_tok.cpu().numpy().copy()

    def enqueue():
        for i, p in enumerate(prms):
            csd.csd_verify_ex(p)
            if i % 3 == 1:
                csd.csd_sample_rows(d_logits, d_uni, d_tok, uncond=d_unc, cfg_scale=d.cfg_scale, top_k=d.top_k,
                                    workspace=ws, back_to_back=b2b, stream=stream)

    def check_all(tag):
        for i, (o, ref) in enumerate(zip(outs, alone)):
            assert np.array_equal(o["tok"].cpu().numpy(), ref["tokens"]), (tag, i)
            assert np.array_equal(o["tau"].cpu().numpy(), ref["accept_len"]), (tag, i)
            assert np.array_equal(o["st"].cpu().numpy(), ref["status"]), (tag, i)
            o["tok"].fill_(-7); o["tau"].fill_(-7); o["st"].fill_(-7)
        assert np.array_equal(d_tok.cpu().numpy(), d_alone), tag
        d_tok.fill_(-7)

    with torch.cuda.stream(stream):
        for _ in range(3):
            enqueue()
    stream.synchronize()
    check_all("direct")
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        enqueue()
    with torch.cuda.stream(stream):
        for _ in range(4):
            g.replay()
    stream.synchronize()
    check_all("graph")


def test_batch_strides_and_unaligned_views():
    """Rows embedded in a larger buffer (batch stride > rows*V) and a base pointer that is
    only element-aligned (forces the scalar path)."""
    L, V, B = 4, 1000, 6
    w = W.make("t", B=B, gamma=L, V=V, rho=0.85, bonus_row=True, schedule=sched(L), seed=2, device=DEV)
    ref_rep, got_plain, ref = check(w)
    assert_ok(ref_rep)
    pad = 24
    big_t = torch.zeros(B, (L + 1) * V + pad, device=DEV)
    big_d = torch.zeros(B, L * V + pad, device=DEV)
    big_t[:, :(L + 1) * V] = w.target_logits.reshape(B, -1)
    big_d[:, :L * V] = w.draft_logits.reshape(B, -1)
    out_t = torch.empty(B, L + 1, dtype=torch.int32, device=DEV)
    out_l = torch.empty(B, dtype=torch.int32, device=DEV)
    ws = csd.new_workspace(B, L, V, w.dtype)   # (held: the parameter block keeps raw pointers)
    prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                          out_t, out_l, workspace=ws)
    prm.target_logits = big_t.data_ptr()
    prm.draft_logits = big_d.data_ptr()
    prm.target_batch_stride = big_t.shape[1]
    prm.draft_batch_stride = big_d.shape[1]
    csd.csd_verify_ex(prm)
    torch.cuda.synchronize()
    assert np.array_equal(out_t.cpu().numpy(), got_plain["tokens"])
    assert np.array_equal(out_l.cpu().numpy(), got_plain["accept_len"])
    # element-aligned only: shift everything by one float
    flat_t = torch.zeros(B * (L + 1) * V + 1, device=DEV)
    flat_d = torch.zeros(B * L * V + 1, device=DEV)
    flat_t[1:] = w.target_logits.reshape(-1)
    flat_d[1:] = w.draft_logits.reshape(-1)
    prm.target_logits = flat_t.data_ptr() + 4
    prm.draft_logits = flat_d.data_ptr() + 4
    prm.target_batch_stride = (L + 1) * V
    prm.draft_batch_stride = L * V
    csd.csd_verify_ex(prm)
    torch.cuda.synchronize()
    assert np.array_equal(out_t.cpu().numpy(), got_plain["tokens"])
    assert np.array_equal(out_l.cpu().numpy(), got_plain["accept_len"])


@pytest.mark.parametrize("i", range(12))
def test_seeded_sweep_of_batch_strides(i):
    """Sequences embedded in larger buffers (batch stride > rows x V) on random shapes: with a padding that
    keeps rows 16-byte aligned (single-launch kernels) and one that does not (multi-launch path), the
    same integers as from contiguous inputs."""
    kw, b2b = _random_case(1500 + i)
    kw["B"] = min(kw["B"], 200)
    L = kw["gamma"]
    w = W.make("t", schedule=sched(L), seed=1600 + i, device=DEV, **kw)
    base = run_gpu(w, want_dbg=False, back_to_back=b2b)
    B, V, T = w.B, w.V, w.target_logits.shape[1]
    for pad in (64, 3):
        def embed(t, rows):
            if t is None:
                return None
            big = torch.zeros(B, rows * V + pad, dtype=t.dtype, device=DEV)
            big[:, :rows * V] = t.reshape(B, -1)
            return big
        bt, bd, btu, bdu = embed(w.target_logits, T), embed(w.draft_logits, L), embed(w.target_uncond, T), embed(w.draft_uncond, L)
        out_t = torch.full((B, L + 1), -7, dtype=torch.int32, device=DEV)
        out_l = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        out_s = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        ws = csd.new_workspace(B, L, V, w.dtype)   # (held: the parameter block keeps raw pointers)
        prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                              out_t, out_l, target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                              cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=out_s,
                              workspace=ws, back_to_back=b2b)
        prm.target_logits, prm.draft_logits = bt.data_ptr(), bd.data_ptr()
        if btu is not None:
            prm.target_uncond, prm.draft_uncond = btu.data_ptr(), bdu.data_ptr()
        prm.target_batch_stride, prm.draft_batch_stride = bt.shape[1], bd.shape[1]
        csd.csd_verify_ex(prm)
        torch.cuda.synchronize()
        assert np.array_equal(out_t.cpu().numpy(), base["tokens"]), (pad, kw)
        assert np.array_equal(out_l.cpu().numpy(), base["accept_len"]), (pad, kw)
        assert np.array_equal(out_s.cpu().numpy(), base["status"]), (pad, kw)


@pytest.mark.parametrize("kw", [dict(dtype=W.BF16, cfg=True, top_k=1000), dict(dtype=W.F32, top_k=500),
                                dict(dtype=W.BF16, top_k=700), dict(dtype=W.F32)])
@pytest.mark.parametrize("b2b", [False, True])
def test_nan_of_either_sign_marks_its_row(kw, b2b):
    """A NaN with the sign bit set (0xFFC0... is as much a NaN as 0x7FC0...) must reach the row's
    statistics like any other: the top-k gather tests values by the sign of a difference."""
    B, L, V = 6, 4, 16384
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=np.full(L, 1e6, np.float32), seed=11,
               device=DEV, **kw)
    neg_nan = torch.tensor([-1], dtype=torch.int32).view(torch.float32).item()   # all bits set: a negative NaN
    assert neg_nan != neg_nan
    def put(t, b, i, x):
        if t.dtype == torch.bfloat16:
            t.view(torch.int16)[b, i, x] = -64          # 0xFFC0
        else:
            t.view(torch.int32)[b, i, x] = -4194304     # 0xFFC00000
    put(w.target_logits, 0, 1, 5)                       # in the first stage (the sample of the guess)
    put(w.draft_logits, 1, 2, V - 3)                    # in the last stage
    put(w.target_logits, 2, 0, V // 2 + 1)
    if w.draft_uncond is not None:
        put(w.draft_uncond, 3, 1, 9000)
    rep, got, ref = check(w, back_to_back=b2b)
    assert_ok(rep)
    # (a drafted token outside the target's top-k rejects before the bad row is reached: the oracle says which)
    assert np.array_equal(got["status"], ref.status) and np.array_equal(got["accept_len"], ref.accept_len)
    assert got["status"][2] & 1 and got["accept_len"][2] == 0 and (ref.status[:4] & 1).sum() >= 2


def test_bad_data_is_reported_not_trapped():
    B, L, V = 5, 3, 64
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=np.full(L, 1e6, np.float32),
               seed=2, device=DEV)
    w.draft_logits[0, 1, 5] = float("nan")
    w.target_logits[1, 0, 7] = float("inf")
    w.draft_tokens[2, 2] = V
    w.draft_tokens[3, 0] = -1
    rep, got, ref = check(w)
    assert_ok(rep)
    assert got["accept_len"].tolist() == [1, 0, 2, 0, 3]
    assert got["status"].tolist() == [1, 1, 2, 2, 0]
    assert got["tokens"][1, 0] == -1
    # -inf entries are legal (masked tokens); a row of only -inf is not
    w2 = W.make("t", B=2, gamma=2, V=40, rho=0.9, schedule=sched(2), seed=3, device=DEV)
    w2.target_logits[0, 0, :20] = float("-inf")
    w2.draft_logits[0, 1, 3] = float("-inf")
    w2.target_logits[1, 0, :] = float("-inf")
    rep, got, ref = check(w2)
    assert_ok(rep)
    assert got["status"][1] == 1


@pytest.mark.parametrize("i", range(24))
def test_seeded_sweep_of_unusable_inputs(i):
    """NaN, +inf, masked (-inf) entries, fully masked rows and out-of-range draft tokens scattered over
    random shapes: reported in the status word and handled as the oracle handles them, on every kernel
    and partition (the first draft positions are made very likely to accept so later ones count)."""
    kw, b2b = _random_case(500 + i)
    kw["B"] = max(kw["B"], 4)
    B, L, V = kw["B"], kw["gamma"], kw["V"]
    r = np.random.default_rng(7000 + i)
    schedule = np.full(L, 50.0, np.float32) if i % 2 else sched(L)
    w = W.make("t", schedule=schedule, seed=900 + i, device=DEV, **kw)
    T = w.target_logits.shape[1]
    for _ in range(max(2, B // 4)):
        b, what = int(r.integers(B)), int(r.integers(6))
        if what == 0: w.draft_logits[b, int(r.integers(L)), int(r.integers(V))] = float("nan")
        elif what == 1: w.target_logits[b, int(r.integers(T)), int(r.integers(V))] = float("inf")
        elif what == 2: w.draft_tokens[b, int(r.integers(L))] = int(r.choice([-1, V, V + 7, 2 ** 30]))
        elif what == 3: w.target_logits[b, int(r.integers(T)), : int(r.integers(1, V))] = float("-inf")
        elif what == 4: w.draft_logits[b, int(r.integers(L)), int(r.integers(V)):] = float("-inf")
        else: w.target_logits[b, int(r.integers(T)), :] = float("-inf")
    rep, got, ref = check(w, back_to_back=b2b, want_dbg=B * V <= 4e6)
    # A forced rejection (out-of-range draft token) can land where both models put all but 1e-10 or less
    # of their mass on the same token, a position where a valid draft token is rejected with that
    # probability.  There the fp64 oracle runs out of digits (it forms P - Q f from probabilities next to
    # 1; pinned in tests/test_oracle_exact.py), so such a draw is adjudicated by the extended-precision
    # statement of Eq. opt_G instead: the kernel must have drawn ITS token.  Everything else about the
    # sequence, and every other sequence, must agree with the fp64 oracle as usual.
    differing = {b for b, _ in rep.unexplained} | set(np.flatnonzero(
        (got["status"] != ref.status) & (got["accept_len"] == ref.accept_len)).tolist())
    for b in sorted(differing):
        assert _adjudicated_by_extended_precision(w, got, ref, b), (b, rep.summary(), rep.unexplained[:3])
    assert len(differing) <= max(2, B // 25), rep.summary()
    other = run_gpu(w, want_dbg=False, back_to_back=not b2b)
    for key in ("tokens", "accept_len", "status"):
        assert np.array_equal(got[key], other[key]), (key, kw, b2b)
    # the per-position monitors: NaN exactly where a row is unusable, the oracle's values elsewhere
    mon = run_gpu(w, want_dbg=False, want_terms=True, back_to_back=b2b)
    assert np.array_equal(mon["tokens"], got["tokens"]) and np.array_equal(mon["status"], got["status"])
    _, ref_t = run_oracle(w, want_G=False, want_terms=True)
    usable = np.isfinite(ref_t.accept_mass)
    assert np.array_equal(np.isfinite(mon["accept_mass"]), usable) and np.array_equal(np.isfinite(mon["bound_term"]), usable)
    tol = 1e-5 if w.dtype == W.F32 else 2e-3
    if usable.any():
        assert np.abs(mon["accept_mass"][usable] - ref_t.accept_mass[usable]).max() < tol
        assert np.abs(mon["bound_term"][usable] - ref_t.bound_term[usable]).max() < 2 * tol * max(1.0, float(schedule.max()))
    # the drafting-stage draw on the same damaged rows (the drafter's first and the target's last)
    h = w.host_arrays()   # bf16 as bit patterns, like every oracle input
    for key_l, key_u, col, dev_l, dev_u in (("draft_logits", "draft_uncond", 0, w.draft_logits, w.draft_uncond),
                                            ("target_logits", "target_uncond", T - 1, w.target_logits, w.target_uncond)):
        tok = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        st = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        csd.csd_sample_rows(dev_l[:, col].contiguous(), w.uniforms[:, L].contiguous(), tok,
                            uncond=None if dev_u is None else dev_u[:, col].contiguous(), cfg_scale=w.cfg_scale,
                            top_k=w.top_k, out_status=st, back_to_back=b2b)
        torch.cuda.synchronize()
        ref_tok, ref_st, margin = oracle.sample_rows(
            h[key_l][:, col], h["uniforms"][:, L], dtype=w.dtype,
            uncond=None if h[key_u] is None else h[key_u][:, col], cfg_scale=w.cfg_scale, top_k=w.top_k)
        differ = tok.cpu().numpy() != ref_tok
        assert np.all(margin[differ] < 1e-6) and differ.sum() <= max(1, B // 50), (key_l, np.flatnonzero(differ)[:5])
        assert np.array_equal(st.cpu().numpy(), ref_st), key_l


def _adjudicated_by_extended_precision(w, got, ref, b):
    """Sequence b differs from the fp64 oracle.  True only if (i) it differs in nothing but the token
    drawn at its first rejection (and, at most, the Z-fallback status bit on either side), (ii) the fp64
    normaliser Z of Eq. opt_G at that position is below 1e-10, the regime the fp64 oracle does not
    resolve, and (iii) the kernel's token is the one the extended-precision statement of Eq. opt_G
    draws with the same uniform (or that draw lies within 1e-6 of a CDF boundary).  Where the exact Z is
    below what the kernel's fp32 weights can hold (1e-37) the kernel reports CSD_STATUS_ZFALLBACK and
    must then have drawn from the target distribution P_j, as documented."""
    from oracle import exact
    L = w.gamma
    if b < 0 or got["accept_len"][b] != ref.accept_len[b] or (got["status"][b] & ~4) != (ref.status[b] & ~4):
        return False
    j = int(ref.accept_len[b])
    if j >= L or not np.array_equal(got["tokens"][b, :j], ref.tokens[b, :j]):
        return False
    h = w.host_arrays()

    def prepared(key, key_u):
        un = None if h[key_u] is None else h[key_u][b, j]
        return oracle.prepare_row(h[key][b, j], un, w.dtype, w.cfg_scale, w.top_k)

    zt, zd = prepared("target_logits", "target_uncond"), prepared("draft_logits", "draft_uncond")
    P64, Q64 = oracle.softmax(zt), oracle.softmax(zd)
    if P64 is None:
        return False
    omega, u = float(h["relax_schedule"][j]), float(h["uniforms"][b, L])
    if Q64 is not None:
        _, Z64 = oracle.resample_weights(P64, Q64, omega)
        if not Z64 < 1e-10:
            return False          # the fp64 oracle resolves this draw: the mismatch stands
    res = exact.draw(zt, zd if Q64 is not None else None, omega, u)
    drawn = int(got["tokens"][b, j])
    if got["status"][b] & 4:      # the kernel's fp32 weights underflowed (or the positive part is empty)
        if not (res["fallback"] or res["Z"] < 1e-37):
            return False
        res = exact.draw(zt, None, omega, u)
    return drawn == res["token"] or float(res["margin"]) < 1e-6


@pytest.mark.parametrize("kw", [
    dict(B=6, gamma=3, V=4096, dtype=W.F32), dict(B=6, gamma=3, V=16384, dtype=W.BF16, cfg=True, top_k=500),
    dict(B=6, gamma=3, V=66, dtype=W.F32), dict(B=40, gamma=4, V=2048, dtype=W.BF16, bonus_row=True)])
@pytest.mark.parametrize("b2b", [False, True])
def test_resample_uniform_outside_the_open_interval(kw, b2b):
    """The draw's uniform is documented as lying in (0, 1).  A generator that can return 1.0, or a NaN,
    must still give the documented result -- no crossing C(x) > u Z exists, so the last token with
    positive weight -- and 0 gives the first such token; nothing may be read outside the rows.  The
    damaged sequences have index > 0.  Every position is made to reject (omega = 0) or to accept
    (a huge omega, so that the bonus draw is reached where there is a bonus row)."""
    L = kw["gamma"]
    for schedule in (np.zeros(L, np.float32), np.full(L, 1e9, np.float32)):
        w = W.make("t", rho=0.9, schedule=schedule, seed=77, device=DEV, **kw)
        B = w.B
        for b, u in ((1, 1.0), (2, float("nan")), (3, 0.0), (B - 1, 1.0), (4, 1.5)):
            w.uniforms[b, L] = u
        rep, got, ref = check(w, back_to_back=b2b, want_dbg=B * w.V <= 4e6)
        assert_ok(rep)
        for b in (1, 2, B - 1, 4):
            j = got["accept_len"][b]
            if got["tokens"][b, j] >= 0:
                assert got["tokens"][b, j] == ref.tokens[b, j]


@pytest.mark.parametrize("kw", [dict(B=20, gamma=4, V=8192, dtype=W.F32),
                                dict(B=20, gamma=4, V=16384, dtype=W.BF16, cfg=True, top_k=300)])
@pytest.mark.parametrize("b2b", [False, True])
def test_wait_that_runs_out_is_reported_not_hung(kw, b2b):
    """Every wait of a kernel on a copy into shared memory is bounded.  With the testing aid the first
    copy of block 0 is announced but never issued and the limit is about a millisecond: the call must
    return, set CSD_STATUS_TIMEOUT for the sequences of the block that gave up, keep the condition in
    the workspace (later calls on it report it for every sequence) until csd_workspace_init clears it,
    and leave the context usable."""
    L = kw["gamma"]
    w = W.make("t", rho=0.9, schedule=sched(L), seed=31, device=DEV, **kw)
    ws = csd.new_workspace(w.B, L, w.V, w.dtype)
    good = run_gpu(w, want_dbg=False, workspace=ws, back_to_back=b2b)
    assert np.all(good["status"] == 0)
    csd.csd_test_hooks(21, True)
    try:
        bad = run_gpu(w, want_dbg=False, workspace=ws, back_to_back=b2b)
    finally:
        csd.csd_test_hooks()
    assert bad["status"][0] & csd.CSD_STATUS_TIMEOUT
    assert np.all(bad["accept_len"] >= 0) and np.all(bad["accept_len"] <= L)
    sticky = run_gpu(w, want_dbg=False, workspace=ws, back_to_back=b2b)     # normal call, same workspace
    assert np.all(sticky["status"] & csd.CSD_STATUS_TIMEOUT)
    assert np.array_equal(sticky["tokens"], good["tokens"]) and np.array_equal(sticky["accept_len"], good["accept_len"])
    csd.csd_workspace_init(ws)
    clean = run_gpu(w, want_dbg=False, workspace=ws, back_to_back=b2b)
    for key in ("tokens", "accept_len", "status"):
        assert np.array_equal(clean[key], good[key]), key


def test_multiplier_that_is_negative_or_nan_counts_as_zero():
    """Eq. relax is stated for omega >= 0; a negative or NaN entry of the schedule is read as 0 on both
    sides: the position rejects (for q > 0) and the draw is from the target distribution."""
    L = 4
    schedule = np.array([50.0, float("nan"), -2.0, 1.0], np.float32)
    for kw in (dict(V=4096, dtype=W.F32), dict(V=66, dtype=W.F32), dict(V=8192, dtype=W.BF16, cfg=True, top_k=100)):
        w = W.make("t", B=12, gamma=L, rho=0.95, schedule=schedule, seed=12, device=DEV, **kw)
        rep, got, ref = check(w)
        assert_ok(rep)
        assert np.all(got["accept_len"] <= 1) and np.all(got["f"][:, 1:3] == 0.0)


@pytest.mark.parametrize("V,dtype", [(4096, W.F32), (16384, W.BF16), (66, W.F32)])
@pytest.mark.parametrize("b2b", [False, True])
def test_draw_where_both_models_peak_on_one_token(V, dtype, b2b):
    """Both models put all but exp(-gap) of their mass on the same token and the drafted token is out of
    range, which forces a rejection there: the normaliser Z of Eq. opt_G is of the order exp(-gap).  The
    fp64 oracle resolves this down to about 1e-10 only (tests/test_oracle_exact.py), so the drawn token
    is compared with the extended-precision statement of Eq. opt_G: identical for every gap the kernel's
    fp32 weights can hold; beyond (Z < 1e-37) the kernel must report CSD_STATUS_ZFALLBACK and draw from
    the target distribution."""
    from oracle import exact
    gaps = [12.0, 24.0, 30.0, 40.0, 52.0, 64.0, 76.0, 120.0]
    B, L = len(gaps), 2
    w = W.make("t", B=B, gamma=L, V=V, dtype=dtype, rho=0.5, schedule=np.array([1.0, 1.1], np.float32), seed=91,
               device=DEV)
    peak = 11
    for b, gap in enumerate(gaps):
        w.target_logits[b, :, peak] = w.target_logits[b].float().amax() + gap
        w.draft_logits[b, :, peak] = w.draft_logits[b].float().amax() + gap
    w.draft_tokens[:, 0] = V + 3          # forced rejection at the first position
    got = run_gpu(w, want_dbg=False, back_to_back=b2b)
    h = w.host_arrays()
    assert np.all(got["accept_len"] == 0) and np.all(got["status"] & 2)
    checked = 0
    for b, gap in enumerate(gaps):
        zt = oracle.prepare_row(h["target_logits"][b, 0], None, w.dtype, 1.0, 0)
        zd = oracle.prepare_row(h["draft_logits"][b, 0], None, w.dtype, 1.0, 0)
        res = exact.draw(zt, zd, 1.0, float(h["uniforms"][b, L]))
        tok = int(got["tokens"][b, 0])
        if got["status"][b] & 4:
            assert res["Z"] < 1e-37, (gap, res["Z"])
            res = exact.draw(zt, None, 1.0, float(h["uniforms"][b, L]))
        else:
            assert res["Z"] > 1e-39, (gap, res["Z"])
        if float(res["margin"]) >= 1e-6:
            assert tok == res["token"], (gap, tok, res["token"], float(res["Z"]))
            checked += 1
    assert checked >= B - 2
    assert got["status"][-1] & 4          # exp(-120) is below what fp32 weights hold


def test_identical_models_and_zero_omega():
    L = 3
    w = W.make("t", B=16, gamma=L, V=512, rho=1.0, schedule=np.array([1.0, 0.3, 0.0], np.float32),
               seed=6, device=DEV)
    w.draft_logits.copy_(w.target_logits[:, :L])
    rep, got, ref = check(w)
    assert_ok(rep)
    assert np.all(got["accept_len"] >= 1) and np.all(got["accept_len"] <= 2)


def test_simple_form_and_determinism():
    L, V, B = 8, 16384, 16
    w = W.config("C2", step=1, schedule=sched(L), device=DEV)
    out_t = torch.empty(B, L + 1, dtype=torch.int32, device=DEV)
    out_l = torch.empty(B, dtype=torch.int32, device=DEV)
    csd.csd_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                   out_t, out_l)
    torch.cuda.synchronize()
    got = run_gpu(w, want_dbg=False)
    assert np.array_equal(out_t.cpu().numpy(), got["tokens"])
    assert np.array_equal(out_l.cpu().numpy(), got["accept_len"])
    for _ in range(3):      # same inputs, same outputs
        again = run_gpu(w, want_dbg=False)
        assert np.array_equal(again["tokens"], got["tokens"])
    # a second, larger problem (the simple form keeps no state between calls)
    w2 = W.make("t", B=40, gamma=8, V=16384, rho=0.9, schedule=sched(8), seed=9, device=DEV)
    out_t2 = torch.empty(40, 9, dtype=torch.int32, device=DEV)
    out_l2 = torch.empty(40, dtype=torch.int32, device=DEV)
    csd.csd_verify(w2.target_logits, w2.draft_logits, w2.draft_tokens, w2.uniforms, w2.relax_schedule,
                   out_t2, out_l2)
    torch.cuda.synchronize()
    got2 = run_gpu(w2, want_dbg=False)
    assert np.array_equal(out_t2.cpu().numpy(), got2["tokens"])
    # rows the single-launch path cannot take need a workspace, which this form does not have
    w3 = W.make("t", B=3, gamma=2, V=66, rho=0.9, schedule=sched(2), seed=10, device=DEV)
    with pytest.raises(csd.CsdError) as err:
        csd.csd_verify(w3.target_logits, w3.draft_logits, w3.draft_tokens, w3.uniforms, w3.relax_schedule,
                       torch.empty(3, 3, dtype=torch.int32, device=DEV), torch.empty(3, dtype=torch.int32, device=DEV))
    assert err.value.code == -7


def test_host_buffer_form():
    L, V, B = 4, 4096, 8
    w = W.make("t", B=B, gamma=L, V=V, dtype=W.BF16, rho=0.9, bonus_row=True, schedule=sched(L), seed=4,
               device=DEV)
    got = run_gpu(w, want_dbg=False)
    pin = lambda t: t.cpu().pin_memory()
    h = dict(t=pin(w.target_logits), d=pin(w.draft_logits), tok=pin(w.draft_tokens), u=pin(w.uniforms),
             s=pin(w.relax_schedule))
    out_t = torch.empty(B, L + 1, dtype=torch.int32).pin_memory()
    out_l = torch.empty(B, dtype=torch.int32).pin_memory()
    out_s = torch.empty(B, dtype=torch.int32).pin_memory()
    prm = csd.make_params(h["t"], h["d"], h["tok"], h["u"], h["s"], out_t, out_l, out_status=out_s, host=True)
    n = csd.csd_host_staging_size(prm)
    assert n > w.logits_bytes()
    staging = torch.empty(n, dtype=torch.uint8, device=DEV)
    csd.csd_verify_host(prm, staging)
    torch.cuda.synchronize()
    assert np.array_equal(out_t.numpy(), got["tokens"])
    assert np.array_equal(out_l.numpy(), got["accept_len"])
    assert np.array_equal(out_s.numpy(), got["status"])


@pytest.mark.parametrize("i", range(10))
def test_seeded_sweep_of_host_form_and_static_scratch(i):
    """The entry points that wrap the device call -- host buffers with copies enqueued by the library,
    and (fp32, plain inputs) the form whose scratch is a fixed array inside the library -- on random
    shapes: the same integers as csd_verify_ex on device buffers."""
    kw, _ = _random_case(800 + i)
    kw["B"] = min(kw["B"], 300)
    L = kw["gamma"]
    w = W.make("t", schedule=sched(L), seed=1300 + i, device=DEV, **kw)
    got = run_gpu(w, want_dbg=False)
    pin = lambda t: None if t is None else t.cpu().pin_memory()
    out_t = torch.full((w.B, L + 1), -7, dtype=torch.int32).pin_memory()
    out_l = torch.full((w.B,), -7, dtype=torch.int32).pin_memory()
    out_s = torch.full((w.B,), -7, dtype=torch.int32).pin_memory()
    prm = csd.make_params(pin(w.target_logits), pin(w.draft_logits), pin(w.draft_tokens), pin(w.uniforms),
                          pin(w.relax_schedule), out_t, out_l, target_uncond=pin(w.target_uncond),
                          draft_uncond=pin(w.draft_uncond), cfg_scale=w.cfg_scale, top_k=w.top_k,
                          out_status=out_s, host=True)
    staging = torch.empty(csd.csd_host_staging_size(prm), dtype=torch.uint8, device=DEV)
    csd.csd_verify_host(prm, staging)
    torch.cuda.synchronize()
    assert np.array_equal(out_t.numpy(), got["tokens"])
    assert np.array_equal(out_l.numpy(), got["accept_len"])
    assert np.array_equal(out_s.numpy(), got["status"])
    plain = w.dtype == W.F32 and w.target_uncond is None and not w.top_k and w.target_logits.shape[1] == L
    if plain and csd.csd_workspace_size(w.B, L, w.V, W.F32) <= csd.CSD_STATIC_SCRATCH_BYTES:
        tok = torch.full((w.B, L + 1), -9, dtype=torch.int32, device=DEV)
        tau = torch.full((w.B,), -9, dtype=torch.int32, device=DEV)
        csd.csd_verify_static(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule, tok, tau)
        torch.cuda.synchronize()
        assert np.array_equal(tok.cpu().numpy(), got["tokens"]) and np.array_equal(tau.cpu().numpy(), got["accept_len"])


def test_argument_errors():
    w = W.make("t", B=2, gamma=2, V=64, schedule=sched(2), device=DEV)
    out_t = torch.empty(2, 3, dtype=torch.int32, device=DEV)
    out_l = torch.empty(2, dtype=torch.int32, device=DEV)
    ws = csd.new_workspace(2, 2, 64, 0)
    prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                          out_t, out_l, workspace=ws)
    lib = csd.library()
    import ctypes as C
    bad = csd.csd_params.from_buffer_copy(prm); bad.workspace_bytes = 16
    assert lib.csd_verify_ex(C.byref(bad)) == -4
    bad = csd.csd_params.from_buffer_copy(prm); bad.gamma = 33
    assert lib.csd_verify_ex(C.byref(bad)) == -2
    bad = csd.csd_params.from_buffer_copy(prm); bad.dtype = 5
    assert lib.csd_verify_ex(C.byref(bad)) == -3
    bad = csd.csd_params.from_buffer_copy(prm); bad.out_tokens = None
    assert lib.csd_verify_ex(C.byref(bad)) == -1
    bad = csd.csd_params.from_buffer_copy(prm); bad.target_uncond = prm.target_logits
    assert lib.csd_verify_ex(C.byref(bad)) == -5
    assert lib.csd_verify_ex(None) == -1
