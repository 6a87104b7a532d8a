"""The benchmark's four fixed configurations at full size against the oracle: C1-C3 on 16 seeded steps
each (C2 at all three drafter correlations, with the vanilla and the default schedule), C4 on all 256
sequences of two steps, in both stream modes.  Prints per configuration the counts that the report quotes:
sequences, near-threshold accept tests and draws on the oracle's side, and mismatches (all of which must be
explained by such a near-threshold decision)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W
from gpu_util import check

DEV = "cuda"


def _sched(L, vanilla=False):
    return np.ones(L, np.float32) if vanilla else csd.csd_make_schedule(1, 1.1, 0.7, L)


def _run(name, steps, **over):
    L = W.CONFIGS[name]["gamma"]
    tot = dict(seq=0, near_accept=0, near_cdf=0, tau_near=0, tok_near=0, mean_emit=0.0)
    for step in range(steps):
        w = W.config(name, step=step, device=DEV, **over)
        rep, got, ref = check(w, want_dbg=False, back_to_back=bool(step & 1))
        assert rep.ok, (name, step, rep.summary(), rep.unexplained[:3])
        tot["seq"] += rep.n_seq
        tot["near_accept"] += rep.near_accept_tests
        tot["near_cdf"] += rep.near_cdf_draws
        tot["tau_near"] += rep.tau_mismatch_near
        tot["tok_near"] += rep.token_mismatch_near
        tot["mean_emit"] += float(got["accept_len"].mean() + 1) / steps
    print(f"CONFIG {name} {over.get('rho', '')} {'vanilla' if over.get('_vanilla') else ''}: {tot}")
    assert tot["tau_near"] + tot["tok_near"] <= max(2, tot["seq"] // 200)
    return tot


def test_c1_sixteen_steps():
    _run("C1", 16, schedule=_sched(4))


@pytest.mark.parametrize("rho", [0.7, 0.9, 0.97])
@pytest.mark.parametrize("vanilla", [True, False])
def test_c2_sixteen_steps(rho, vanilla):
    tot = _run("C2", 16, rho=rho, schedule=_sched(8, vanilla))
    assert tot["mean_emit"] > 1.0


def test_c3_sixteen_steps():
    _run("C3", 16, schedule=_sched(8))


def test_c4_all_sequences_of_two_steps():
    _run("C4", 2, schedule=_sched(16))


def test_widened_rounds_on_c3_shapes():
    """The tree and the similarity-relaxed rounds at the shapes bench.py times them on (C3: 64 sequences,
    V = 16384, bf16, guidance mix, top-k 1000): their row statistics come from the streaming kernels'
    stats-only mode there.  Every output against the oracle."""
    from oracle.compare import compare
    from gpu_util import run_oracle
    from test_gpu_similar import run_similar
    from test_gpu_tree import compare_tree, run_tree_gpu, run_tree_oracle
    kw = {k: v for k, v in W.CONFIGS["C3"].items() if k not in ("B", "gamma", "V", "bonus_row", "steps")}
    B, V = W.CONFIGS["C3"]["B"], W.CONFIGS["C3"]["V"]
    parent = W.static_tree([4, 3, 2, 2])
    D = csd.csd_tree_depth(parent)
    for step in range(2):
        wt = W.make_tree(parent, B=B, V=V, schedule=_sched(D), seed=21, step=step, device=DEV, **kw)
        n_near, bad = compare_tree(wt, run_tree_gpu(wt, want_G=False), run_tree_oracle(wt))
        assert not bad, bad[:4]
        assert n_near <= 2
        w = W.config("C3", step=step, schedule=_sched(8), device=DEV)
        r = np.random.default_rng(step)
        nbr = ((np.arange(V)[:, None] + 1 + r.integers(0, V - 1, size=(V, 10))) % V).astype(np.int32)
        got = run_similar(w, nbr, 2.0)
        h, ref = run_oracle(w, neighbours=nbr, nbr_lambda=2.0)
        rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"],
                      p=got["p"], q=got["q"], f=got["f"], tol=2e-3)
        assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
        assert rep.tau_mismatch_near + rep.token_mismatch_near <= 2, rep.summary()
