"""GPU parity of the similarity-relaxed round (csd_verify_similar: LANTERN++'s acceptance with the paper's
G*) against the oracle on the same seeded inputs, uniforms and a synthetic neighbour table (the paper's
tables come from the image tokenizer's codebook, which is absent: random distinct neighbours stand in)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import oracle
from oracle.compare import compare
import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W
from gpu_util import TOL, run_gpu, run_oracle

DEV = "cuda"


def neighbour_table(V, k, seed):
    r = np.random.default_rng(seed)
    nb = (np.arange(V)[:, None] + 1 + r.integers(0, V - 1, size=(V, k))) % V      # never the token itself
    nb[r.random((V, k)) < 0.05] = -1                                              # some empty slots
    return nb.astype(np.int32)


def run_similar(w, nbr, lam):
    B, L, V = w.B, w.gamma, w.V
    out = dict(tokens=torch.full((B, L + 1), -7, dtype=torch.int32, device=DEV),
               accept_len=torch.full((B,), -7, dtype=torch.int32, device=DEV),
               status=torch.full((B,), -7, dtype=torch.int32, device=DEV),
               p=torch.empty((B, L), device=DEV), q=torch.empty((B, L), device=DEV), f=torch.empty((B, L), device=DEV),
               G=torch.full((B, V), -1.0, device=DEV))
    ws = csd.new_workspace(B, L, V, w.dtype)  # (the parameter block holds raw pointers: both buffers are kept
    table = torch.from_numpy(nbr).to(DEV)     #  alive until the stream has been synchronised)
    prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                          out["tokens"], out["accept_len"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                          cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=out["status"], dbg_p=out["p"], dbg_q=out["q"],
                          dbg_f=out["f"], dbg_G=out["G"], workspace=ws)
    csd.csd_verify_similar(prm, table, lam)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.parametrize("kw", [dict(V=4096, dtype=W.F32), dict(V=16384, dtype=W.BF16, bonus_row=True),
                                dict(V=2000, dtype=W.F32, top_k=200), dict(V=8192, dtype=W.BF16, cfg=True, top_k=500),
                                dict(V=66, dtype=W.F32, bonus_row=True)])
@pytest.mark.parametrize("k,lam", [(10, 2.0), (3, 0.5), (16, 8.0)])
def test_similar_parity(kw, k, lam):
    L = 5
    # multipliers on both sides of 1: below it the aggregated mass enters the resampling weights too
    for sched in (np.array([1.0, 1.2, 0.8, 0.5, 0.3], np.float32), np.ones(L, np.float32)):
        w = W.make("t", B=20, gamma=L, rho=0.85, schedule=sched, seed=k + kw["V"], device=DEV, **kw)
        nbr = neighbour_table(w.V, k, seed=k)
        got = run_similar(w, nbr, lam)
        h, ref = run_oracle(w, neighbours=nbr, nbr_lambda=lam)
        rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"],
                      p=got["p"], q=got["q"], f=got["f"], G=got["G"], tol=TOL[w.dtype])
        assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
        assert rep.tau_mismatch_near + rep.token_mismatch_near <= 2, rep.summary()
        plain = run_gpu(w)
        assert np.all(got["f"] >= plain["f"] - TOL[w.dtype])       # never below the plain acceptance


def test_similar_without_selection_equals_plain_round():
    L = 4
    w = W.make("t", B=16, gamma=L, V=4096, rho=0.9, schedule=csd.csd_make_schedule(1, 1.1, 0.7, L), seed=3, device=DEV)
    plain = run_gpu(w)
    for nbr, lam in ((neighbour_table(w.V, 6, 1), 0.0), (np.full((w.V, 4), -1, np.int32), 5.0)):
        got = run_similar(w, nbr, lam)
        for key in ("tokens", "accept_len", "status"):
            assert np.array_equal(got[key], plain[key]), key
        assert np.abs(got["f"] - plain["f"]).max() < 1e-6


def test_similar_argument_errors():
    w = W.make("t", B=2, gamma=2, V=256, schedule=np.ones(2, np.float32), device=DEV)
    out_t = torch.empty(2, 3, dtype=torch.int32, device=DEV)
    out_l = torch.empty(2, dtype=torch.int32, device=DEV)
    ws = csd.new_workspace(2, 2, 256, 0)
    prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule, out_t, out_l,
                          workspace=ws)
    nbr = torch.zeros(256, 4, dtype=torch.int32, device=DEV)
    lib = csd.library()
    import ctypes as C
    assert lib.csd_verify_similar(C.byref(prm), None, 4, 1.0) == -1
    assert lib.csd_verify_similar(C.byref(prm), nbr.data_ptr(), 0, 1.0) == -5
    assert lib.csd_verify_similar(C.byref(prm), nbr.data_ptr(), 4, -1.0) == -5
    assert lib.csd_verify_similar(C.byref(prm), nbr.data_ptr(), 4, float("nan")) == -5
