"""GPU parity of the vocabulary-sharded round against the oracle on the unsharded rows.  This run has one
GPU, so the n ranks are emulated by ONE process that holds all n slices and runs each of the four library
calls for every slice in turn, the all-gathers being a torch.stack in rank order; no kernel waits for
another.  (The exchange wiring over torch.distributed is covered by tests/test_sharded_vocab_gloo.py.)"""
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
from paper_2601_09212_b200.vocab_sharded import ShardedRound
from gpu_util import TOL, run_gpu, run_oracle

DEV = "cuda"


def run_sharded(w, bounds):
    """bounds: slice boundaries [0, ..., V] in vocabulary order."""
    n = len(bounds) - 1
    B, L = w.B, w.gamma
    cut = lambda t, r: None if t is None else t[:, :, bounds[r]:bounds[r + 1]].contiguous()
    rounds = [ShardedRound(cut(w.target_logits, r), cut(w.draft_logits, r), w.draft_tokens, w.uniforms, w.relax_schedule,
                           v_offset=bounds[r], V_total=w.V, shard=r, n_shards=n, target_uncond=cut(w.target_uncond, r),
                           draft_uncond=cut(w.draft_uncond, r), cfg_scale=w.cfg_scale) for r in range(n)]
    dbg = dict(p=torch.empty(B, L, device=DEV), q=torch.empty(B, L, device=DEV), f=torch.empty(B, L, device=DEV))
    records_all = torch.stack([rd.stats() for rd in rounds]).contiguous()
    totals_all = torch.stack([rd.partial(records_all, dbg["p"], dbg["q"], dbg["f"]) for rd in rounds]).contiguous()
    cand_all = torch.stack([rd.pick(totals_all) for rd in rounds]).contiguous()
    outs = []
    for rd in rounds:
        o = dict(tokens=torch.full((B, L + 1), -7, dtype=torch.int32, device=DEV),
                 accept_len=torch.full((B,), -7, dtype=torch.int32, device=DEV),
                 status=torch.full((B,), -7, dtype=torch.int32, device=DEV))
        rd.emit(cand_all, o["tokens"], o["accept_len"], o["status"])
        outs.append(o)
    torch.cuda.synchronize()
    res = [{k: v.cpu().numpy() for k, v in o.items()} for o in outs]
    for r in range(1, n):                       # every rank emits the same
        for k in ("tokens", "accept_len", "status"):
            assert np.array_equal(res[r][k], res[0][k]), (k, r)
    res[0].update({k: v.cpu().numpy() for k, v in dbg.items()})
    return res[0]


@pytest.mark.parametrize("kw", [dict(V=16384, dtype=W.F32), dict(V=16384, dtype=W.BF16, bonus_row=True),
                                dict(V=8192, dtype=W.BF16, cfg=True), dict(V=4100, dtype=W.F32, bonus_row=True),
                                dict(V=1000, dtype=W.BF16)])
@pytest.mark.parametrize("n", [1, 2, 4, 8])
def test_sharded_parity(kw, n):
    L, V = 6, kw["V"]
    w = W.make("t", B=24, gamma=L, rho=0.9, schedule=csd.csd_make_schedule(1, 1.3, 0.5, L), seed=n + V, device=DEV, **kw)
    r = np.random.default_rng(n)
    even = [V * k // n for k in range(n + 1)]
    ragged = [0] + sorted(r.choice(np.arange(1, V), size=n - 1, replace=False).tolist()) + [V]
    for bounds in (even, ragged):
        got = run_sharded(w, bounds)
        h, ref = run_oracle(w, want_G=True)
        rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"],
                      p=got["p"], q=got["q"], f=got["f"], tol=TOL[w.dtype])
        assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
        assert rep.tau_mismatch_near + rep.token_mismatch_near <= 2, rep.summary()
    one = run_gpu(w, want_dbg=False)            # and the unsharded kernels agree with the sharded ones
    same = (one["tokens"] == got["tokens"]).all(axis=1)
    assert same.sum() >= w.B - 1


def test_sharded_bad_data_fallback_and_edge_uniforms():
    L, V, n = 4, 4096, 4
    w = W.make("t", B=12, gamma=L, V=V, rho=1.0, bonus_row=True, schedule=np.full(L, 1.0, np.float32), seed=3, device=DEV)
    w.draft_logits[:, :, :] = w.target_logits[:, :L, :]      # identical models: an empty positive part on a rejection
    w.draft_tokens[0, 0] = V + 1                              # forced rejection there: falls back to P_j (status 2 | 4)
    w.draft_tokens[1, 2] = -5
    w.target_logits[2, 1, 100] = float("nan")
    w.draft_logits[3, 0, 3000] = float("inf")
    w.target_logits[4, 0, :] = float("-inf")
    w.uniforms[5, L] = 1.0                                    # no crossing: the last token with weight (in the last slice)
    w.uniforms[6, L] = 0.0
    got = run_sharded(w, [0, 1000, 2048, 3000, V])
    h, ref = run_oracle(w, want_G=True)
    rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"], tol=1e-5)
    assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
    assert got["status"][0] == 6 and got["status"][2] & 1 and got["tokens"][4, 0] == -1
