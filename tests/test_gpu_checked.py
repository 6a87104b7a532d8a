"""The small cases once more through the bounds-checked build of the library (-DCSD_CHECKED): every
access of a logit row whose index comes from a drafted token, a neighbour id or the row length is
tested against the row's length before it happens.  The record must stay empty -- also for rows with
tokens out of range, ragged vocabularies and uniforms at the ends of [0, 1] -- and the results must
still be the oracle's."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from oracle.compare import compare
import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W
from gpu_util import check, run_gpu, run_oracle
from test_gpu_sharded import run_sharded
from test_gpu_similar import neighbour_table, run_similar
from test_gpu_tree import TREES, compare_tree, run_tree_gpu, run_tree_oracle

DEV = "cuda"


@pytest.fixture()
def checked():
    with csd.checked_library() as report:
        before = report()[0]
        yield lambda: (report()[0] - before,) + report()[1:]


def clean(checked):
    rec = checked()
    assert rec[0] == 0, f"bad index {rec[1]} against row length {rec[2]} at site {rec[3]} ({rec[0]} in all)"


def test_it_is_the_checked_build(checked):
    assert csd.library().csd_checked_report(None) == -1
    clean(checked)
    with csd.checked_library():                 # nests, and gives the normal build back afterwards
        pass
    rec = np.zeros(4, np.int32)
    assert csd.library().csd_checked_report(rec.ctypes.data) == 1


def test_normal_build_reports_zero():
    rec = np.full(4, 9, np.int32)
    assert csd.library().csd_checked_report(rec.ctypes.data) == 0 and not rec.any()


@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("V", [2, 8, 33, 1000, 1024, 4100, 16384])
def test_shapes(checked, dtype, V):
    L = 4
    for b2b in (False, True):
        for kw in (dict(), dict(top_k=max(1, V // 7)), dict(cfg=True, bonus_row=True)):
            w = W.make("t", B=6, gamma=L, V=V, dtype=dtype, rho=0.8, schedule=csd.csd_make_schedule(1, 1.2, 0.6, L),
                       seed=V, device=DEV, **kw)
            rep, got, ref = check(w, back_to_back=b2b)
            assert rep.ok, rep.summary()
    clean(checked)


@pytest.mark.parametrize("V,top_k", [(66, 0), (4100, 0), (20000, 300), (152064, 1000)])
def test_bad_tokens_edge_uniforms_and_unusable_rows(checked, V, top_k):
    L, B = 5, 12
    for dtype in (W.F32, W.BF16):
        w = W.make("t", B=B, gamma=L, V=V, dtype=dtype, rho=0.9, top_k=top_k, bonus_row=True,
                   schedule=np.full(L, 1.5, np.float32), seed=V + 1, device=DEV)
        w.draft_tokens[0, 0] = V
        w.draft_tokens[1, 2] = -1
        w.draft_tokens[2, 1] = 2 ** 31 - 1
        w.draft_tokens[3, 4] = -(2 ** 31)
        w.draft_tokens[4, 0] = V - 1
        w.uniforms[5, :] = 1.0
        w.uniforms[6, :] = 0.0
        w.target_logits[7, 1, V // 2] = float("nan")
        w.draft_logits[8, 0, :] = float("-inf")
        for b2b in (False, True):
            rep, got, ref = check(w, back_to_back=b2b)
            assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
    clean(checked)


def test_simple_forms_and_host_form(checked):
    L, B, V = 4, 8, 4100
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, schedule=np.ones(L, np.float32), seed=3, device=DEV)
    ref = run_gpu(w, want_dbg=False)
    for fn in (csd.csd_verify, csd.csd_verify_static):
        tok = torch.full((B, L + 1), -7, dtype=torch.int32, device=DEV)
        ln = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        fn(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule, tok, ln)
        torch.cuda.synchronize()
        assert np.array_equal(tok.cpu().numpy(), ref["tokens"]) and np.array_equal(ln.cpu().numpy(), ref["accept_len"])
    clean(checked)


@pytest.mark.parametrize("kw", [dict(V=4096, dtype=W.F32), dict(V=2000, dtype=W.BF16, top_k=150), dict(V=66, dtype=W.F32)])
def test_similarity_relaxed_round(checked, kw):
    L = 4
    w = W.make("t", B=10, gamma=L, rho=0.85, schedule=np.array([1.0, 0.8, 0.5, 1.3], np.float32), seed=5, device=DEV, **kw)
    w.draft_tokens[1, 1] = w.V + 3
    nbr = neighbour_table(w.V, 6, seed=1)
    nbr[5, 2], nbr[7, 0] = w.V, -5                     # ids outside the vocabulary are skipped, not read
    got = run_similar(w, nbr, 2.0)
    h, ref = run_oracle(w, neighbours=nbr, nbr_lambda=2.0)
    rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"],
                  tol=1e-5 if w.dtype == W.F32 else 2e-3)
    assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
    clean(checked)


@pytest.mark.parametrize("tree", ["static_4_3_2_2", "bushy"])
def test_tree_round(checked, tree):
    parent = TREES[tree]
    for kw in (dict(V=1000, dtype=W.F32, top_k=100), dict(V=4100, dtype=W.BF16)):
        w = W.make_tree(parent, B=10, rho=0.9, schedule=np.full(8, 1.2, np.float32)[:csd.csd_tree_depth(parent)],
                        seed=7, device=DEV, **kw)
        w.draft_tokens[0, 0] = w.V
        w.draft_tokens[1, :] = -1
        w.uniforms[2, :] = 1.0
        got, ref = run_tree_gpu(w), run_tree_oracle(w)
        n_near, bad = compare_tree(w, got, ref)
        assert not bad, bad[:4]
    clean(checked)


@pytest.mark.parametrize("n", [1, 3])
def test_vocabulary_sharded_round(checked, n):
    L, V = 4, 4100
    w = W.make("t", B=10, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=np.ones(L, np.float32), seed=9, device=DEV)
    w.draft_tokens[0, 1] = V
    w.draft_tokens[1, 0] = -1
    w.uniforms[2, :] = 1.0
    bounds = [0, V] if n == 1 else [0, 1367, 1368, V]
    got = run_sharded(w, bounds)
    h, ref = run_oracle(w)
    rep = compare(ref, got["tokens"], got["accept_len"], h["draft_tokens"], h["uniforms"], status=got["status"], tol=1e-5)
    assert rep.ok, rep.summary() + " :: " + str(rep.unexplained[:4])
    clean(checked)
