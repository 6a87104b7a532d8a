"""GPU parity of the tree-structured verification (csd_verify_tree) against the oracle's orc_verify_tree
on the same seeded inputs and uniforms: accepted paths, emitted tokens and status identical except for
decisions the oracle flags as within 1e-6 of a threshold (counted), the distribution drawn from within
1e-5 (fp32 logits) / 2e-3 (bf16 logits) absolute."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import oracle
import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W

DEV = "cuda"
TOL = {W.F32: 1e-5, W.BF16: 2e-3}


def run_tree_gpu(w, want_G=True):
    D = csd.csd_tree_depth(w.parent)
    out = dict(tokens=torch.full((w.B, D + 1), -7, dtype=torch.int32, device=DEV),
               accept_len=torch.full((w.B,), -7, dtype=torch.int32, device=DEV),
               nodes=torch.full((w.B, D), -7, dtype=torch.int32, device=DEV),
               status=torch.full((w.B,), -7, dtype=torch.int32, device=DEV))
    if want_G:
        out["G"] = torch.full((w.B, w.V), -1.0, device=DEV)
    csd.csd_verify_tree(w.target_logits, w.draft_logits, w.parent, w.draft_tokens, w.uniforms, w.relax_schedule,
                        out["tokens"], out["accept_len"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                        cfg_scale=w.cfg_scale, top_k=w.top_k, out_nodes=out["nodes"], out_status=out["status"],
                        dbg_G=out.get("G"))
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def run_tree_oracle(w):
    h = w.host_arrays()
    return oracle.verify_tree(h["target_logits"], h["draft_logits"], h["parent"], h["draft_tokens"], h["uniforms"],
                              h["relax_schedule"], dtype=w.dtype, target_uncond=h["target_uncond"],
                              draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k)


def compare_tree(w, got, ref, near=1e-6):
    """Returns (near-threshold mismatches, list of unexplained differences)."""
    n_near, bad = 0, []
    for b in range(w.B):
        lo, lg = int(ref.accept_len[b]), int(got["accept_len"][b])
        same_path = lo == lg and np.array_equal(ref.nodes[b], got["nodes"][b])
        if not same_path:
            tested = np.isfinite(ref.margin_accept[b])
            if tested.any() and ref.margin_accept[b][tested].min() < near:
                n_near += 1
            else:
                bad.append((b, f"path {got['nodes'][b].tolist()} vs oracle {ref.nodes[b].tolist()}"))
            continue
        if not np.array_equal(ref.tokens[b, :lo], got["tokens"][b, :lo]) or np.any(got["tokens"][b, lo + 1:] != -1):
            bad.append((b, "accepted tokens or padding differ"))
        if int(ref.status[b]) != int(got["status"][b]):
            bad.append((b, f"status {got['status'][b]} vs oracle {ref.status[b]}"))
        if "G" in got:
            err = np.abs(got["G"][b].astype(np.float64) - ref.G[b]).max()
            if err > TOL[w.dtype]:
                bad.append((b, f"G max abs error {err:.2e}"))
        if int(ref.tokens[b, lo]) != int(got["tokens"][b, lo]):
            if ref.margin_cdf[b] < near:
                n_near += 1
            else:
                bad.append((b, f"token {got['tokens'][b, lo]} vs oracle {ref.tokens[b, lo]}, margin {ref.margin_cdf[b]:.2e}"))
    return n_near, bad


TREES = {
    "chain5": np.arange(-1, 4),
    "static_4_3_2_2": W.static_tree([4, 3, 2, 2]),
    "wide_root": W.static_tree([8, 1]),
    "bushy": np.array([-1, -1, -1, 0, 0, 1, 1, 2, 3, 3, 5, 5, 5, 8, 10], dtype=np.int32),
}


@pytest.mark.parametrize("tree", sorted(TREES))
@pytest.mark.parametrize("kw", [dict(V=4096, dtype=W.F32), dict(V=16384, dtype=W.BF16),
                                dict(V=1000, dtype=W.F32, top_k=100), dict(V=8192, dtype=W.BF16, cfg=True, top_k=300),
                                dict(V=66, dtype=W.F32), dict(V=4100, dtype=W.BF16)])
def test_tree_parity(tree, kw):
    parent = TREES[tree]
    D = oracle.tree_depth(parent)
    for sched in (np.ones(D, np.float32), csd.csd_make_schedule(1, 1.6, 0.5, D)):
        w = W.make_tree(parent, B=24, rho=0.9, schedule=sched, seed=len(parent) + kw["V"], device=DEV, **kw)
        got, ref = run_tree_gpu(w), run_tree_oracle(w)
        n_near, bad = compare_tree(w, got, ref)
        assert not bad, bad[:4]
        assert n_near <= 2
        assert got["accept_len"].max() >= 1 and got["accept_len"].min() <= D
        for b in range(w.B):                     # the accepted path is a path of the tree carrying the drafted tokens
            prev = -1
            for lvl in range(got["accept_len"][b]):
                n = got["nodes"][b, lvl]
                assert parent[n] == prev and got["tokens"][b, lvl] == w.draft_tokens[b, n].item()
                prev = n


def test_chain_shaped_tree_equals_the_chain_entry_point():
    """A chain is Algorithm 1: the tree entry point must emit what csd_verify_ex emits."""
    L, V, B = 6, 8192, 32
    sched = csd.csd_make_schedule(1, 1.1, 0.7, L)
    w = W.make_tree(np.arange(-1, L - 1), B=B, V=V, rho=0.9, schedule=sched, seed=5, device=DEV)
    got = run_tree_gpu(w, want_G=False)
    out_t = torch.empty(B, L + 1, dtype=torch.int32, device=DEV)
    out_l = torch.empty(B, dtype=torch.int32, device=DEV)
    ws, chain_draft = csd.new_workspace(B, L, V, w.dtype), w.draft_logits[:, :L].contiguous()
    prm = csd.make_params(w.target_logits, chain_draft, w.draft_tokens, w.uniforms, w.relax_schedule,
                          out_t, out_l, workspace=ws)
    csd.csd_verify_ex(prm)
    torch.cuda.synchronize()
    assert np.array_equal(out_l.cpu().numpy(), got["accept_len"])
    assert np.array_equal(out_t.cpu().numpy(), got["tokens"])


def test_tree_bad_data_and_forced_rejections():
    parent = TREES["bushy"]
    D = oracle.tree_depth(parent)
    w = W.make_tree(parent, B=12, V=2048, rho=0.95, schedule=np.full(D, 30.0, np.float32), seed=9, device=DEV)
    w.target_logits[1, 0, 17] = float("nan")
    w.draft_logits[2, 0, 5] = float("inf")
    w.draft_tokens[3, 0] = -1
    w.draft_tokens[4, :3] = w.V + 2               # every candidate of the root unusable: three passes, then the draw
    w.target_logits[5, 1, :] = float("-inf")      # the context after node 0 has no usable target row
    w.uniforms[6, len(parent)] = 1.0              # a draw with no crossing
    got, ref = run_tree_gpu(w), run_tree_oracle(w)
    n_near, bad = compare_tree(w, got, ref)
    assert not bad, bad[:4]
    assert got["status"][1] & 1 and got["tokens"][1, 0] == -1 and got["accept_len"][1] == 0
    assert got["status"][4] & 2 and got["accept_len"][4] == 0 and got["tokens"][4, 0] >= 0


def test_tree_argument_errors():
    lib = csd.library()
    import ctypes as C
    bad = np.array([0, -1], np.int32)
    assert lib.csd_tree_depth(bad.ctypes.data_as(C.c_void_p), 2) == -5      # a parent must be an earlier node
    many = np.full(9, -1, np.int32)
    assert lib.csd_tree_depth(many.ctypes.data_as(C.c_void_p), 9) == -2     # more than 8 candidates of one node
    assert lib.csd_verify_tree(None) == -1
    assert csd.csd_tree_workspace_size(4, 64, 1000, 0) == 0 and csd.csd_tree_workspace_size(4, 63, 1000, 0) > 0


@pytest.mark.parametrize("i", range(24))
def test_seeded_sweep_of_random_trees(i):
    """Random trees (up to 39 nodes, up to 8 candidates per node, any depth the limits allow), vocabularies
    with and without a ragged tail, both dtypes, guidance mix, top-k below and above the small candidate
    lists, heavy-tailed logits, batch sizes 1 - 40, multipliers on both sides of 1."""
    r = np.random.default_rng(50000 + i)
    N = int(r.integers(1, 40))
    parent, kids, depth = [], {}, {}
    for n in range(N):
        while True:
            p = int(r.integers(-1, n))
            d = 0 if p < 0 else depth[p] + 1
            if kids.get(p, 0) < 8 and d < 31:
                break
        parent.append(p); kids[p] = kids.get(p, 0) + 1; depth[n] = d
    parent = np.array(parent, np.int32)
    D = oracle.tree_depth(parent)
    V = int(r.choice([66, 1000, 2048, 4100, 8192, 16384, 20000]))
    kw = dict(V=V, dtype=[W.F32, W.BF16][int(r.integers(2))])
    if r.integers(3) == 0:
        kw["cfg"] = True
    if r.integers(2) == 0:
        kw["top_k"] = int(min(V - 1, r.choice([5, 100, 1000, 1500])))
    if r.integers(5) == 0:
        kw["law"] = "student3"
    B = int(r.choice([1, 3, 17, 40]))
    sched = (np.exp(-0.3 * np.arange(D)) * r.choice([1.0, 1.5, 3.0])).astype(np.float32)
    w = W.make_tree(parent, B=B, rho=float(r.choice([0.7, 0.9, 0.99])), schedule=sched, seed=i, device=DEV, **kw)
    got, ref = run_tree_gpu(w, want_G=B * V <= 2e6), run_tree_oracle(w)
    n_near, bad = compare_tree(w, got, ref)
    assert not bad, (N, D, kw, B, bad[:3])
    assert n_near <= 2
