"""csd_verify_static: the entry point for callers that cannot allocate device memory.

A caller inside a stream capture, under an allocator that owns the whole GPU, or on a thread
that must never hit cudaMalloc's implicit synchronisation, uses csd_verify_static; its scratch
is a fixed array inside the library.  The check here: called through the C ABI twice in a row
(a larger problem, then a smaller one, so the second call runs over whatever the first left in
the shared scratch), it must give exactly the accepted lengths and tokens of csd_verify, the
simple entry point that takes the same arguments, and of the fp64 oracle on the same inputs (up
to decisions the oracle flags as within 1e-6 of a threshold).  These are integer outputs, so the
comparison is exact.  The file name makes pytest collect it last.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import paper_2601_09212_b200 as csd
from paper_2601_09212_b200 import workloads as W
from gpu_util import run_oracle
from oracle.compare import compare

DEV = "cuda"


def _both(w):
    B, L = w.B, w.gamma
    res = []
    for fn in (csd.csd_verify_static, csd.csd_verify):
        tok = torch.full((B, L + 1), -9, dtype=torch.int32, device=DEV)
        tau = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        fn(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule, tok, tau)
        torch.cuda.synchronize()
        res.append((tok.cpu().numpy(), tau.cpu().numpy()))
    return res


def test_static_scratch_matches_allocating_entry_point_twice_in_a_row():
    first = W.make("t", B=24, gamma=8, V=16384, rho=0.9, schedule=csd.csd_make_schedule(1, 1.1, 0.7, 8),
                   seed=21, device=DEV)
    second = W.make("t", B=5, gamma=3, V=1000, rho=0.8, schedule=csd.csd_make_schedule(0, 1.5, 0.0, 3),
                    seed=22, device=DEV)
    for w in (first, second):
        (tok_s, tau_s), (tok_a, tau_a) = _both(w)
        assert np.array_equal(tau_s, tau_a)
        assert np.array_equal(tok_s, tok_a)
        assert tau_s.min() >= 0 and tau_s.max() <= w.gamma
        assert (tok_s[np.arange(w.B), tau_s] >= 0).sum() > 0 or (tau_s == w.gamma).all()
        h, ref = run_oracle(w, want_G=True)
        rep = compare(ref, tok_s, tau_s, h["draft_tokens"], h["uniforms"])
        assert rep.ok and rep.tau_mismatch_near + rep.token_mismatch_near <= 1, rep.summary()


def test_static_scratch_refuses_what_does_not_fit():
    B, L, V = 256, 16, 65536
    assert csd.csd_workspace_size(B, L, V, csd.CSD_F32) > csd.CSD_STATIC_SCRATCH_BYTES
    lib = csd.library()
    # refused on the host before any pointer is looked at or anything is enqueued
    assert lib.csd_verify_static(None, None, None, None, None, B, L, V, None, None, None) == -8
    assert "csd_verify_static" in csd.error_string(-8)
