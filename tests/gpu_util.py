"""Helpers for the GPU parity tests: run a Workload through the C ABI and through the oracle."""
import numpy as np
import torch

import oracle
from oracle.compare import compare
import paper_2601_09212_b200 as csd

TOL = {csd.CSD_F32: 1e-5, csd.CSD_BF16: 2e-3}   # absolute, on p, q, f and on the distribution drawn from


def run_gpu(w, *, want_dbg=True, stream=None, workspace=None, back_to_back=False, want_terms=False):
    dev = w.target_logits.device
    B, L, V = w.B, w.gamma, w.V
    out = dict(
        tokens=torch.full((B, L + 1), -7, dtype=torch.int32, device=dev),
        accept_len=torch.full((B,), -7, dtype=torch.int32, device=dev),
        status=torch.full((B,), -7, dtype=torch.int32, device=dev))
    if want_dbg:
        out.update(p=torch.empty((B, L), device=dev), q=torch.empty((B, L), device=dev),
                   f=torch.empty((B, L), device=dev), G=torch.full((B, V), -1.0, device=dev))
    if want_terms:
        out.update(accept_mass=torch.full((B, L), -7.0, device=dev), bound_term=torch.full((B, L), -7.0, device=dev))
    ws = workspace if workspace is not None else csd.new_workspace(B, L, V, w.dtype, dev)
    prm = csd.make_params(
        w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
        out["tokens"], out["accept_len"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
        cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=out["status"],
        dbg_p=out.get("p"), dbg_q=out.get("q"), dbg_f=out.get("f"), dbg_G=out.get("G"),
        workspace=ws, stream=stream, back_to_back=back_to_back,
        diag_accept_mass=out.get("accept_mass"), diag_bound_term=out.get("bound_term"))
    csd.csd_verify_ex(prm)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def run_oracle(w, rows=None, **kw):
    h = w.host_arrays()
    if rows is not None:
        h = {k: (v[rows] if v is not None and k != "relax_schedule" else v) for k, v in h.items()}
    ref = oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                        h["relax_schedule"], dtype=w.dtype, target_uncond=h["target_uncond"],
                        draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k, **kw)
    return h, ref


def check(w, rows=None, want_dbg=True, **gpu_kw):
    got = run_gpu(w, want_dbg=want_dbg, **gpu_kw)
    h, ref = run_oracle(w, rows)
    sel = (lambda a: a if rows is None else a[rows])
    rep = compare(ref, sel(got["tokens"]), sel(got["accept_len"]), h["draft_tokens"], h["uniforms"],
                  status=sel(got["status"]),
                  p=sel(got["p"]) if want_dbg else None, q=sel(got["q"]) if want_dbg else None,
                  f=sel(got["f"]) if want_dbg else None, G=sel(got["G"]) if want_dbg else None,
                  tol=TOL[w.dtype])
    return rep, got, ref
