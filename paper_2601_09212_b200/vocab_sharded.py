"""Vocabulary-sharded verification: binding of the four ``csd_shard_*`` entry points and the three
all-gathers between them (see csd.h).  Each rank of a tensor-parallel LM head holds a contiguous slice
of every logit row; the kernels work on the slice, the exchanges carry a few KB.  Marshalling and
``torch.distributed`` calls only -- every step of the method runs in the library's kernels."""
from __future__ import annotations

import ctypes as C
from typing import Callable, Optional

import torch

from . import CsdError, _dev_ptr, _logit_dtype, _stream_handle, library


class csd_shard_params(C.Structure):
    """Mirror of ``struct csd_shard_params``."""
    _fields_ = [
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("target_uncond", C.c_void_p), ("draft_uncond", C.c_void_p),
        ("cfg_scale", C.c_float), ("dtype", C.c_int32),
        ("B", C.c_int32), ("gamma", C.c_int32), ("target_rows", C.c_int32),
        ("Vs", C.c_int32), ("V_total", C.c_int32), ("v_offset", C.c_int32),
        ("n_shards", C.c_int32), ("shard", C.c_int32),
        ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p), ("relax_schedule", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p),
    ]


def _bind(lib):
    if getattr(lib, "_csd_shard_bound", False):
        return lib
    lib.csd_shard_workspace_size.argtypes = [C.c_int] * 5
    lib.csd_shard_workspace_size.restype = C.c_size_t
    lib.csd_shard_stats.argtypes = [C.POINTER(csd_shard_params), C.c_void_p]
    lib.csd_shard_partial.argtypes = [C.POINTER(csd_shard_params), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.csd_shard_pick.argtypes = [C.POINTER(csd_shard_params), C.c_void_p, C.c_void_p, C.c_void_p]
    lib.csd_shard_emit.argtypes = [C.POINTER(csd_shard_params), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    for name in ("csd_shard_stats", "csd_shard_partial", "csd_shard_pick", "csd_shard_emit"):
        getattr(lib, name).restype = C.c_int
    lib._csd_shard_bound = True
    return lib


class ShardedRound:
    """One rank's side of one round.  The four methods are the four library calls; what each returns is
    what the next all-gather carries.  Keeps its buffers (and the caller's tensors) alive: the calls are
    asynchronous."""

    def __init__(self, target_slice, draft_slice, draft_tokens, uniforms, relax_schedule, *, v_offset: int,
                 V_total: int, shard: int, n_shards: int, target_uncond=None, draft_uncond=None, cfg_scale=1.0,
                 stream=None):
        lib = _bind(library())
        B, T, Vs = target_slice.shape
        gamma = draft_slice.shape[1]
        if draft_slice.shape != (B, gamma, Vs) or T not in (gamma, gamma + 1):
            raise ValueError("shapes: target [B, gamma or gamma+1, Vs], draft [B, gamma, Vs]")
        dt, ldt, dev = _logit_dtype(target_slice), target_slice.dtype, target_slice.device
        self.B, self.gamma, self.T, self.n = B, gamma, T, int(n_shards)
        self.rows = B * (T + gamma)
        self._keep = (target_slice, draft_slice, draft_tokens, uniforms, relax_schedule, target_uncond, draft_uncond)
        need = int(lib.csd_shard_workspace_size(B, gamma, T, Vs, dt))
        if need == 0:
            raise CsdError(-2, "csd_shard_workspace_size")
        self.ws = torch.zeros(need, dtype=torch.uint8, device=dev)
        self.records = torch.empty(self.rows, 4, dtype=torch.float32, device=dev)
        self.totals = torch.empty(B, 2, dtype=torch.float64, device=dev)
        self.cand = torch.empty(B, 2, dtype=torch.int32, device=dev)
        p = csd_shard_params()
        p.target_logits = _dev_ptr(target_slice, "target_slice", ldt)
        p.draft_logits = _dev_ptr(draft_slice, "draft_slice", ldt)
        p.target_uncond = _dev_ptr(target_uncond, "target_uncond", ldt)
        p.draft_uncond = _dev_ptr(draft_uncond, "draft_uncond", ldt)
        p.cfg_scale, p.dtype = float(cfg_scale), dt
        p.B, p.gamma, p.target_rows, p.Vs = B, gamma, T, Vs
        p.V_total, p.v_offset, p.n_shards, p.shard = int(V_total), int(v_offset), int(n_shards), int(shard)
        p.draft_tokens = _dev_ptr(draft_tokens, "draft_tokens", torch.int32)
        p.uniforms = _dev_ptr(uniforms, "uniforms", torch.float32)
        p.relax_schedule = _dev_ptr(relax_schedule, "relax_schedule", torch.float32)
        p.workspace, p.workspace_bytes = self.ws.data_ptr(), need
        p.stream = _stream_handle(stream)
        self.p, self.lib = p, lib

    @staticmethod
    def _check(rc, where):
        if rc != 0:
            raise CsdError(rc, where)

    def stats(self) -> torch.Tensor:
        self._check(self.lib.csd_shard_stats(C.byref(self.p), self.records.data_ptr()), "csd_shard_stats")
        return self.records

    def partial(self, records_all: torch.Tensor, dbg_p=None, dbg_q=None, dbg_f=None) -> torch.Tensor:
        self._records_all = records_all
        self._check(self.lib.csd_shard_partial(
            C.byref(self.p), _dev_ptr(records_all, "records_all", torch.float32), self.totals.data_ptr(),
            _dev_ptr(dbg_p, "dbg_p", torch.float32), _dev_ptr(dbg_q, "dbg_q", torch.float32),
            _dev_ptr(dbg_f, "dbg_f", torch.float32)), "csd_shard_partial")
        return self.totals

    def pick(self, totals_all: torch.Tensor) -> torch.Tensor:
        self._totals_all = totals_all
        self._check(self.lib.csd_shard_pick(
            C.byref(self.p), self._records_all.data_ptr(), _dev_ptr(totals_all, "totals_all", torch.float64),
            self.cand.data_ptr()), "csd_shard_pick")
        return self.cand

    def emit(self, cand_all: torch.Tensor, out_tokens, out_accept_len, out_status=None) -> None:
        self._cand_all = cand_all
        self._check(self.lib.csd_shard_emit(
            C.byref(self.p), _dev_ptr(cand_all, "cand_all", torch.int32), _dev_ptr(out_tokens, "out_tokens", torch.int32),
            _dev_ptr(out_accept_len, "out_accept_len", torch.int32), _dev_ptr(out_status, "out_status", torch.int32)),
            "csd_shard_emit")


def all_gather_rank_major(t: torch.Tensor, n: int, group=None) -> torch.Tensor:
    """[n, *t.shape]: every rank's tensor, in rank order."""
    import torch.distributed as dist
    t = t.contiguous()
    out = torch.empty((n * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)   # concatenated along dim 0
    dist.all_gather_into_tensor(out, t, group=group)
    return out.view((n,) + tuple(t.shape))


def csd_verify_sharded(round_: ShardedRound, out_tokens, out_accept_len, out_status=None, *, group=None,
                       gather: Optional[Callable[[torch.Tensor], torch.Tensor]] = None, dbg_p=None, dbg_q=None,
                       dbg_f=None) -> None:
    """The whole round on this rank: four library calls with an all-gather after each of the first three
    (``torch.distributed`` over ``group``; ``gather`` replaces it, e.g. for one process that holds several
    slices).  Ranks must be numbered in vocabulary order."""
    g = gather if gather is not None else (lambda t: all_gather_rank_major(t, round_.n, group))
    records_all = g(round_.stats())
    totals_all = g(round_.partial(records_all, dbg_p, dbg_q, dbg_f))
    cand_all = g(round_.pick(totals_all))
    round_.emit(cand_all, out_tokens, out_accept_len, out_status)
