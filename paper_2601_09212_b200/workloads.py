"""Seeded synthetic inputs for the verify-and-resample round.

This module only MAKES inputs (logit rows, draft tokens, uniforms); it holds
none of the method's arithmetic and imports neither the CUDA binding nor the
CPU oracle, so both can be fed from it.  The rows stand in for what a target
model and a drafter would emit on the paper's text-to-image workloads: image
vocabularies of 4k-64k tokens, draft blocks of 4-16 positions, and a drafter
whose logits correlate with the target's (correlation ``rho`` plays the role of
drafter quality).  Draft tokens are drawn from the drafter's own (mixed,
filtered) softmax with library routines, which is the drafting stage the
verify step takes as given.

Randomness: logits and draft tokens come from ``torch.Generator(device)``
(Philox on CUDA) seeded from ``(seed, step)``; the uniforms come from NumPy's
Philox bit generator on the host, mapped to the open interval (0, 1) as
``(2*(k >> 9) + 1) * 2**-24`` for a 32-bit word ``k`` -- exactly representable
in fp32 and fp64, never 0 or 1.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

F32, BF16 = 0, 1
_TORCH_DTYPE = {F32: torch.float32, BF16: torch.bfloat16}


def open_uniforms(shape, seed: int) -> np.ndarray:
    """float32 uniforms strictly inside (0, 1) from Philox."""
    n = int(np.prod(shape))
    words = np.random.Generator(np.random.Philox(key=int(seed))).integers(
        0, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32)
    u = ((2 * (words >> np.uint32(9)).astype(np.float64) + 1.0) * 2.0 ** -24).astype(np.float32)
    return u.reshape(shape)


@dataclass
class Workload:
    """One batch of inputs for one verify call.  Tensors live on ``device``."""
    name: str
    dtype: int                       # F32 or BF16 (storage type of the logits)
    B: int
    gamma: int
    V: int
    target_rows: int                 # gamma or gamma + 1
    target_logits: torch.Tensor      # [B, target_rows, V]
    draft_logits: torch.Tensor       # [B, gamma, V]
    draft_tokens: torch.Tensor       # [B, gamma] int32
    uniforms: torch.Tensor           # [B, gamma + 1] float32
    relax_schedule: torch.Tensor     # [gamma] float32
    target_uncond: Optional[torch.Tensor] = None
    draft_uncond: Optional[torch.Tensor] = None
    cfg_scale: float = 1.0
    top_k: int = 0
    meta: dict = field(default_factory=dict)

    def logits_bytes(self) -> int:
        n = self.target_logits.numel() + self.draft_logits.numel()
        if self.target_uncond is not None:
            n += self.target_uncond.numel() + self.draft_uncond.numel()
        return n * self.target_logits.element_size()

    def host_arrays(self) -> dict:
        """NumPy copies (bf16 as uint16 bit patterns) for a CPU consumer."""
        def conv(t):
            if t is None:
                return None
            t = t.detach().cpu().contiguous()
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).numpy().view(np.uint16).copy()
            return t.numpy().copy()
        return dict(
            target_logits=conv(self.target_logits), draft_logits=conv(self.draft_logits),
            target_uncond=conv(self.target_uncond), draft_uncond=conv(self.draft_uncond),
            draft_tokens=conv(self.draft_tokens), uniforms=conv(self.uniforms),
            relax_schedule=conv(self.relax_schedule))


def _gen(device, seed: int, step: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(step)) & 0x7FFFFFFFFFFFFFFF)
    return g


def _noise(shape, law: str, scale: float, g: torch.Generator, device) -> torch.Tensor:
    z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if law == "gauss":
        return z * scale
    if law == "student3":
        # Student-t with 3 degrees of freedom: N / sqrt(chi2_3 / 3)
        chi = torch.zeros(shape, device=device, dtype=torch.float32)
        for _ in range(3):
            chi += torch.randn(shape, generator=g, device=device, dtype=torch.float32) ** 2
        return z / torch.sqrt(chi / 3.0) * scale
    raise ValueError(law)


def _sample_tokens(drafter_rows_f32: torch.Tensor, g: torch.Generator) -> torch.Tensor:
    """Drafting-stage stand-in: one categorical draw per drafter row."""
    B, L, V = drafter_rows_f32.shape
    probs = torch.softmax(drafter_rows_f32.reshape(B * L, V), dim=-1)
    return torch.multinomial(probs, 1, generator=g).reshape(B, L).to(torch.int32)


def _effective_rows(d_c: torch.Tensor, d_u: Optional[torch.Tensor], cfg_scale: float, top_k: int) -> torch.Tensor:
    """The drafter's effective rows (what it would sample from), in fp32 from the stored values:
    mixed with the unconditional rows if there are any, then top-k filtered."""
    eff = d_c.float()
    if d_u is not None:
        eff = torch.addcmul(d_u.float(), d_c.float() - d_u.float(), torch.tensor(
            cfg_scale, device=d_c.device, dtype=torch.float32))
    if 0 < top_k < eff.shape[-1]:
        kth = torch.topk(eff, top_k, dim=-1).values[..., -1:]
        eff = torch.where(eff >= kth, eff, torch.full_like(eff, float("-inf")))
    return eff


def make(name: str, *, B: int, gamma: int, V: int, dtype: int = F32, rho: float = 0.9,
         law: str = "gauss", scale: float = 3.0, bonus_row: bool = False, cfg: bool = False,
         cfg_scale: float = 4.0, top_k: int = 0, schedule: Optional[np.ndarray] = None,
         seed: int = 0, step: int = 0, device="cpu") -> Workload:
    """Correlated target/drafter logit rows and everything else a call needs.

    ``schedule`` is the caller's relaxation multipliers omega_1..omega_gamma (from
    the library's or the oracle's schedule helper -- this module computes none);
    the default is all ones, i.e. vanilla speculative decoding."""
    device = torch.device(device)
    g = _gen(device, seed, step)
    T = gamma + 1 if bonus_row else gamma
    td = _TORCH_DTYPE[dtype]
    mixw = math.sqrt(max(0.0, 1.0 - rho * rho))

    def pair():
        t = _noise((B, T, V), law, scale, g, device)
        d = rho * t[:, :gamma, :] + mixw * _noise((B, gamma, V), law, scale, g, device)
        return t.to(td), d.to(td)

    t_c, d_c = pair()
    t_u = d_u = None
    if cfg:
        t_u, d_u = pair()
    eff = _effective_rows(d_c, d_u, cfg_scale, top_k)
    tokens = _sample_tokens(eff, g)
    uni = torch.from_numpy(open_uniforms((B, gamma + 1), seed=(seed * 7919 + step))).to(device)
    if schedule is None:
        schedule = np.ones(gamma, dtype=np.float32)
    sched = torch.from_numpy(np.asarray(schedule, dtype=np.float32)).to(device)
    return Workload(name=name, dtype=dtype, B=B, gamma=gamma, V=V, target_rows=T,
                    target_logits=t_c.contiguous(), draft_logits=d_c.contiguous(),
                    draft_tokens=tokens.contiguous(), uniforms=uni, relax_schedule=sched,
                    target_uncond=None if t_u is None else t_u.contiguous(),
                    draft_uncond=None if d_u is None else d_u.contiguous(),
                    cfg_scale=cfg_scale if cfg else 1.0, top_k=top_k,
                    meta=dict(rho=rho, law=law, scale=scale, seed=seed, step=step))


# The four fixed configurations and the sweep grid of the benchmark definition.
CONFIGS = {
    "C1": dict(B=1, gamma=4, V=16384, dtype=F32, rho=0.9, steps=256),
    "C2": dict(B=16, gamma=8, V=16384, dtype=F32, rho=0.9, steps=256),
    "C3": dict(B=64, gamma=8, V=16384, dtype=BF16, rho=0.9, cfg=True, cfg_scale=4.0, top_k=1000,
               steps=576),
    "C4": dict(B=256, gamma=16, V=16384, dtype=BF16, rho=0.85, law="student3", steps=1024),
}
SWEEP = dict(V=(4096, 8192, 16384, 32768, 65536), gamma=(4, 8, 16), B=(1, 16, 64, 256),
             dtype=(F32, BF16), rho=0.9)


def config(name: str, *, step: int = 0, seed: int = 0, device="cpu", **overrides) -> Workload:
    kw = dict(CONFIGS[name])
    kw.pop("steps", None)
    kw.update(overrides)
    return make(name, seed=seed, step=step, device=device, **kw)


# ---- static draft trees -----------------------------------------------------------------------------
@dataclass
class TreeWorkload:
    """One batch of inputs for one tree-structured verify call.  Contexts: 0 is the root, n + 1 the
    context after node n; row c of the logit arrays is the model's output in context c."""
    dtype: int
    B: int
    N: int
    V: int
    parent: np.ndarray               # [N] int32, -1 for a child of the root, else an earlier node
    target_logits: torch.Tensor      # [B, N + 1, V]
    draft_logits: torch.Tensor       # [B, N + 1, V]
    draft_tokens: torch.Tensor       # [B, N] int32
    uniforms: torch.Tensor           # [B, N + 1] float32
    relax_schedule: torch.Tensor     # [D] float32
    target_uncond: Optional[torch.Tensor] = None
    draft_uncond: Optional[torch.Tensor] = None
    cfg_scale: float = 1.0
    top_k: int = 0

    def host_arrays(self) -> dict:
        def conv(t):
            if t is None:
                return None
            t = t.detach().cpu().contiguous()
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).numpy().view(np.uint16).copy()
            return t.numpy().copy()
        return dict(target_logits=conv(self.target_logits), draft_logits=conv(self.draft_logits),
                    target_uncond=conv(self.target_uncond), draft_uncond=conv(self.draft_uncond),
                    draft_tokens=conv(self.draft_tokens), uniforms=conv(self.uniforms),
                    relax_schedule=conv(self.relax_schedule), parent=self.parent.copy())


def static_tree(widths) -> np.ndarray:
    """Parent indices of a static tree in which the first node of every level carries the next level
    (the shape of a top-heavy static draft tree): widths[i] candidates at level i + 1."""
    parent, first_of_prev = [], -1
    for w in widths:
        start = len(parent)
        parent.extend([first_of_prev] * int(w))
        first_of_prev = start
    return np.asarray(parent, dtype=np.int32)


def make_tree(parent, *, B: int, V: int, schedule: np.ndarray, dtype: int = F32, rho: float = 0.9,
              law: str = "gauss", scale: float = 3.0, cfg: bool = False, cfg_scale: float = 4.0, top_k: int = 0,
              seed: int = 0, step: int = 0, device="cpu") -> TreeWorkload:
    """Synthetic inputs for a static draft tree: correlated target/drafter rows for every context, and
    for every node one independent categorical draw from the drafter's effective row of its parent's
    context (the drafting rule the tree verification assumes)."""
    parent = np.asarray(parent, dtype=np.int32)
    N = len(parent)
    w = make("tree", B=B, gamma=N + 1, V=V, dtype=dtype, rho=rho, law=law, scale=scale, cfg=cfg, cfg_scale=cfg_scale,
             top_k=top_k, seed=seed, step=step, device=device)
    eff = _effective_rows(w.draft_logits, w.draft_uncond, cfg_scale, top_k)       # [B, N + 1, V]
    g = _gen(torch.device(device), seed + 77, step)
    ctx = torch.from_numpy(parent.astype(np.int64) + 1).to(eff.device)
    tokens = _sample_tokens(eff[:, ctx, :].contiguous(), g)                         # node n draws in context parent[n] + 1
    sched = torch.from_numpy(np.asarray(schedule, dtype=np.float32)).to(eff.device)
    return TreeWorkload(dtype=dtype, B=B, N=N, V=V, parent=parent, target_logits=w.target_logits,
                        draft_logits=w.draft_logits, draft_tokens=tokens.contiguous(),
                        uniforms=w.uniforms[:, :N + 1].contiguous(), relax_schedule=sched,
                        target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                        cfg_scale=w.cfg_scale, top_k=top_k)
