"""Comparison of a candidate implementation's outputs with the oracle's -- TEST INFRASTRUCTURE.

Accepted lengths and emitted tokens must be identical, except where the
oracle itself says the decision was within ``near`` (1e-6) of a threshold:
an accept test with |r_i - f_i| < near, or an inverse-CDF draw whose uniform
lies within ``near`` of the boundary between the two candidate tokens.  Such
cases are counted, never ignored silently, and a mismatch must be the decision
on the other side of exactly that threshold.  Probabilities (p, q, f) and the
distribution drawn from must agree within ``tol`` absolute.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

NEAR = 1e-6


@dataclass
class Report:
    n_seq: int = 0
    tau_mismatch_near: int = 0        # accepted length differs, explained by a near-threshold accept test
    token_mismatch_near: int = 0      # emitted token differs, explained by a near-threshold CDF boundary
    unexplained: list = field(default_factory=list)   # (b, reason)
    near_accept_tests: int = 0        # oracle-side count of accept tests within NEAR of f
    near_cdf_draws: int = 0           # oracle-side count of draws within NEAR of a boundary
    max_err_p: float = 0.0
    max_err_q: float = 0.0
    max_err_f: float = 0.0
    max_err_G: float = 0.0
    status_mismatch: int = 0

    @property
    def ok(self) -> bool:
        return not self.unexplained and self.status_mismatch == 0

    def summary(self) -> str:
        return (f"{self.n_seq} sequences: tau mismatches (near-threshold) {self.tau_mismatch_near}, "
                f"token mismatches (near-threshold) {self.token_mismatch_near}, unexplained "
                f"{len(self.unexplained)}, status mismatches {self.status_mismatch}; oracle-side near "
                f"accept tests {self.near_accept_tests}, near CDF draws {self.near_cdf_draws}; max |err| "
                f"p {self.max_err_p:.2e} q {self.max_err_q:.2e} f {self.max_err_f:.2e} G {self.max_err_G:.2e}")


def compare(ref, tokens, accept_len, draft_tokens, uniforms, *, status=None, p=None, q=None, f=None,
            G=None, tol: float = 1e-5, near: float = NEAR) -> Report:
    """``ref`` is an ``oracle.VerifyResult``; the other arrays are the candidate's outputs
    (NumPy, same shapes) and the inputs both sides consumed."""
    tokens = np.asarray(tokens)
    accept_len = np.asarray(accept_len)
    B, L1 = tokens.shape
    L = L1 - 1
    rep = Report(n_seq=B)
    fin = np.isfinite(ref.margin_accept)
    rep.near_accept_tests = int((ref.margin_accept[fin] < near).sum())
    rep.near_cdf_draws = int((ref.margin_cdf[np.isfinite(ref.margin_cdf)] < near).sum())

    for name, mine, theirs in (("p", p, ref.p), ("q", q, ref.q), ("f", f, ref.f)):
        if mine is None:
            continue
        mine = np.asarray(mine, dtype=np.float64)
        okm = np.isfinite(theirs)
        if np.any(np.isfinite(mine) != okm):
            rep.unexplained.append((-1, f"{name}: finite/NaN pattern differs"))
        err = float(np.abs(mine[okm] - theirs[okm]).max()) if okm.any() else 0.0
        setattr(rep, f"max_err_{name}", err)
        if err > tol:
            rep.unexplained.append((-1, f"{name}: max abs error {err:.3e} > {tol:.1e}"))

    for b in range(B):
        to, tg = int(ref.accept_len[b]), int(accept_len[b])
        if tg < 0 or tg > L:
            rep.unexplained.append((b, f"accept_len {tg} out of range"))
            continue
        if to != tg:
            first = min(to, tg)   # the first decision on which the two sides differ
            if first < L and ref.margin_accept[b, first] < near:
                rep.tau_mismatch_near += 1
            else:
                rep.unexplained.append((b, f"accept_len {tg} vs oracle {to}, margin "
                                           f"{ref.margin_accept[b, min(first, L - 1)]:.3e}"))
            # structure must still hold on the candidate's side
            if not np.array_equal(tokens[b, :tg], draft_tokens[b, :tg]) or np.any(tokens[b, tg + 1:] != -1):
                rep.unexplained.append((b, "emitted block is not draft-prefix + one token + padding"))
            continue
        if not np.array_equal(tokens[b, :to], draft_tokens[b, :to]):
            rep.unexplained.append((b, "accepted prefix differs from the draft tokens"))
        if np.any(tokens[b, to + 1:] != -1):
            rep.unexplained.append((b, "padding after the emitted block is not -1"))
        if status is not None and int(status[b]) != int(ref.status[b]):
            rep.status_mismatch += 1
        xo, xg = int(ref.tokens[b, to]), int(tokens[b, to])
        if G is not None and ref.G is not None:
            err = float(np.abs(np.asarray(G[b], dtype=np.float64) - ref.G[b]).max())
            rep.max_err_G = max(rep.max_err_G, err)
            if err > tol:
                rep.unexplained.append((b, f"G: max abs error {err:.3e} > {tol:.1e}"))
        if xo != xg:
            explained = False
            if xo >= 0 and 0 <= xg < ref.G.shape[1] and ref.margin_cdf[b] < near and ref.G is not None:
                cum = np.cumsum(ref.G[b])
                lo = cum[xg - 1] if xg > 0 else 0.0
                hi = cum[xg]
                u = float(uniforms[b, L])
                dist = 0.0 if lo <= u * cum[-1] <= hi else min(abs(u * cum[-1] - lo), abs(u * cum[-1] - hi))
                explained = ref.G[b, xg] > 0 and dist < 2 * near
            if explained:
                rep.token_mismatch_near += 1
            else:
                rep.unexplained.append((b, f"token {xg} vs oracle {xo} at slot {to}, cdf margin "
                                           f"{ref.margin_cdf[b]:.3e}"))
    return rep
