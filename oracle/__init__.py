"""fp64 CPU oracle for the Cool-SD verify-and-resample round -- TEST INFRASTRUCTURE.

A thin ``ctypes`` wrapper around ``csd_oracle.c`` (plain C, fp64).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product (``paper_2601_09212_b200``) never does, and this package
never imports the product.

The wrapper does marshalling only; all arithmetic lives in the C file, which
cites the passages of the paper it follows (Algorithm 1, Eq. relax, Eq. sdar,
Eq. opt_G).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csd_oracle.c")
_LIB = os.path.join(_HERE, "libcsd_oracle.so")

F32, BF16, F64 = 0, 1, 2
STATUS_BADROW, STATUS_BADTOKEN, STATUS_ZFALLBACK = 1, 2, 4


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP on, no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"   # moved into place when complete: no process sees half a library
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        try:
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
        finally:
            if os.path.exists(tmp):
                os.remove(tmp)
    return _LIB


class _Params(C.Structure):
    _fields_ = [
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("target_uncond", C.c_void_p), ("draft_uncond", C.c_void_p),
        ("dtype", C.c_int32), ("cfg_scale", C.c_float), ("top_k", C.c_int32),
        ("B", C.c_int32), ("gamma", C.c_int32), ("V", C.c_int32), ("target_rows", C.c_int32),
        ("target_batch_stride", C.c_int64), ("draft_batch_stride", C.c_int64),
        ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p), ("relax_schedule", C.c_void_p),
        ("out_tokens", C.c_void_p), ("out_accept_len", C.c_void_p), ("out_status", C.c_void_p),
        ("p", C.c_void_p), ("q", C.c_void_p), ("f", C.c_void_p), ("G", C.c_void_p),
        ("margin_accept", C.c_void_p), ("margin_cdf", C.c_void_p),
        ("accept_mass", C.c_void_p), ("bound_term", C.c_void_p),
        ("neighbours", C.c_void_p), ("nbr_k", C.c_int32), ("nbr_lambda", C.c_float),
    ]


class _TreeParams(C.Structure):
    _fields_ = [
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("target_uncond", C.c_void_p), ("draft_uncond", C.c_void_p),
        ("dtype", C.c_int32), ("cfg_scale", C.c_float), ("top_k", C.c_int32),
        ("B", C.c_int32), ("N", C.c_int32), ("V", C.c_int32), ("D", C.c_int32),
        ("parent", C.c_void_p), ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p),
        ("relax_schedule", C.c_void_p),
        ("out_tokens", C.c_void_p), ("out_accept_len", C.c_void_p), ("out_nodes", C.c_void_p),
        ("out_status", C.c_void_p), ("G", C.c_void_p), ("margin_accept", C.c_void_p), ("margin_cdf", C.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = C.CDLL(_LIB)
        lib.orc_num_threads.restype = C.c_int
        lib.orc_set_num_threads.argtypes = [C.c_int]
        lib.orc_make_schedule.argtypes = [C.c_int, C.c_double, C.c_double, C.c_int, C.c_void_p]
        lib.orc_make_schedule.restype = C.c_int
        lib.orc_accept_prob.argtypes = [C.c_double, C.c_double, C.c_double]
        lib.orc_accept_prob.restype = C.c_double
        lib.orc_softmax.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        lib.orc_softmax.restype = C.c_int
        lib.orc_resample_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_int, C.c_void_p]
        lib.orc_resample_weights.restype = C.c_double
        lib.orc_resample_dist.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_int, C.c_void_p]
        lib.orc_resample_dist.restype = C.c_double
        lib.orc_position_terms.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_int, C.c_void_p, C.c_void_p]
        lib.orc_position_terms.restype = None
        lib.orc_neighbour_mass.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_double, C.c_int]
        lib.orc_neighbour_mass.restype = C.c_double
        lib.orc_resample_weights_nbr.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_int, C.c_void_p, C.c_int,
                                                 C.c_double, C.c_void_p]
        lib.orc_resample_weights_nbr.restype = C.c_double
        lib.orc_inverse_cdf.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_void_p]
        lib.orc_inverse_cdf.restype = C.c_int
        lib.orc_prepare_row.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int,
                                        C.c_float, C.c_int, C.c_void_p, C.c_void_p]
        lib.orc_prepare_row.restype = None
        lib.orc_sample_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_float, C.c_int, C.c_int, C.c_int,
                                        C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.orc_sample_rows.restype = C.c_int
        lib.orc_verify.argtypes = [C.POINTER(_Params)]
        lib.orc_verify.restype = C.c_int
        lib.orc_verify_tree.argtypes = [C.POINTER(_TreeParams)]
        lib.orc_verify_tree.restype = C.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def set_num_threads(n: int) -> None:
    _load().orc_set_num_threads(int(n))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def make_schedule(kind: int, delta: float, nu_or_ell: float, L: int) -> np.ndarray:
    """omega_1..omega_L; kind 0 uniform, 1 exponential (Eq. sdar), 2 linear."""
    out = np.empty(max(L, 0), dtype=np.float64)
    rc = _load().orc_make_schedule(int(kind), float(delta), float(nu_or_ell), int(L), _ptr(out))
    if rc != 0:
        raise ValueError("orc_make_schedule: bad arguments")
    return out


def accept_prob(p: float, q: float, omega: float) -> float:
    """Eq. relax at one token."""
    return float(_load().orc_accept_prob(float(p), float(q), float(omega)))


def softmax(z) -> Optional[np.ndarray]:
    z = _f64(z)
    P = np.empty_like(z)
    ok = _load().orc_softmax(_ptr(z), int(z.size), _ptr(P))
    return P if ok else None


def resample_weights(P, Q, omega: float):
    """Unnormalised Eq. opt_G and its total Z."""
    P, Q = _f64(P), _f64(Q)
    g = np.empty_like(P)
    Z = _load().orc_resample_weights(_ptr(P), _ptr(Q), float(omega), int(P.size), _ptr(g))
    return g, float(Z)


def resample_dist(P, Q, omega: float) -> np.ndarray:
    """Eq. opt_G (falls back to P when the positive part is empty)."""
    P, Q = _f64(P), _f64(Q)
    G = np.empty_like(P)
    _load().orc_resample_dist(_ptr(P), _ptr(Q), float(omega), int(P.size), _ptr(G))
    return G


def position_terms(P, Q, omega: float):
    """(sum_x Q f, sum_x |P - Q f| - sum_x (1 - f) Q) with f = min{1, omega P/Q}: the inner sum of
    Eq. token_exp and the bracket of Eq. bd2 for one pair of distributions."""
    P, Q = _f64(P), _f64(Q)
    a, b = C.c_double(), C.c_double()
    _load().orc_position_terms(_ptr(P), _ptr(Q), float(omega), int(P.size), C.byref(a), C.byref(b))
    return a.value, b.value


def neighbour_mass(P, nbr_row, lam: float, x: int) -> float:
    """LANTERN++'s aggregated mass of token x over its selected nearest tokens."""
    P = _f64(P)
    nb = np.ascontiguousarray(nbr_row, dtype=np.int32)
    return float(_load().orc_neighbour_mass(_ptr(P), int(P.size), _ptr(nb), int(nb.size), float(lam), int(x)))


def resample_weights_nbr(P, Q, omega: float, neighbours, lam: float):
    """Unnormalised Eq. opt_G with LANTERN++'s acceptance at every candidate, and its total Z."""
    P, Q = _f64(P), _f64(Q)
    nb = np.ascontiguousarray(neighbours, dtype=np.int32)
    g = np.empty_like(P)
    Z = _load().orc_resample_weights_nbr(_ptr(P), _ptr(Q), float(omega), int(P.size), _ptr(nb), int(nb.shape[1]),
                                         float(lam), _ptr(g))
    return g, float(Z)


def inverse_cdf(g, Z: float, u: float):
    g = _f64(g)
    margin = C.c_double(0.0)
    tok = _load().orc_inverse_cdf(_ptr(g), int(g.size), float(Z), float(u), C.byref(margin))
    return int(tok), float(margin.value)


def _raw(a: np.ndarray, dtype: int) -> np.ndarray:
    """Stored logits as the bytes the C side reads (bf16 travels as uint16)."""
    want = {F32: np.float32, BF16: np.uint16, F64: np.float64}[dtype]
    a = np.ascontiguousarray(a)
    if a.dtype != want:
        raise TypeError(f"logits must be {want} for dtype code {dtype}, got {a.dtype}")
    return a


def prepare_row(cond, uncond, dtype: int, cfg_scale: float, top_k: int) -> np.ndarray:
    cond = _raw(cond, dtype)
    un = None if uncond is None else _raw(uncond, dtype)
    V = int(cond.size)
    z = np.empty(V, dtype=np.float64)
    scratch = np.empty(V, dtype=np.float64)
    _load().orc_prepare_row(_ptr(cond), _ptr(un), int(dtype), 0, V, float(cfg_scale), int(top_k),
                            _ptr(z), _ptr(scratch))
    return z


def sample_rows(logits, uniforms, *, dtype: int = F32, uncond=None, cfg_scale: float = 1.0, top_k: int = 0):
    """Algorithm 1, drafting stage: one inverse-CDF draw per row of ``logits`` [R, V] with ``uniforms`` [R].
    Returns (tokens int32 [R], status int32 [R], margin float64 [R])."""
    z = _raw(logits, dtype)
    R, V = z.shape
    zu = None if uncond is None else _raw(uncond, dtype)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert uni.shape == (R,)
    tok, st, mg = np.empty(R, np.int32), np.zeros(R, np.int32), np.empty(R)
    rc = _load().orc_sample_rows(_ptr(z), _ptr(zu), int(dtype), float(cfg_scale), int(top_k), R, V, V,
                                 _ptr(uni), _ptr(tok), _ptr(st), _ptr(mg))
    if rc != 0:
        raise RuntimeError(f"orc_sample_rows failed with code {rc}")
    return tok, st, mg


@dataclass
class VerifyResult:
    tokens: np.ndarray        # [B, gamma+1] int32, -1 padded
    accept_len: np.ndarray    # [B] int32
    status: np.ndarray        # [B] int32
    p: np.ndarray             # [B, gamma] float64
    q: np.ndarray
    f: np.ndarray
    G: Optional[np.ndarray]   # [B, V] float64 (distribution drawn from; zeros if none)
    margin_accept: np.ndarray  # [B, gamma]
    margin_cdf: np.ndarray     # [B]
    accept_mass: Optional[np.ndarray] = None   # [B, gamma]: sum_x Q_i f_i (NaN where a row is unusable)
    bound_term: Optional[np.ndarray] = None    # [B, gamma]: the bracket of Eq. bd2


def verify(target_logits, draft_logits, draft_tokens, uniforms, relax_schedule, *,
           dtype: int = F32, target_uncond=None, draft_uncond=None, cfg_scale: float = 1.0,
           top_k: int = 0, want_G: bool = True, want_pqf: bool = True,
           want_terms: bool = False, neighbours=None, nbr_lambda: float = 0.0) -> VerifyResult:
    """One verification round for B sequences (Algorithm 1, verification stage).

    target_logits [B, T, V] with T in {gamma, gamma+1}; draft_logits [B, gamma, V];
    draft_tokens [B, gamma] int32; uniforms [B, gamma+1] float32 (columns
    0..gamma-1 are r_i, column gamma is the resample / bonus draw);
    relax_schedule [gamma] float32.
    """
    t = _raw(target_logits, dtype)
    d = _raw(draft_logits, dtype)
    B, T, V = t.shape
    gamma = d.shape[1]
    assert d.shape == (B, gamma, V) and T in (gamma, gamma + 1)
    tu = None if target_uncond is None else _raw(target_uncond, dtype)
    du = None if draft_uncond is None else _raw(draft_uncond, dtype)
    if (tu is None) != (du is None):
        raise ValueError("guidance needs both unconditional arrays")
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    om = np.ascontiguousarray(relax_schedule, dtype=np.float32)
    assert tok.shape == (B, gamma) and uni.shape == (B, gamma + 1) and om.shape == (gamma,)
    res = VerifyResult(
        tokens=np.empty((B, gamma + 1), np.int32), accept_len=np.empty(B, np.int32),
        status=np.zeros(B, np.int32),
        p=np.empty((B, gamma)), q=np.empty((B, gamma)), f=np.empty((B, gamma)),
        G=np.zeros((B, V)) if want_G else None,
        margin_accept=np.empty((B, gamma)), margin_cdf=np.empty(B),
        accept_mass=np.empty((B, gamma)) if want_terms else None,
        bound_term=np.empty((B, gamma)) if want_terms else None)
    prm = _Params(
        _ptr(t), _ptr(d), _ptr(tu), _ptr(du), int(dtype), float(cfg_scale), int(top_k),
        B, gamma, V, T, T * V, gamma * V, _ptr(tok), _ptr(uni), _ptr(om),
        _ptr(res.tokens), _ptr(res.accept_len), _ptr(res.status),
        _ptr(res.p) if want_pqf else None, _ptr(res.q) if want_pqf else None,
        _ptr(res.f) if want_pqf else None, _ptr(res.G),
        _ptr(res.margin_accept), _ptr(res.margin_cdf), _ptr(res.accept_mass), _ptr(res.bound_term),
        None, 0, 0.0)
    if neighbours is not None:
        nb = np.ascontiguousarray(neighbours, dtype=np.int32)
        assert nb.ndim == 2 and nb.shape[0] == V
        prm.neighbours, prm.nbr_k, prm.nbr_lambda = _ptr(nb), nb.shape[1], float(nbr_lambda)
    rc = _load().orc_verify(C.byref(prm))
    if rc != 0:
        raise RuntimeError(f"orc_verify failed with code {rc}")
    return res


def tree_depth(parent) -> int:
    """Deepest level of a tree given as parent indices (-1: child of the root)."""
    parent = np.asarray(parent, dtype=np.int64)
    level = np.zeros(len(parent), dtype=np.int64)
    for n, p in enumerate(parent):
        if p < -1 or p >= n:
            raise ValueError("parent[n] must be -1 or an earlier node")
        level[n] = 1 if p < 0 else level[p] + 1
    return int(level.max()) if len(parent) else 0


@dataclass
class TreeResult:
    tokens: np.ndarray        # [B, D+1] int32: accepted path, the drawn token, -1 padding
    accept_len: np.ndarray    # [B] int32
    nodes: np.ndarray         # [B, D] int32: node accepted at each level, -1 padding
    status: np.ndarray        # [B] int32
    G: Optional[np.ndarray]   # [B, V] float64
    margin_accept: np.ndarray  # [B, N]
    margin_cdf: np.ndarray     # [B]


def verify_tree(target_logits, draft_logits, parent, draft_tokens, uniforms, relax_schedule, *,
                dtype: int = F32, target_uncond=None, draft_uncond=None, cfg_scale: float = 1.0,
                top_k: int = 0, want_G: bool = True) -> TreeResult:
    """One verification round over a static tree of candidates (see orc_verify_tree in csd_oracle.c).

    target_logits, draft_logits [B, N+1, V]: row 0 is the root context, row n+1 the context after node n;
    parent [N] int32; draft_tokens [B, N] int32; uniforms [B, N+1] float32 (one accept draw per node, then
    the resample / bonus draw); relax_schedule [D] float32, one multiplier per level."""
    t = _raw(target_logits, dtype)
    d = _raw(draft_logits, dtype)
    B, N1, V = t.shape
    N = N1 - 1
    assert d.shape == (B, N1, V)
    par = np.ascontiguousarray(parent, dtype=np.int32)
    assert par.shape == (N,)
    D = tree_depth(par)
    tu = None if target_uncond is None else _raw(target_uncond, dtype)
    du = None if draft_uncond is None else _raw(draft_uncond, dtype)
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    om = np.ascontiguousarray(relax_schedule, dtype=np.float32)
    assert tok.shape == (B, N) and uni.shape == (B, N + 1) and om.shape == (D,)
    res = TreeResult(tokens=np.empty((B, D + 1), np.int32), accept_len=np.empty(B, np.int32),
                     nodes=np.empty((B, D), np.int32), status=np.zeros(B, np.int32),
                     G=np.zeros((B, V)) if want_G else None,
                     margin_accept=np.empty((B, N)), margin_cdf=np.empty(B))
    prm = _TreeParams(_ptr(t), _ptr(d), _ptr(tu), _ptr(du), int(dtype), float(cfg_scale), int(top_k),
                      B, N, V, D, _ptr(par), _ptr(tok), _ptr(uni), _ptr(om),
                      _ptr(res.tokens), _ptr(res.accept_len), _ptr(res.nodes), _ptr(res.status),
                      _ptr(res.G), _ptr(res.margin_accept), _ptr(res.margin_cdf))
    rc = _load().orc_verify_tree(C.byref(prm))
    if rc != 0:
        raise RuntimeError(f"orc_verify_tree failed with code {rc}")
    return res
