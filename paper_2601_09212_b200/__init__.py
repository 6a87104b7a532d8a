"""B200-native batched verify-and-resample for Cool-SD (annealed relaxed speculative decoding).

Thin binding over the C ABI of ``libcsd.so`` (declared in ``include/csd.h``): the
functions here have the ABI's names and only marshal arguments -- pointers of
``torch`` tensors, sizes, the current CUDA stream.  Every step of the method
runs in the library's CUDA kernels.  There is no CPU fallback: if the library
has not been built, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from ._build import LIB_PATH

CSD_F32, CSD_BF16 = 0, 1
CSD_STATUS_BADROW, CSD_STATUS_BADTOKEN, CSD_STATUS_ZFALLBACK, CSD_STATUS_TIMEOUT = 1, 2, 4, 8
CSD_STATIC_SCRATCH_BYTES = 2 * 1024 * 1024
EXPORTS = ("csd_verify", "csd_verify_static", "csd_verify_ex", "csd_workspace_size", "csd_workspace_init", "csd_launch_count", "csd_verify_host",
           "csd_host_staging_size", "csd_make_schedule", "csd_error_string", "csd_version",
           "csd_sample_rows", "csd_sample_workspace_size", "csd_test_hooks", "csd_checked_report",
           "csd_verify_tree", "csd_tree_workspace_size", "csd_tree_depth", "csd_verify_similar",
           "csd_shard_workspace_size", "csd_shard_stats", "csd_shard_partial", "csd_shard_pick", "csd_shard_emit")


class CsdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {error_string(code)} (code {code})")


class csd_params(C.Structure):
    """Mirror of ``struct csd_params``."""
    _fields_ = [
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("target_uncond", C.c_void_p), ("draft_uncond", C.c_void_p),
        ("cfg_scale", C.c_float), ("top_k", C.c_int32), ("dtype", C.c_int32),
        ("B", C.c_int32), ("gamma", C.c_int32), ("V", C.c_int32), ("target_rows", C.c_int32),
        ("target_batch_stride", C.c_int64), ("draft_batch_stride", C.c_int64),
        ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p), ("relax_schedule", C.c_void_p),
        ("out_tokens", C.c_void_p), ("out_accept_len", C.c_void_p), ("out_status", C.c_void_p),
        ("dbg_p", C.c_void_p), ("dbg_q", C.c_void_p), ("dbg_f", C.c_void_p), ("dbg_G", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p),
        ("back_to_back", C.c_int32),
        ("diag_accept_mass", C.c_void_p), ("diag_bound_term", C.c_void_p),
    ]


class csd_tree_params(C.Structure):
    """Mirror of ``struct csd_tree_params``."""
    _fields_ = [
        ("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
        ("target_uncond", C.c_void_p), ("draft_uncond", C.c_void_p),
        ("cfg_scale", C.c_float), ("top_k", C.c_int32), ("dtype", C.c_int32),
        ("B", C.c_int32), ("N", C.c_int32), ("V", C.c_int32),
        ("parent", C.c_void_p), ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p),
        ("relax_schedule", C.c_void_p),
        ("out_tokens", C.c_void_p), ("out_accept_len", C.c_void_p), ("out_nodes", C.c_void_p),
        ("out_status", C.c_void_p), ("dbg_G", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p),
    ]


_lib = None


def library() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2601_09212_b200._build` "
                "(there is no fallback path)")
        _lib = _configure(C.CDLL(LIB_PATH))
    return _lib


def _configure(lib: C.CDLL) -> C.CDLL:
    lib.csd_verify.argtypes = [C.c_void_p] * 5 + [C.c_int] * 3 + [C.c_void_p] * 3
    lib.csd_verify.restype = C.c_int
    lib.csd_verify_static.argtypes = lib.csd_verify.argtypes
    lib.csd_verify_static.restype = C.c_int
    lib.csd_verify_ex.argtypes = [C.POINTER(csd_params)]
    lib.csd_verify_ex.restype = C.c_int
    lib.csd_workspace_size.argtypes = [C.c_int] * 4
    lib.csd_workspace_size.restype = C.c_size_t
    lib.csd_launch_count.argtypes = [C.POINTER(csd_params)]
    lib.csd_launch_count.restype = C.c_int
    lib.csd_workspace_init.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.csd_workspace_init.restype = C.c_int
    lib.csd_verify_host.argtypes = [C.POINTER(csd_params), C.c_void_p, C.c_size_t]
    lib.csd_verify_host.restype = C.c_int
    lib.csd_host_staging_size.argtypes = [C.POINTER(csd_params)]
    lib.csd_host_staging_size.restype = C.c_size_t
    lib.csd_make_schedule.argtypes = [C.c_int, C.c_double, C.c_double, C.c_int, C.c_void_p]
    lib.csd_make_schedule.restype = C.c_int
    lib.csd_error_string.argtypes = [C.c_int]
    lib.csd_error_string.restype = C.c_char_p
    lib.csd_version.restype = C.c_int
    lib.csd_test_hooks.argtypes = [C.c_int, C.c_int]
    lib.csd_test_hooks.restype = C.c_int
    lib.csd_verify_similar.argtypes = [C.POINTER(csd_params), C.c_void_p, C.c_int, C.c_float]
    lib.csd_verify_similar.restype = C.c_int
    lib.csd_verify_tree.argtypes = [C.POINTER(csd_tree_params)]
    lib.csd_verify_tree.restype = C.c_int
    lib.csd_tree_workspace_size.argtypes = [C.c_int] * 4
    lib.csd_tree_workspace_size.restype = C.c_size_t
    lib.csd_tree_depth.argtypes = [C.c_void_p, C.c_int]
    lib.csd_tree_depth.restype = C.c_int
    lib.csd_sample_workspace_size.argtypes = [C.c_int] * 3
    lib.csd_sample_workspace_size.restype = C.c_size_t
    lib.csd_sample_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                    C.c_int, C.c_void_p]
    lib.csd_sample_rows.restype = C.c_int
    lib.csd_checked_report.argtypes = [C.c_void_p]
    lib.csd_checked_report.restype = C.c_int
    return lib


@contextlib.contextmanager
def checked_library():
    """Testing aid: inside the block every call of this module goes to the bounds-checked build of the
    library (csd.h, csd_checked_report), compiled on first use.  Yields a function that returns the
    record (bad indices seen, first index, row length, site) after synchronising the device."""
    global _lib
    from ._build import CHECKED_LIB_PATH, build_checked_library
    if not os.path.exists(CHECKED_LIB_PATH):
        build_checked_library()
    lib = _configure(C.CDLL(CHECKED_LIB_PATH))

    def report():
        rec = (C.c_int32 * 4)()
        rc = lib.csd_checked_report(rec)
        if rc != 1:
            raise CsdError(rc, "csd_checked_report") if rc < 0 else RuntimeError("not a checked build")
        return tuple(rec)

    before, _lib = library(), lib
    try:
        yield report
    finally:
        _lib = before


def error_string(code: int) -> str:
    return library().csd_error_string(int(code)).decode()


csd_error_string = error_string


def csd_version() -> int:
    return int(library().csd_version())


def csd_test_hooks(wait_limit_log2_cycles: int = 0, drop_first_copy: bool = False) -> None:
    """Testing aid for the bounded waits (see csd.h); ``csd_test_hooks()`` restores normal operation."""
    rc = library().csd_test_hooks(int(wait_limit_log2_cycles), int(bool(drop_first_copy)))
    if rc != 0:
        raise CsdError(rc, "csd_test_hooks")


def csd_make_schedule(kind: int, delta: float, nu_or_ell: float, L: int) -> np.ndarray:
    """omega_1..omega_L as float32 (host).  kind 0 uniform, 1 exponential, 2 linear."""
    out = np.empty(max(int(L), 1), dtype=np.float32)
    rc = library().csd_make_schedule(int(kind), float(delta), float(nu_or_ell), int(L),
                                     out.ctypes.data_as(C.c_void_p))
    if rc != 0:
        raise CsdError(rc, "csd_make_schedule")
    return out[:L]


def csd_workspace_size(B: int, gamma: int, V: int, dtype: int) -> int:
    return int(library().csd_workspace_size(int(B), int(gamma), int(V), int(dtype)))


def _dev_ptr(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _host_ptr(t, name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        if not t.flags.c_contiguous:
            raise ValueError(f"{name} must be contiguous")
        return t.ctypes.data
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _logit_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CSD_F32
    if t.dtype == torch.bfloat16:
        return CSD_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


def csd_verify(target_logits, draft_logits, draft_tokens, uniforms, relax_schedule, out_tokens,
               out_accept_len, stream=None) -> None:
    """Simple form: fp32 [B, gamma, V] logits; see ``csd_verify`` in csd.h."""
    B, gamma, V = target_logits.shape
    if draft_logits.shape != (B, gamma, V):
        raise ValueError("target_logits and draft_logits must both be [B, gamma, V]")
    rc = library().csd_verify(
        _dev_ptr(target_logits, "target_logits", torch.float32),
        _dev_ptr(draft_logits, "draft_logits", torch.float32),
        _dev_ptr(draft_tokens, "draft_tokens", torch.int32),
        _dev_ptr(uniforms, "uniforms", torch.float32),
        _dev_ptr(relax_schedule, "relax_schedule", torch.float32),
        B, gamma, V,
        _dev_ptr(out_tokens, "out_tokens", torch.int32),
        _dev_ptr(out_accept_len, "out_accept_len", torch.int32),
        _stream_handle(stream))
    if rc != 0:
        raise CsdError(rc, "csd_verify")


def csd_verify_static(target_logits, draft_logits, draft_tokens, uniforms, relax_schedule, out_tokens,
                      out_accept_len, stream=None) -> None:
    """``csd_verify`` for callers that must not allocate on the device (inside a stream capture,
    under a memory pool that owns the whole GPU, on a latency-critical thread): same arguments
    and results, scratch taken from a fixed array inside the library, so nothing is allocated.
    Raises ``CsdError`` (code -8) when the problem needs more than ``CSD_STATIC_SCRATCH_BYTES``;
    calls on one device share that array and must not overlap on the GPU."""
    B, gamma, V = target_logits.shape
    if draft_logits.shape != (B, gamma, V):
        raise ValueError("target_logits and draft_logits must both be [B, gamma, V]")
    rc = library().csd_verify_static(
        _dev_ptr(target_logits, "target_logits", torch.float32),
        _dev_ptr(draft_logits, "draft_logits", torch.float32),
        _dev_ptr(draft_tokens, "draft_tokens", torch.int32),
        _dev_ptr(uniforms, "uniforms", torch.float32),
        _dev_ptr(relax_schedule, "relax_schedule", torch.float32),
        B, gamma, V,
        _dev_ptr(out_tokens, "out_tokens", torch.int32),
        _dev_ptr(out_accept_len, "out_accept_len", torch.int32),
        _stream_handle(stream))
    if rc != 0:
        raise CsdError(rc, "csd_verify_static")


def make_params(target_logits, draft_logits, draft_tokens, uniforms, relax_schedule, out_tokens,
                out_accept_len, *, target_uncond=None, draft_uncond=None, cfg_scale=1.0, top_k=0,
                out_status=None, dbg_p=None, dbg_q=None, dbg_f=None, dbg_G=None, workspace=None,
                stream=None, host=False, back_to_back=False, diag_accept_mass=None,
                diag_bound_term=None) -> csd_params:
    """Fill a ``csd_params`` from tensors (device tensors, or host ones with ``host=True``)."""
    B, T, V = target_logits.shape
    gamma = draft_logits.shape[1]
    if draft_logits.shape != (B, gamma, V) or T not in (gamma, gamma + 1):
        raise ValueError("shapes: target [B, gamma or gamma+1, V], draft [B, gamma, V]")
    ptr = _host_ptr if host else _dev_ptr
    dt = _logit_dtype(target_logits)
    ldt = target_logits.dtype
    p = csd_params()
    p.target_logits = ptr(target_logits, "target_logits", ldt)
    p.draft_logits = ptr(draft_logits, "draft_logits", ldt)
    p.target_uncond = ptr(target_uncond, "target_uncond", ldt)
    p.draft_uncond = ptr(draft_uncond, "draft_uncond", ldt)
    p.cfg_scale = float(cfg_scale)
    p.top_k = int(top_k)
    p.dtype = dt
    p.B, p.gamma, p.V, p.target_rows = B, gamma, V, T
    p.target_batch_stride = T * V
    p.draft_batch_stride = gamma * V
    p.draft_tokens = ptr(draft_tokens, "draft_tokens", torch.int32)
    p.uniforms = ptr(uniforms, "uniforms", torch.float32)
    p.relax_schedule = ptr(relax_schedule, "relax_schedule", torch.float32)
    p.out_tokens = ptr(out_tokens, "out_tokens", torch.int32)
    p.out_accept_len = ptr(out_accept_len, "out_accept_len", torch.int32)
    p.out_status = ptr(out_status, "out_status", torch.int32)
    p.dbg_p = ptr(dbg_p, "dbg_p", torch.float32)
    p.dbg_q = ptr(dbg_q, "dbg_q", torch.float32)
    p.dbg_f = ptr(dbg_f, "dbg_f", torch.float32)
    p.dbg_G = ptr(dbg_G, "dbg_G", torch.float32)
    if workspace is not None:
        p.workspace = _dev_ptr(workspace, "workspace")
        p.workspace_bytes = workspace.numel() * workspace.element_size()
    p.stream = _stream_handle(stream)
    p.back_to_back = 1 if back_to_back else 0
    p.diag_accept_mass = ptr(diag_accept_mass, "diag_accept_mass", torch.float32)
    p.diag_bound_term = ptr(diag_bound_term, "diag_bound_term", torch.float32)
    return p


def csd_verify_ex(params: csd_params) -> None:
    rc = library().csd_verify_ex(C.byref(params))
    if rc != 0:
        raise CsdError(rc, "csd_verify_ex")


def csd_launch_count(params: csd_params) -> int:
    n = library().csd_launch_count(C.byref(params))
    if n < 0:
        raise CsdError(n, "csd_launch_count")
    return int(n)


def csd_host_staging_size(params: csd_params) -> int:
    return int(library().csd_host_staging_size(C.byref(params)))


def csd_verify_host(params: csd_params, staging: torch.Tensor) -> None:
    rc = library().csd_verify_host(C.byref(params), _dev_ptr(staging, "staging"),
                                   staging.numel() * staging.element_size())
    if rc != 0:
        raise CsdError(rc, "csd_verify_host")


def new_workspace(B: int, gamma: int, V: int, dtype: int, device="cuda") -> torch.Tensor:
    """A zero-filled device buffer of the size csd_verify_ex asks for (torch's allocator gives
    512-byte alignment)."""
    n = csd_workspace_size(B, gamma, V, dtype)
    if n == 0:
        raise CsdError(-2, "csd_workspace_size")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def csd_sample_workspace_size(R: int, V: int, dtype: int) -> int:
    return int(library().csd_sample_workspace_size(int(R), int(V), int(dtype)))


def csd_sample_rows(logits, uniforms, out_tokens, *, uncond=None, cfg_scale=1.0, top_k=0, out_status=None,
                    workspace=None, back_to_back=False, stream=None) -> None:
    """Drafting stage: one inverse-CDF draw per row of ``logits`` [R, V] (device tensors).

    ``logits`` (and ``uncond``, with the same strides) may be a view whose rows are contiguous but
    spaced apart, such as ``all_logits[:, -1]`` of a ``[B, T, V]`` tensor: the row stride is passed on."""
    R, V = logits.shape
    dt = _logit_dtype(logits)
    ldt = logits.dtype

    def rows_ptr(t, name):
        if t is None:
            return None
        if (not t.is_cuda or t.dtype != ldt or t.dim() != 2 or t.shape != logits.shape or t.stride(1) != 1
                or t.stride(0) != logits.stride(0) or t.stride(0) < V):
            raise ValueError(f"{name} must be a CUDA tensor [R, V] of {ldt} with contiguous rows and the row stride of logits")
        return t.data_ptr()

    if workspace is None:
        workspace = torch.zeros(csd_sample_workspace_size(R, V, dt), dtype=torch.uint8, device=logits.device)
    rc = library().csd_sample_rows(
        rows_ptr(logits, "logits"), rows_ptr(uncond, "uncond"), float(cfg_scale), int(top_k), dt, R, V,
        int(logits.stride(0)) if R > 1 else V, _dev_ptr(uniforms, "uniforms", torch.float32), _dev_ptr(out_tokens, "out_tokens", torch.int32),
        _dev_ptr(out_status, "out_status", torch.int32), _dev_ptr(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), 1 if back_to_back else 0, _stream_handle(stream))
    if rc != 0:
        raise CsdError(rc, "csd_sample_rows")


def csd_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    rc = library().csd_workspace_init(_dev_ptr(workspace, "workspace"),
                                      workspace.numel() * workspace.element_size(), _stream_handle(stream))
    if rc != 0:
        raise CsdError(rc, "csd_workspace_init")


_tree_ws = {}


def csd_tree_depth(parent) -> int:
    """Deepest level of a static tree given as parent indices; raises on a malformed tree."""
    par = np.ascontiguousarray(parent, dtype=np.int32)
    d = library().csd_tree_depth(par.ctypes.data_as(C.c_void_p), int(par.size))
    if d < 0:
        raise CsdError(d, "csd_tree_depth")
    return int(d)


def csd_tree_workspace_size(B: int, N: int, V: int, dtype: int) -> int:
    return int(library().csd_tree_workspace_size(int(B), int(N), int(V), int(dtype)))


def csd_verify_tree(target_logits, draft_logits, parent, draft_tokens, uniforms, relax_schedule, out_tokens,
                    out_accept_len, *, target_uncond=None, draft_uncond=None, cfg_scale=1.0, top_k=0,
                    out_nodes=None, out_status=None, dbg_G=None, workspace=None, stream=None) -> None:
    """Tree-structured verification (see ``csd_verify_tree`` in csd.h): logits [B, N + 1, V] per context,
    ``parent`` a host array [N], ``draft_tokens`` [B, N], ``uniforms`` [B, N + 1], ``relax_schedule`` [D]."""
    B, C1, V = target_logits.shape
    N = C1 - 1
    par = np.ascontiguousarray(parent, dtype=np.int32)
    if draft_logits.shape != (B, C1, V) or par.shape != (N,):
        raise ValueError("shapes: target and draft [B, N + 1, V], parent [N]")
    dt = _logit_dtype(target_logits)
    ldt = target_logits.dtype
    if workspace is None:
        # one grow-only buffer per device, kept by the module: the call is asynchronous, so a buffer made
        # here must outlive this function
        need = csd_tree_workspace_size(B, N, V, dt)
        key = target_logits.device
        workspace = _tree_ws.get(key)
        if workspace is None or workspace.numel() < need:
            workspace = torch.zeros(need, dtype=torch.uint8, device=key)
            _tree_ws[key] = workspace
    p = csd_tree_params()
    p.target_logits = _dev_ptr(target_logits, "target_logits", ldt)
    p.draft_logits = _dev_ptr(draft_logits, "draft_logits", ldt)
    p.target_uncond = _dev_ptr(target_uncond, "target_uncond", ldt)
    p.draft_uncond = _dev_ptr(draft_uncond, "draft_uncond", ldt)
    p.cfg_scale, p.top_k, p.dtype = float(cfg_scale), int(top_k), dt
    p.B, p.N, p.V = B, N, V
    p.parent = par.ctypes.data
    p.draft_tokens = _dev_ptr(draft_tokens, "draft_tokens", torch.int32)
    p.uniforms = _dev_ptr(uniforms, "uniforms", torch.float32)
    p.relax_schedule = _dev_ptr(relax_schedule, "relax_schedule", torch.float32)
    p.out_tokens = _dev_ptr(out_tokens, "out_tokens", torch.int32)
    p.out_accept_len = _dev_ptr(out_accept_len, "out_accept_len", torch.int32)
    p.out_nodes = _dev_ptr(out_nodes, "out_nodes", torch.int32)
    p.out_status = _dev_ptr(out_status, "out_status", torch.int32)
    p.dbg_G = _dev_ptr(dbg_G, "dbg_G", torch.float32)
    p.workspace = _dev_ptr(workspace, "workspace")
    p.workspace_bytes = workspace.numel() * workspace.element_size()
    p.stream = _stream_handle(stream)
    rc = library().csd_verify_tree(C.byref(p))
    if rc != 0:
        raise CsdError(rc, "csd_verify_tree")


def csd_verify_similar(params: csd_params, neighbours: torch.Tensor, nbr_lambda: float) -> None:
    """``csd_verify_ex`` with LANTERN++'s similarity-relaxed acceptance and the paper's G* (see csd.h):
    ``neighbours`` is a device int32 tensor [V, k]."""
    if neighbours.dim() != 2 or neighbours.shape[0] != params.V:
        raise ValueError("neighbours must be [V, k]")
    rc = library().csd_verify_similar(C.byref(params), _dev_ptr(neighbours, "neighbours", torch.int32),
                                      int(neighbours.shape[1]), float(nbr_lambda))
    if rc != 0:
        raise CsdError(rc, "csd_verify_similar")
