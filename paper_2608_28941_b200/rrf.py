"""ctypes binding of librrf.so: same names as include/rrf.h, argument marshalling only.

Every function takes torch CUDA tensors (device memory and streams are PyTorch's),
passes raw pointers, sizes and the current CUDA stream to the C ABI and returns
what the library wrote.  Nothing is computed here, and there is no fallback: a
missing or unloadable library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

RRF_F64, RRF_F32 = 0, 1
RRF_OK, RRF_MAX_RANK_REACHED = 0, 1
RRF_ERR_INVALID_ARG, RRF_ERR_WORKSPACE, RRF_ERR_CUDA, RRF_ERR_TIMEOUT, RRF_ERR_NONFINITE = -1, -2, -3, -4, -5
RRF_FLAG_INPLACE, RRF_FLAG_FIXED_RANK, RRF_FLAG_ONE_QUEUE, RRF_FLAG_TWO_QUEUES, RRF_FLAG_NO_GRAPH = 1, 2, 4, 8, 16
RRF_FLAG_SAMPLE_ALWAYS, RRF_FLAG_SAMPLE_NEVER, RRF_FLAG_PANEL_TREE = 32, 64, 128
RRF_FLAG_NO_UPDATE = 256
RRF_FLAG_PANEL_BLOCKED = 512

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "librrf.so")
_lib = None


class rrf_params_t(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("b", C.c_int32), ("max_rank", C.c_int32), ("estimator", C.c_int32),
                ("m", C.c_int64), ("n", C.c_int64), ("tol", C.c_double), ("tol_is_relative", C.c_int32),
                ("flags", C.c_uint32), ("seed", C.c_uint64), ("tune_panel_ctas", C.c_int32), ("tune_gate", C.c_int32)]


class rrf_result_t(C.Structure):
    _fields_ = [("status", C.c_int32), ("k", C.c_int32), ("steps", C.c_int32), ("cuda_error", C.c_int32),
                ("normA2", C.c_double), ("sigma2", C.c_double), ("E_sub", C.c_double), ("E_dir", C.c_double),
                ("queues", C.c_int32), ("panel_ctas", C.c_int32), ("fused_samples", C.c_int32),
                ("extra_samples", C.c_int32), ("kernel_launches", C.c_int32), ("n_est", C.c_int32)]


RRF_PHASES = ["init", "sample", "panel", "tfactor", "vtw", "tz", "update", "stop", "skipped"]


class rrf_profile_t(C.Structure):
    _fields_ = [("ms", C.c_double * 9), ("launches", C.c_int32 * 9), ("pad", C.c_int32)]


EXPORTS = ["rrf_run_colmajor", "rrf_colmajor_workspace_bytes", "rrf_transpose", "rrf_set_single_engine", "rrf_sample_workspace_bytes", "rrf_sample_panel", "rrf_frobenius_sq", "rrf_panel_qr_blocked", "rrf_panel_qr_tree", "rrf_transfer_workspace_bytes", "rrf_subspace_transfer", "rrf_selftest_timeout", "rrf_panel_qr_static", "rrf_set_profiling", "rrf_get_profile", "rrf_measure_peak", "rrf_create", "rrf_destroy", "rrf_workspace_bytes", "rrf_run", "rrf_panel_workspace_bytes",
           "rrf_panel_qr", "rrf_apply_workspace_bytes", "rrf_apply_qt", "rrf_apply_q", "rrf_form_q",
           "rrf_fill_omega", "rrf_last_status", "rrf_status_string"]


def load():
    """Open librrf.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_28941_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64, u64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_size_t
    lib.rrf_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.rrf_destroy.argtypes = [vp]
    lib.rrf_workspace_bytes.argtypes = [C.POINTER(rrf_params_t), C.POINTER(sz)]
    lib.rrf_run.argtypes = [vp, C.POINTER(rrf_params_t), vp, i64, vp, i64, vp, i64, vp, vp, i64, vp, sz, vp,
                            C.POINTER(rrf_result_t), C.POINTER(C.c_double), C.POINTER(C.c_double),
                            C.POINTER(C.c_double)]
    lib.rrf_run_colmajor.argtypes = lib.rrf_run.argtypes
    lib.rrf_colmajor_workspace_bytes.argtypes = [C.POINTER(rrf_params_t), C.POINTER(sz)]
    lib.rrf_transpose.argtypes = [vp, i32, i64, i64, vp, i64, vp, i64, vp]
    lib.rrf_panel_workspace_bytes.argtypes = [i32, i64, i32, C.POINTER(sz)]
    lib.rrf_panel_qr.argtypes = [vp, i32, i64, i32, vp, i64, vp, i64, vp, i64, vp, sz, vp]
    lib.rrf_panel_qr_tree.argtypes = [vp, i32, i64, i32, vp, i64, vp, i64, vp, i64, vp, sz, vp]
    lib.rrf_panel_qr_blocked.argtypes = [vp, i32, i64, i32, vp, i64, vp, i64, vp, i64, vp, sz, vp]
    lib.rrf_panel_qr_static.argtypes = [i32, i64, i32, vp, i64, vp, i64, vp, i64, vp]
    lib.rrf_apply_workspace_bytes.argtypes = [i32, i64, i64, i32, C.POINTER(sz)]
    lib.rrf_sample_workspace_bytes.argtypes = [i32, i64, i32, C.POINTER(sz)]
    lib.rrf_sample_panel.argtypes = [vp, i32, i64, i64, i32, vp, i64, vp, i64, vp, vp, sz, vp]
    lib.rrf_frobenius_sq.argtypes = [vp, i32, i64, i64, vp, i64, vp, vp, sz, vp]
    for f in (lib.rrf_apply_qt, lib.rrf_apply_q):
        f.argtypes = [vp, i32, i64, i32, i32, vp, i64, vp, i64, vp, i64, i64, vp, sz, vp]
    lib.rrf_form_q.argtypes = [vp, i32, i64, i32, i32, vp, i64, vp, i64, vp, i64, vp, sz, vp]
    lib.rrf_fill_omega.argtypes = [vp, i32, u64, i64, i32, i32, vp, i64, vp]
    lib.rrf_transfer_workspace_bytes.argtypes = [i32, i64, i64, i32, C.POINTER(sz)]
    lib.rrf_subspace_transfer.argtypes = [vp, i32, i64, i32, i32, vp, i64, vp, i64, i32, vp, i64, vp, i64, vp, i64, i64,
                                          vp, i64, vp, sz, vp]
    lib.rrf_last_status.argtypes = [vp, vp]
    lib.rrf_selftest_timeout.argtypes = [vp, C.c_double, vp]
    lib.rrf_set_single_engine.argtypes = [vp, i32, i32]
    lib.rrf_set_profiling.argtypes = [vp, i32]
    lib.rrf_get_profile.argtypes = [vp, C.POINTER(rrf_profile_t)]
    lib.rrf_measure_peak.argtypes = [vp, i32, C.c_double, C.POINTER(C.c_double)]
    lib.rrf_status_string.argtypes = [C.c_int]
    lib.rrf_status_string.restype = C.c_char_p
    for name in EXPORTS:
        if name != "rrf_status_string":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


class RrfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {rrf_status_string(status)} ({status})")


def rrf_status_string(status: int) -> str:
    return load().rrf_status_string(int(status)).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float64:
        return RRF_F64
    if t.dtype == torch.float32:
        return RRF_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _rowmajor(t: torch.Tensor, name: str) -> int:
    """Leading dimension of a 2-D row-major tensor (last stride 1)."""
    if t.dim() != 2 or t.stride(1) != 1 or not t.is_cuda:
        raise ValueError(f"{name} must be a 2-D CUDA tensor with unit inner stride")
    return t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))


def _empty(rows: int, cols: int, dtype, device) -> torch.Tensor:
    """rows x cols view whose leading dimension keeps every row 16-byte aligned."""
    pad = 2 if dtype == torch.float64 else 4
    ld = (cols + pad - 1) // pad * pad
    return torch.empty((rows, ld), dtype=dtype, device=device)[:, :cols]


def rrf_create(device: int = 0) -> C.c_void_p:
    h = C.c_void_p()
    s = load().rrf_create(C.byref(h), int(device))
    if s != RRF_OK:
        raise RrfError(s, "rrf_create")
    return h


def rrf_destroy(h) -> None:
    load().rrf_destroy(h)


def make_params(dtype: int, m: int, n: int, b: int, tol: float, max_rank: int, relative: bool = True,
                estimator: int = 0, flags: int = 0, seed: int = 0, panel_ctas: int = 0, gate: int = 0) -> rrf_params_t:
    return rrf_params_t(dtype=dtype, b=b, max_rank=max_rank, estimator=estimator, m=m, n=n, tol=tol,
                        tol_is_relative=1 if relative else 0, flags=flags, seed=seed,
                        tune_panel_ctas=panel_ctas, tune_gate=gate)


def rrf_workspace_bytes(p: rrf_params_t) -> int:
    out = C.c_size_t()
    s = load().rrf_workspace_bytes(C.byref(p), C.byref(out))
    if s != RRF_OK:
        raise RrfError(s, "rrf_workspace_bytes")
    return out.value


@dataclass
class RunResult:
    status: int
    k: int
    steps: int
    normA2: float
    sigma2: float
    E_sub: float
    E_dir: float
    E_sub_trace: list
    E_dir_trace: list
    V: torch.Tensor   # m x max_rank buffer; columns [:k] are defined
    T: torch.Tensor   # b x max_rank
    B: torch.Tensor   # max_rank x n buffer; rows [:k] are defined
    queues: int = 1   # schedule used: 1 sequential, 2 look-ahead
    panel_ctas: int = 0
    fused_samples: int = 0
    extra_samples: int = 0
    kernel_launches: int = 0
    E_est_trace: list = None   # estimators 2, 3: estimate of the residual before each sampled panel


def rrf_run(h, A: torch.Tensor, b: int, tol: float, max_rank: int, omegaT: torch.Tensor | None = None,
            relative: bool = True, estimator: int = 0, flags: int = 0, seed: int = 0,
            V: torch.Tensor | None = None, T: torch.Tensor | None = None, B: torch.Tensor | None = None,
            workspace: torch.Tensor | None = None, check: bool = True, panel_ctas: int = 0, gate: int = 0) -> RunResult:
    """Algorithm 2 on the device.  `omegaT` is max_rank x n (row j = j-th Gaussian vector) or None."""
    lib = load()
    m, n = A.shape
    dt = _dtype_code(A)
    p = make_params(dt, m, n, b, tol, max_rank, relative, estimator, flags, seed, panel_ctas, gate)
    need = C.c_size_t()
    s = lib.rrf_workspace_bytes(C.byref(p), C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_workspace_bytes")
    dev = A.device
    if V is None:
        V = _empty(m, max_rank, A.dtype, dev)
    if T is None:
        T = torch.empty((b, max_rank), dtype=A.dtype, device=dev)   # leading dimension max_rank
    no_update = bool(flags & RRF_FLAG_NO_UPDATE)
    if B is None and not no_update:
        B = _empty(max_rank, n, A.dtype, dev)
    if workspace is None:
        workspace = torch.empty(need.value, dtype=torch.uint8, device=dev)
    res = rrf_result_t()
    steps = max_rank // b
    tr_sub = (C.c_double * steps)()
    tr_dir = (C.c_double * steps)()
    tr_est = (C.c_double * (steps + 1))()
    om_ptr, ldo = (None, 0) if omegaT is None else (C.c_void_p(omegaT.data_ptr()), _rowmajor(omegaT, "omegaT"))
    s = lib.rrf_run(h, C.byref(p), C.c_void_p(A.data_ptr()), _rowmajor(A, "A"), om_ptr, ldo,
                    C.c_void_p(V.data_ptr()), _rowmajor(V, "V"), C.c_void_p(T.data_ptr()),
                    None if B is None else C.c_void_p(B.data_ptr()), 0 if B is None else _rowmajor(B, "B"),
                    C.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(), C.byref(res), tr_sub, tr_dir, tr_est)
    if check and s < 0:
        raise RrfError(s, "rrf_run")
    return RunResult(res.status, res.k, res.steps, res.normA2, res.sigma2, res.E_sub, res.E_dir,
                     list(tr_sub)[:res.steps], list(tr_dir)[:res.steps], V, T, B, res.queues, res.panel_ctas,
                     res.fused_samples, res.extra_samples, res.kernel_launches, list(tr_est)[:res.n_est])


def rrf_resume(h, W: torch.Tensor, prev: RunResult, b: int, max_rank: int, omegaT: torch.Tensor | None = None,
               seed: int = 0, flags: int = 0) -> RunResult:
    """Carry on a run that ended at its rank cap (status RRF_MAX_RANK_REACHED) up to the larger cap `max_rank`.

    `W` is the matrix the earlier run worked on IN PLACE (RRF_FLAG_INPLACE): its rows [:prev.k] hold B, the rest is
    the residual.  The blocks still to come are Algorithm 2 on that residual W[prev.k:, :] with the absolute
    tolerance of the first run, so this is one more rrf_run call on offset pointers: V and B continue below and to
    the right of what exists, the sample vectors continue at number prev.k (`omegaT`, max_rank x n, or the built-in
    generator from `seed`).  Returns the merged result (V: m x max_rank, T: b x max_rank, B: rows of W)."""
    k0 = prev.k
    m, n = W.shape
    if prev.status != RRF_MAX_RANK_REACHED or max_rank <= k0 or max_rank % b or k0 % b:
        raise ValueError("rrf_resume continues a run that stopped at its cap, up to a larger cap that is a multiple of b")
    V = _empty(m, max_rank, W.dtype, W.device)
    V[:, :k0] = prev.V[:, :k0]
    V[:k0, k0:].zero_()                      # the new blocks' reflectors start at row k0
    if omegaT is None:
        om = rrf_fill_omega(h, n, max_rank - k0, seed, dtype=W.dtype, first_vec=k0, device=W.device)
    else:
        om = omegaT[k0:max_rank]
    r = rrf_run(h, W[k0:], b, float(prev.sigma2) ** 0.5, max_rank - k0, omegaT=om, relative=False,
                flags=flags | RRF_FLAG_INPLACE, V=V[k0:, k0:], B=W[k0:max_rank])
    T = torch.cat([prev.T[:, :k0], r.T], dim=1)
    return RunResult(r.status, k0 + r.k, prev.steps + r.steps, prev.normA2, prev.sigma2, r.E_sub, r.E_dir,
                     prev.E_sub_trace + r.E_sub_trace, prev.E_dir_trace + r.E_dir_trace, V, T, W[:max_rank], r.queues,
                     r.panel_ctas, prev.fused_samples + r.fused_samples, prev.extra_samples + r.extra_samples,
                     prev.kernel_launches + r.kernel_launches, [])


def _colmajor(t: torch.Tensor, name: str) -> int:
    """Leading dimension of a 2-D column-major tensor (first stride 1)."""
    if t.dim() != 2 or t.stride(0) != 1 or not t.is_cuda:
        raise ValueError(f"{name} must be a 2-D CUDA tensor with unit stride along its columns")
    return t.stride(1) if t.shape[1] > 1 else max(t.shape[0], t.stride(1))


def rrf_run_colmajor(h, A: torch.Tensor, b: int, tol: float, max_rank: int, omega: torch.Tensor | None = None,
                     relative: bool = True, estimator: int = 0, flags: int = 0, seed: int = 0,
                     check: bool = True) -> RunResult:
    """Algorithm 2 on column-major storage.  `A` (m x n) and `omega` (n x max_rank) are tensors whose FIRST stride
    is 1 (e.g. `X.t()` of a contiguous X); V (m x max_rank), T (b x max_rank) and B (max_rank x n) come back as
    such tensors too."""
    lib = load()
    m, n = A.shape
    dt = _dtype_code(A)
    p = make_params(dt, m, n, b, tol, max_rank, relative, estimator, flags, seed)
    need = C.c_size_t()
    s = lib.rrf_colmajor_workspace_bytes(C.byref(p), C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_colmajor_workspace_bytes")
    dev = A.device
    V = torch.empty((max_rank, m), dtype=A.dtype, device=dev).t()
    T = torch.empty((max_rank, b), dtype=A.dtype, device=dev).t()
    B = None if flags & RRF_FLAG_NO_UPDATE else torch.empty((n, max_rank), dtype=A.dtype, device=dev).t()
    workspace = torch.empty(need.value, dtype=torch.uint8, device=dev)
    res = rrf_result_t()
    steps = max_rank // b
    tr_sub = (C.c_double * steps)()
    tr_dir = (C.c_double * steps)()
    tr_est = (C.c_double * (steps + 1))()
    om_ptr, ldo = (None, 0) if omega is None else (C.c_void_p(omega.data_ptr()), _colmajor(omega, "omega"))
    s = lib.rrf_run_colmajor(h, C.byref(p), C.c_void_p(A.data_ptr()), _colmajor(A, "A"), om_ptr, ldo,
                             C.c_void_p(V.data_ptr()), _colmajor(V, "V"), C.c_void_p(T.data_ptr()),
                             None if B is None else C.c_void_p(B.data_ptr()), 0 if B is None else _colmajor(B, "B"),
                             C.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(), C.byref(res),
                             tr_sub, tr_dir, tr_est)
    if check and s < 0:
        raise RrfError(s, "rrf_run_colmajor")
    return RunResult(res.status, res.k, res.steps, res.normA2, res.sigma2, res.E_sub, res.E_dir,
                     list(tr_sub)[:res.steps], list(tr_dir)[:res.steps], V, T, B, res.queues, res.panel_ctas,
                     res.fused_samples, res.extra_samples, res.kernel_launches, list(tr_est)[:res.n_est])


def rrf_transpose(h, src: torch.Tensor) -> torch.Tensor:
    """A new row-major tensor holding src^T (src row-major)."""
    rows, cols = src.shape
    dst = _empty(cols, rows, src.dtype, src.device)
    s = load().rrf_transpose(h, _dtype_code(src), rows, cols, C.c_void_p(src.data_ptr()), _rowmajor(src, "src"),
                             C.c_void_p(dst.data_ptr()), _rowmajor(dst, "dst"), _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_transpose")
    return dst


def rrf_panel_qr(h, Y: torch.Tensor, tree: bool = False, blocked: bool = False):
    """Householder QR of a tall panel: returns (V, T) as the library writes them
    (`tree`: rrf_panel_qr_tree, `blocked`: rrf_panel_qr_blocked)."""
    lib = load()
    rows, b = Y.shape
    dt = _dtype_code(Y)
    need = C.c_size_t()
    s = lib.rrf_panel_workspace_bytes(dt, rows, b, C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_panel_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=Y.device)
    V = torch.empty_like(Y)
    T = torch.empty((b, b), dtype=Y.dtype, device=Y.device)
    fn = lib.rrf_panel_qr_tree if tree else (lib.rrf_panel_qr_blocked if blocked else lib.rrf_panel_qr)
    s = fn(h, dt, rows, b, C.c_void_p(Y.data_ptr()), _rowmajor(Y, "Y"), C.c_void_p(V.data_ptr()),
                         _rowmajor(V, "V"), C.c_void_p(T.data_ptr()), b, C.c_void_p(ws.data_ptr()), ws.numel(),
                         _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_panel_qr")
    s = lib.rrf_last_status(h, _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_panel_qr (device)")
    return V, T


def rrf_panel_qr_static(Y: torch.Tensor, V: torch.Tensor, T: torch.Tensor) -> int:
    """Panel QR through the entry point that allocates nothing: no handle, no workspace.

    The caller owns Y (rows x b), V (rows x b) and T (b x b); returns the status the call reports
    (it synchronises the current stream).  Calls that overlap on the GPU race on the library's
    built-in scratch array.
    """
    rows, b = Y.shape
    return load().rrf_panel_qr_static(_dtype_code(Y), rows, b, C.c_void_p(Y.data_ptr()), _rowmajor(Y, "Y"),
                                      C.c_void_p(V.data_ptr()), _rowmajor(V, "V"), C.c_void_p(T.data_ptr()),
                                      _rowmajor(T, "T"), _stream())


def _apply(fn_name: str, h, V: torch.Tensor, T: torch.Tensor, b: int, k: int, Cm: torch.Tensor) -> torch.Tensor:
    lib = load()
    m, ncols = Cm.shape
    dt = _dtype_code(Cm)
    need = C.c_size_t()
    s = lib.rrf_apply_workspace_bytes(dt, m, ncols, b, C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_apply_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=Cm.device)
    s = getattr(lib, fn_name)(h, dt, m, b, k, C.c_void_p(V.data_ptr()), _rowmajor(V, "V"), C.c_void_p(T.data_ptr()),
                              _rowmajor(T, "T"), C.c_void_p(Cm.data_ptr()), _rowmajor(Cm, "C"), ncols,
                              C.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    if s != RRF_OK:
        raise RrfError(s, fn_name)
    torch.cuda.current_stream().synchronize()   # the workspace is freed on return
    return Cm


def rrf_apply_qt(h, V, T, b: int, k: int, Cm: torch.Tensor) -> torch.Tensor:
    """C <- Q^T C in place."""
    return _apply("rrf_apply_qt", h, V, T, b, k, Cm)


def rrf_apply_q(h, V, T, b: int, k: int, Cm: torch.Tensor) -> torch.Tensor:
    """C <- Q C in place."""
    return _apply("rrf_apply_q", h, V, T, b, k, Cm)


def rrf_form_q(h, V: torch.Tensor, T: torch.Tensor, b: int, k: int) -> torch.Tensor:
    """Explicit m x k orthonormal basis."""
    lib = load()
    m = V.shape[0]
    dt = _dtype_code(V)
    Q = _empty(m, k, V.dtype, V.device)
    need = C.c_size_t()
    s = lib.rrf_apply_workspace_bytes(dt, m, k, b, C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_apply_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=V.device)
    s = lib.rrf_form_q(h, dt, m, b, k, C.c_void_p(V.data_ptr()), _rowmajor(V, "V"), C.c_void_p(T.data_ptr()),
                       _rowmajor(T, "T"), C.c_void_p(Q.data_ptr()), _rowmajor(Q, "Q"), C.c_void_p(ws.data_ptr()),
                       ws.numel(), _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_form_q")
    torch.cuda.current_stream().synchronize()
    return Q


def rrf_subspace_transfer(h, V_old, T_old, k_old: int, V_new, T_new, k_new: int, b: int, M: torch.Tensor) -> torch.Tensor:
    """Mout (k_new x n) = Q_new^T (Q_old M) for M (k_old x n)."""
    lib = load()
    m, ncols = V_old.shape[0], M.shape[1]
    dt = _dtype_code(M)
    out = _empty(k_new, ncols, M.dtype, M.device)
    need = C.c_size_t()
    s = lib.rrf_transfer_workspace_bytes(dt, m, ncols, b, C.byref(need))
    if s != RRF_OK:
        raise RrfError(s, "rrf_transfer_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=M.device)
    s = lib.rrf_subspace_transfer(h, dt, m, b, k_old, C.c_void_p(V_old.data_ptr()), _rowmajor(V_old, "V_old"),
                                  C.c_void_p(T_old.data_ptr()), _rowmajor(T_old, "T_old"), k_new,
                                  C.c_void_p(V_new.data_ptr()), _rowmajor(V_new, "V_new"),
                                  C.c_void_p(T_new.data_ptr()), _rowmajor(T_new, "T_new"),
                                  C.c_void_p(M.data_ptr()), _rowmajor(M, "M"), ncols,
                                  C.c_void_p(out.data_ptr()), _rowmajor(out, "Mout"), C.c_void_p(ws.data_ptr()),
                                  ws.numel(), _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_subspace_transfer")
    torch.cuda.current_stream().synchronize()
    return out


def rrf_fill_omega(h, n: int, nvec: int, seed: int, dtype=torch.float64, first_vec: int = 0,
                   device="cuda") -> torch.Tensor:
    """nvec x n Gaussian matrix (OmegaT layout) from the library's counter-based generator."""
    lib = load()
    pad = 2 if dtype == torch.float64 else 4
    ldo = (n + pad - 1) // pad * pad
    buf = torch.empty((nvec, ldo), dtype=dtype, device=device)
    O = buf[:, :n]
    s = lib.rrf_fill_omega(h, _dtype_code(O), seed, n, nvec, first_vec, C.c_void_p(O.data_ptr()), ldo, _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_fill_omega")
    return O


def rrf_last_status(h) -> int:
    return load().rrf_last_status(h, _stream())


def rrf_set_single_engine(h, engine: int, chunk_tiles: int = 0) -> None:
    s = load().rrf_set_single_engine(h, int(engine), int(chunk_tiles))
    if s != 0:
        raise RrfError(s, "rrf_set_single_engine")


def rrf_set_profiling(h, enable: bool) -> None:
    load().rrf_set_profiling(h, 1 if enable else 0)


def rrf_get_profile(h) -> dict:
    """{phase: (milliseconds, launches)} of the last profiled rrf_run."""
    p = rrf_profile_t()
    s = load().rrf_get_profile(h, C.byref(p))
    if s != RRF_OK:
        raise RrfError(s, "rrf_get_profile")
    return {name: (p.ms[i], p.launches[i]) for i, name in enumerate(RRF_PHASES)}


def rrf_measure_peak(h, kind: int, ms: float = 50.0) -> float:
    """Attainable TFLOP/s of one pipe: 0 f64 mma, 1 f64 FMA, 2 f32 FMA, 3 tf32 mma."""
    out = C.c_double()
    s = load().rrf_measure_peak(h, kind, ms, C.byref(out))
    if s != RRF_OK:
        raise RrfError(s, "rrf_measure_peak")
    return out.value


def rrf_selftest_timeout(h, limit_ms: float = 50.0) -> int:
    """Make a bounded device-side wait run out; returns the status the device recorded."""
    s = load().rrf_selftest_timeout(h, limit_ms, _stream())
    if s != RRF_OK:
        raise RrfError(s, "rrf_selftest_timeout")
    return rrf_last_status(h)
