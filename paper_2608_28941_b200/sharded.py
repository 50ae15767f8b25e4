"""Column-sharded driver of the range finder: one process per GPU, one all-reduce of the m_i x b panel per block.

The outlook of the paper names distributed matrix layouts as the extension a training framework needs.  With the
columns of A split over the ranks (A = [A_1 ... A_P]) and the rows of Omega split to match, block step i is

    Y_i = sum_p W_p[r0:, :] Omega_{i,p}        (rrf_sample_panel on every rank, then ONE all-reduce: the exchange)
    (V_i, T_i) = panel QR of Y_i               (rrf_panel_qr, the same on every rank: nothing to broadcast)
    W_p[r0:, :] <- Q_i^T W_p[r0:, :]           (rrf_apply_qt, local)
    E = sum_p ||W_p[r0+b:, :]||_F^2            (rrf_frobenius_sq, then an all-reduce of two scalars)

Every arithmetic step runs in the library's kernels; this module only marshals pointers and calls
torch.distributed (NCCL over NVLink on GPUs) for the two all-reduces.  The loop condition is evaluated on the host
once per block (the reduced scalars have to be read anyway).  With `group=None` and no initialised process group
it runs as a single rank.  V, T, k and the traces come out identical on every rank; B is the rank's column block.

No kernel reads another GPU's memory: remote data arrives through the all-reduce into this GPU's own memory.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import torch
import torch.distributed as dist

from . import rrf


@dataclass
class ShardedResult:
    k: int
    status: int
    steps: int
    normA2: float
    E_dir_trace: list
    E_sub_trace: list
    V: torch.Tensor      # m x max_rank, replicated
    T: torch.Tensor      # b x max_rank, replicated
    B: torch.Tensor      # max_rank x n_local: this rank's columns of B (rows [:k] defined)


def _allreduce(t: torch.Tensor, group) -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)


def rrf_run_column_sharded(h, A_loc: torch.Tensor, omegaT_loc: torch.Tensor, b: int, tol: float, max_rank: int,
                           group=None, relative: bool = True, fixed_rank: bool = False) -> ShardedResult:
    """A_loc: m x n_p (this rank's columns of A); omegaT_loc: max_rank x n_p (the matching columns of Omega^T)."""
    lib = rrf.load()
    m, n_p = A_loc.shape
    dt = rrf._dtype_code(A_loc)
    dev, tdt = A_loc.device, A_loc.dtype
    st = rrf._stream()
    W = rrf._empty(m, n_p, tdt, dev)
    W.copy_(A_loc)
    V = torch.zeros((m, max_rank), dtype=tdt, device=dev)
    T = torch.zeros((b, max_rank), dtype=tdt, device=dev)
    Y = torch.empty((m, b), dtype=tdt, device=dev)
    Vi = torch.empty((m, b), dtype=tdt, device=dev)
    Ti = torch.empty((b, b), dtype=tdt, device=dev)
    scal = torch.zeros(2, dtype=torch.float64, device=dev)
    need = C.c_size_t()
    sizes = []
    for fn, args in ((lib.rrf_sample_workspace_bytes, (dt, m, b)), (lib.rrf_panel_workspace_bytes, (dt, m, b)),
                     (lib.rrf_apply_workspace_bytes, (dt, m, n_p, b))):
        s = fn(*args, C.byref(need))
        if s != rrf.RRF_OK:
            raise rrf.RrfError(s, fn.__name__)
        sizes.append(need.value)
    ws = torch.empty(max(max(sizes), 8192), dtype=torch.uint8, device=dev)
    wsp, wsn = C.c_void_p(ws.data_ptr()), ws.numel()

    def check(s, where):
        if s != rrf.RRF_OK:
            raise rrf.RrfError(s, where)

    def frob(view: torch.Tensor, slot: int):
        rows = view.shape[0]
        check(lib.rrf_frobenius_sq(h, dt, rows, n_p, C.c_void_p(view.data_ptr()) if rows > 0 else None, W.stride(0),
                                   C.c_void_p(scal[slot:].data_ptr()), wsp, wsn, st), "rrf_frobenius_sq")

    frob(W, 0)
    scal[1] = 0.0
    _allreduce(scal, group)
    normA2 = float(scal[0].item())
    sigma2 = tol * tol * normA2 if relative else tol * tol
    E, E_sub = normA2, normA2
    tr_dir, tr_sub = [], []
    met = (not fixed_rank) and not (E > sigma2)
    i = 0
    while not met and (i + 1) * b <= max_rank:
        r0 = i * b
        rows = m - r0
        Wr = W[r0:]
        check(lib.rrf_sample_panel(h, dt, rows, n_p, b, C.c_void_p(Wr.data_ptr()), W.stride(0),
                                   C.c_void_p(omegaT_loc[r0:].data_ptr()), rrf._rowmajor(omegaT_loc, "omegaT"),
                                   C.c_void_p(Y.data_ptr()), wsp, wsn, st), "rrf_sample_panel")
        _allreduce(Y[:rows], group)                                   # the one exchange of a block step
        check(lib.rrf_panel_qr(h, dt, rows, b, C.c_void_p(Y.data_ptr()), b, C.c_void_p(Vi.data_ptr()), b,
                               C.c_void_p(Ti.data_ptr()), b, wsp, wsn, st), "rrf_panel_qr")
        V[r0:, r0:r0 + b].copy_(Vi[:rows])
        T[:, r0:r0 + b].copy_(Ti)
        check(lib.rrf_apply_qt(h, dt, rows, b, b, C.c_void_p(Vi.data_ptr()), b, C.c_void_p(Ti.data_ptr()), b,
                               C.c_void_p(Wr.data_ptr()), W.stride(0), n_p, wsp, wsn, st), "rrf_apply_qt")
        frob(W[r0:r0 + b], 0)
        frob(W[r0 + b:], 1)
        _allreduce(scal, group)
        top, E = (float(x) for x in scal.tolist())                    # host decision, once per block
        E_sub -= top
        tr_sub.append(E_sub)
        tr_dir.append(E)
        met = (not fixed_rank) and not (E > sigma2)
        i += 1
    s = lib.rrf_last_status(h, st)
    if s != rrf.RRF_OK:
        raise rrf.RrfError(s, "rrf_run_column_sharded (device)")
    k = i * b
    status = rrf.RRF_OK if E <= sigma2 else rrf.RRF_MAX_RANK_REACHED
    return ShardedResult(k, status, i, normA2, tr_dir, tr_sub, V, T, W[:max_rank])
