"""Column-major entry points (rrf_run_colmajor, rrf_transpose) through the C ABI.

The column-major run must return exactly what the row-major run returns for the same matrices (it is the same
arithmetic between two changes of storage), and - independently of that - its B, its first reflector block and
k must match the oracle within the bars of the row-major parity tests."""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf, workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f64": 1e-10, "f32": 1e-4}


@pytest.fixture(scope="module")
def h():
    hd = rrf.rrf_create(0)
    yield hd
    rrf.rrf_destroy(hd)


def _colmajor(x: np.ndarray, ld_extra: int = 0) -> torch.Tensor:
    """Device tensor with the shape and values of x, stored column by column with leading dimension rows + ld_extra."""
    r, c = x.shape
    buf = torch.zeros((c, r + ld_extra), dtype=torch.from_numpy(x).dtype, device="cuda")
    buf[:, :r] = torch.from_numpy(np.ascontiguousarray(x.T)).cuda()
    return buf[:, :r].t()


def _relmax(x, ref):
    s = np.max(np.abs(ref))
    return np.max(np.abs(x - ref)) / (s if s > 0 else 1.0)


@pytest.mark.parametrize("rows,cols", [(1, 1), (31, 33), (32, 32), (257, 70), (1000, 1111), (5, 4097)])
@pytest.mark.parametrize("dtype", [torch.float64, torch.float32])
def test_transpose_is_exact(h, rows, cols, dtype):
    g = torch.Generator(device="cpu").manual_seed(rows * 7919 + cols)
    src = torch.randn((rows, cols + 3), generator=g, dtype=dtype).cuda()[:, :cols]   # leading dimension > cols
    dst = rrf.rrf_transpose(h, src)
    assert dst.shape == (cols, rows)
    assert torch.equal(dst, src.t())


def test_transpose_rejects_bad_arguments(h):
    lib = rrf.load()
    x = torch.zeros((8, 8), dtype=torch.float64, device="cuda")
    y = torch.zeros((8, 8), dtype=torch.float64, device="cuda")
    import ctypes as C
    px, py = C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr())
    assert lib.rrf_transpose(h, 0, 8, 8, px, 7, py, 8, None) == rrf.RRF_ERR_INVALID_ARG    # lds < cols
    assert lib.rrf_transpose(h, 0, 8, 8, px, 8, py, 7, None) == rrf.RRF_ERR_INVALID_ARG    # ldd < rows
    assert lib.rrf_transpose(h, 0, 8, 8, px, 8, px, 8, None) == rrf.RRF_ERR_INVALID_ARG    # in place
    assert lib.rrf_transpose(h, 5, 8, 8, px, 8, py, 8, None) == rrf.RRF_ERR_INVALID_ARG    # dtype
    assert lib.rrf_transpose(h, 0, 0, 8, None, 8, None, 8, None) == rrf.RRF_OK             # empty


@pytest.mark.parametrize("name,kw,ld_extra", [
    ("cfg1", dict(m=512, n=384, max_rank=128), 0),
    ("cfg2", dict(m=1000, n=1111, max_rank=256), 5),          # ragged in both dimensions, odd leading dimensions
    ("cfg3", dict(m=1024, n=1024, max_rank=512), 0),
    ("cfg4", dict(m=1024, n=2752, max_rank=256, rank=64), 3),  # single precision
    ("cfg1", dict(m=900, n=700, max_rank=256, b=128), 1),
])
def test_colmajor_run_matches_oracle_and_row_major_run(h, name, kw, ld_extra):
    w = wl.CONFIGS[name].scaled(**kw)
    A, _ = wl.make_matrix(w)
    A = np.ascontiguousarray(A.astype(w.np_dtype))
    Om = np.ascontiguousarray(wl.make_omega(w).astype(w.np_dtype))          # n x max_rank
    dA = _colmajor(A, ld_extra)
    pad = 2 if w.dtype == "f64" else 4
    dOm = _colmajor(Om, (-w.n) % pad)                                       # leading dimension a multiple of 16 bytes
    gc = rrf.rrf_run_colmajor(h, dA, w.b, w.tol, w.max_rank, omega=dOm)
    assert torch.equal(dA, torch.from_numpy(A).cuda())                      # the input is left alone
    o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, w.tol, w.max_rank)
    assert (gc.k, gc.steps, gc.status) == (o.k, o.steps, o.status)
    k, b = gc.k, w.b
    assert gc.V.stride(0) == 1 and gc.B.stride(0) == 1 and gc.T.stride(0) == 1
    B = gc.B[:k].cpu().numpy().astype(np.float64)
    assert _relmax(B, o.B) <= TOL[w.dtype]
    V0 = gc.V[:, :b].cpu().numpy().astype(np.float64)
    T0 = gc.T[:, :b].cpu().numpy().astype(np.float64)
    assert _relmax(V0, o.V[:, :b]) <= 10 * TOL[w.dtype]
    assert _relmax(T0, o.T[:, :b]) <= 10 * TOL[w.dtype]
    # the row-major call on the same matrices, working in place like the column-major call does inside
    dAr = torch.from_numpy(A).cuda()
    if (w.n % pad) != 0:
        buf = torch.zeros((w.m, w.n + (-w.n) % pad), dtype=dAr.dtype, device="cuda")
        buf[:, :w.n] = dAr
        dAr = buf[:, :w.n]
    gr = rrf.rrf_run(h, dAr, w.b, w.tol, w.max_rank, omegaT=dOm.t(), flags=rrf.RRF_FLAG_INPLACE, B=dAr)
    assert gr.k == k and gr.queues == gc.queues
    assert torch.equal(gc.V[:, :k], gr.V[:, :k])
    assert torch.equal(gc.T[:, :k], gr.T[:, :k])
    assert torch.equal(gc.B[:k], dAr[:k])
    assert gc.E_dir_trace == gr.E_dir_trace and gc.E_sub_trace == gr.E_sub_trace


def test_colmajor_zero_matrix_and_the_variant_that_leaves_A_unchanged(h):
    z = _colmajor(np.zeros((256, 192)))
    g = rrf.rrf_run_colmajor(h, z, 16, 1e-6, 64, seed=3)
    assert g.k == 0 and g.status == rrf.RRF_OK
    w = wl.CONFIGS["cfg1"].scaled(m=900, n=700, max_rank=256)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w)
    tol = 1e-3
    g2 = rrf.rrf_run_colmajor(h, _colmajor(A, 2), w.b, tol, w.max_rank, omega=_colmajor(Om), estimator=2,
                              flags=rrf.RRF_FLAG_NO_UPDATE)
    o2 = orc.rrf(A, Om, w.b, tol, w.max_rank, estimator="sampled_fro", schedule="a_unchanged")
    assert g2.B is None and (g2.k, g2.steps, g2.status) == (o2.k, o2.steps, o2.status) and 0 < g2.k < w.max_rank
    assert np.allclose(g2.E_est_trace, o2.E_est, rtol=1e-9, atol=1e-15 * o2.normA2)
    gr = rrf.rrf_run(h, torch.from_numpy(A).cuda(), w.b, tol, w.max_rank, omegaT=_colmajor(Om).t(), estimator=2,
                     flags=rrf.RRF_FLAG_NO_UPDATE)
    assert gr.k == g2.k and torch.equal(g2.V[:, :gr.k], gr.V[:, :gr.k]) and torch.equal(g2.T[:, :gr.k], gr.T[:, :gr.k])


def test_colmajor_argument_checks(h):
    A = _colmajor(np.ones((128, 96)))
    with pytest.raises(rrf.RrfError):
        rrf.rrf_run_colmajor(h, A, 16, 1e-6, 64, flags=rrf.RRF_FLAG_INPLACE)
