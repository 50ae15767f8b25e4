"""Resuming a run that ended at its rank cap (Algorithm 2 carried on from block `start`): the blocks still to come
are the algorithm on the residual rows with the first run's absolute tolerance, so the continued run must land
where the oracle's single run with the larger cap lands."""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf, workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f64": dict(rel=1e-10, orth=1e-12), "f32": dict(rel=1e-4, orth=1e-5)}


@pytest.fixture(scope="module")
def h():
    hd = rrf.rrf_create(0)
    yield hd
    rrf.rrf_destroy(hd)


def _relmax(x, ref):
    return np.max(np.abs(x - ref)) / np.max(np.abs(ref))


@pytest.mark.parametrize("name,kw,first_cap", [
    ("cfg2", dict(m=1536, n=1280, max_rank=512), 128),
    ("cfg1", dict(m=900, n=700, max_rank=256), 64),
    ("cfg3", dict(m=1024, n=1024, max_rank=512), 96),
    ("cfg4", dict(m=1024, n=2752, max_rank=256, rank=128), 64),    # single precision
])
@pytest.mark.parametrize("sched", [rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES])
def test_resumed_run_matches_the_oracles_single_run(h, name, kw, first_cap, sched):
    w = wl.CONFIGS[name].scaled(**kw)
    A, _ = wl.make_matrix(w)
    A = np.ascontiguousarray(A.astype(w.np_dtype))
    Om = np.ascontiguousarray(wl.make_omega(w).astype(w.np_dtype))
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, w.tol, w.max_rank)
    assert o.k > first_cap                      # the first cap really cuts the run short
    W = torch.from_numpy(A).cuda()
    g1 = rrf.rrf_run(h, W, w.b, w.tol, first_cap, omegaT=dOmT[:first_cap], flags=sched | rrf.RRF_FLAG_INPLACE, B=W[:first_cap])
    assert g1.status == rrf.RRF_MAX_RANK_REACHED and g1.k == first_cap
    g = rrf.rrf_resume(h, W, g1, w.b, w.max_rank, omegaT=dOmT, flags=sched)
    assert (g.k, g.steps, g.status) == (o.k, o.steps, o.status)
    assert np.isclose(g.normA2, o.normA2, rtol=1e-12 if w.dtype == "f64" else 1e-6)
    k, b, tol = g.k, w.b, TOL[w.dtype]
    B = g.B[:k].cpu().numpy().astype(np.float64)
    assert _relmax(B, o.B) <= tol["rel"]
    Qg = rrf.rrf_form_q(h, g.V, g.T, b, k).cpu().numpy().astype(np.float64)
    Qo = orc.form_q(o.V, o.T, b)
    assert np.linalg.norm(Qg.T @ Qg - np.eye(k)) <= tol["orth"]
    assert _relmax(Qg @ B, Qo @ o.B) <= 10 * tol["rel"]
    # both stopping traces run on through the seam
    assert len(g.E_dir_trace) == len(o.E_dir)
    u = 1.1e-16 if w.dtype == "f64" else 6e-8
    d = 2 * max(w.m, w.n) * u * np.sqrt(o.normA2)        # Frobenius size of the residual's rounding noise
    for a, c in zip(g.E_dir_trace, o.E_dir):
        assert abs(a - c) <= (1e-6 if w.dtype == "f64" else 1e-3) * c + 2 * np.sqrt(c) * d + d * d, (a, c)
    assert np.linalg.norm(A.astype(np.float64) - Qg @ B) <= w.tol * np.sqrt(o.normA2) * (1 + 1e-6) or o.status != orc.RRF_OK


def test_resume_with_the_builtin_generator_continues_its_vector_numbers(h):
    # seed-drawn sample vectors: the resumed blocks must use vectors k0, k0 + 1, ... of the same sequence
    w = wl.CONFIGS["cfg2"].scaled(m=1536, n=1280, max_rank=512)
    A, _ = wl.make_matrix(w)
    W1 = torch.from_numpy(A).cuda()
    one = rrf.rrf_run(h, W1, w.b, w.tol, w.max_rank, seed=11, flags=rrf.RRF_FLAG_INPLACE, B=W1[:w.max_rank])
    W2 = torch.from_numpy(A).cuda()
    g1 = rrf.rrf_run(h, W2, w.b, w.tol, 128, seed=11, flags=rrf.RRF_FLAG_INPLACE, B=W2[:128])
    g = rrf.rrf_resume(h, W2, g1, w.b, w.max_rank, seed=11)
    assert g.k == one.k and g.status == one.status and one.k > 128
    k = g.k
    B1, B2 = one.B[:k].cpu().numpy(), g.B[:k].cpu().numpy()
    assert _relmax(B2, B1) <= 1e-10
    assert torch.equal(g.V[:, :128], one.V[:, :128]) and torch.equal(g.T[:, :128], one.T[:, :128])


def test_resume_rejects_a_run_that_did_not_stop_at_its_cap(h):
    w = wl.CONFIGS["cfg1"].scaled(m=512, n=384, max_rank=128)
    A, _ = wl.make_matrix(w)
    W = torch.from_numpy(A).cuda()
    g1 = rrf.rrf_run(h, W, w.b, 1e-2, 128, seed=1, flags=rrf.RRF_FLAG_INPLACE, B=W[:128])
    assert g1.status == rrf.RRF_OK
    with pytest.raises(ValueError):
        rrf.rrf_resume(h, W, g1, w.b, 256, seed=1)
