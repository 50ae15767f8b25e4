"""Seeded random sweep of shapes, block sizes, schedules and sampling modes against the oracle.

Four hundred small problems (ragged sizes, ranks from 1 to full, tolerances over eight decades, both precisions, both
estimators, fixed-rank mode, one and two queues, every sampling mode).  Compared: k (unless the oracle's own
stopping quantity sits within 1e-6 / 1e-2 of the threshold, where either answer is right), Q^T Q, and B and Q B
block by block.  Block i is sampled from a residual of relative size sqrt(E_{i-1}/E_0) (E_{i-2} under the
look-ahead schedule, which samples one update early) that carries rounding noise of the size of u ||A||, so its
rows of B are held to the plain bar times that amplification.  Which blocks are instead sampled from pure rounding
noise is decided from the INPUT: the generated rank is known, and a block that starts at or beyond it (or whose
residual, by the oracle's own trace, is within a factor 1e4 / 1e2 of the rounding floor) has no unique B or Q; for
those the test checks what is unique: the residual norm and the orthogonality.  Inside a block, rows at or beyond
the generated rank are not compared, and rows are compared up to sign from the first reflector whose pivot lies
within the rounding noise of its sampled panel (the Householder sign rule is discontinuous there)."""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf

pytestmark = pytest.mark.gpu


def _relmax(x, ref):
    s = np.max(np.abs(ref)) if ref.size else 1.0
    return np.max(np.abs(x - ref)) / (s if s > 0 else 1.0) if ref.size else 0.0


def _pad(x, mult):
    r, c = x.shape
    ld = (c + mult - 1) // mult * mult
    buf = torch.zeros((r, ld), dtype=torch.from_numpy(x).dtype, device="cuda")
    buf[:, :c] = torch.from_numpy(x).cuda()
    return buf[:, :c]


@pytest.mark.parametrize("seed", range(400))
def test_random_problem(seed):
    rng = np.random.default_rng(9000 + seed)
    h = rrf.rrf_create(0)
    try:
        dt = "f64" if rng.random() < 0.75 else "f32"
        b = int(rng.choice([16, 32, 64, 128] if dt == "f64" else [32, 64, 128]))
        maxr = b * int(rng.integers(1, 7))
        m = int(rng.integers(maxr, maxr + 1500))
        n = int(rng.integers(maxr, maxr + 1500))
        rank = int(rng.integers(1, max(2, min(m, n))))
        sv = np.logspace(0, -float(rng.choice([2.0, 6.0, 12.0])), rank)
        A = (rng.standard_normal((m, rank)) * sv) @ rng.standard_normal((rank, n))
        Om = rng.standard_normal((n, maxr))
        est = int(rng.integers(0, 2))
        if est == 0:
            tol = float(10.0 ** rng.uniform(-9, -1)) if dt == "f64" else float(10.0 ** rng.uniform(-4, -1))
        else:   # Algorithm 2 line 9 cancels: keep the tolerance above its rounding floor
            tol = float(10.0 ** rng.uniform(-6, -1)) if dt == "f64" else float(10.0 ** rng.uniform(-2.3, -1))
        sched = int(rng.choice([0, rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES]))
        samp = int(rng.choice([0, rrf.RRF_FLAG_SAMPLE_ALWAYS, rrf.RRF_FLAG_SAMPLE_NEVER]))
        fixed = rrf.RRF_FLAG_FIXED_RANK if rng.random() < 0.15 else 0
        npdt = np.float64 if dt == "f64" else np.float32
        A = np.ascontiguousarray(A.astype(npdt))
        OmT = np.ascontiguousarray(Om.T.astype(npdt))
        mult = 2 if dt == "f64" else 4
        g = rrf.rrf_run(h, _pad(A, mult), b, tol, maxr, omegaT=_pad(OmT, mult), estimator=est, flags=sched | samp | fixed)
        A64, Om64 = A.astype(np.float64), OmT.T.astype(np.float64)
        if fixed:   # the oracle has no fixed-rank switch: tolerance 0 on the residual norm runs it to the cap
            o = orc.rrf(A64, Om64, b, 0.0, maxr, estimator="direct")
        else:
            o = orc.rrf(A64, Om64, b, tol, maxr, estimator="direct" if est == 0 else "subtractive")
        trace = o.E_dir if est == 0 else o.E_sub
        near = 1e-6 if dt == "f64" else 1e-2
        marginal = (not fixed) and any(abs(e / max(o.normA2 * tol * tol, 1e-300) - 1.0) < near for e in trace)
        if not marginal:
            assert g.k == o.k, (g.k, o.k)
        k = min(g.k, o.k)
        if k == 0:
            return
        B = g.B[:k].cpu().numpy().astype(np.float64)
        Q = rrf.rrf_form_q(h, g.V, g.T, b, k).cpu().numpy().astype(np.float64)
        orth = np.linalg.norm(Q.T @ Q - np.eye(k))
        assert orth <= (1e-11 if dt == "f64" else 1e-4), orth
        bar = 1e-10 if dt == "f64" else 1e-4
        u = 1.1e-16 if dt == "f64" else 6e-8
        Qo = orc.form_q(o.V[:, :k], o.T[:, :k], b)
        E = [o.normA2] + list(o.E_dir)               # E[j]: the oracle's squared residual norm after j blocks
        scaleB = np.max(np.abs(o.B[:k]))
        floor = (1e4 if dt == "f64" else 1e2) * max(m, n) * u
        unique = 0
        signs_fixed = True
        for i in range(k // b):
            lag = 2 if (g.queues == 2 and i >= 2) else 1       # look-ahead: sampled one update earlier
            rel_res = np.sqrt(max(E[i], 0.0) / o.normA2)
            if i * b >= rank or rel_res <= floor:
                break                                          # from here on the blocks are sampled from noise
            amp = np.sqrt(o.normA2 / max(E[i], 1e-300)) * np.sqrt(max(E[max(i - lag + 1, 0)], 0.0) / max(E[i], 1e-300))
            blk = slice(i * b, (i + 1) * b)
            # Inside a block: rows at or beyond the generated rank are reflectors of rounding noise (nothing to
            # compare), and the SIGN of a row is the sign of its reflector's pivot alpha_j (beta = -sign(alpha)
            # ||x||).  The panel's triangular factor is R_i = B_i Omega_i, r_jj = beta_j, alpha_j = beta_j (1 -
            # tau_j); a pivot within the rounding noise of the sampled panel, 64 u max|r_jj|, has no sign the
            # input determines, and the other choice is an equally valid factorisation that also moves the
            # pivots after it - so from the first such row on, rows are compared up to sign.
            rows_i = min(b, rank - i * b)
            Ti = o.T[:, blk]
            rdiag = np.einsum("jn,nj->j", o.B[blk], Om64[:, blk])
            alpha = rdiag * (1.0 - np.diag(Ti))
            noise = 64 * u * np.max(np.abs(rdiag))
            eB = 0.0
            for j in range(rows_i):
                if abs(alpha[j]) <= noise:
                    signs_fixed = False
                dj = np.max(np.abs(B[i * b + j] - o.B[i * b + j]))
                if not signs_fixed:
                    dj = min(dj, np.max(np.abs(B[i * b + j] + o.B[i * b + j])))
                eB = max(eB, dj / scaleB)
            assert eB <= bar * max(1.0, amp), (i, eB, amp)
            unique = i + 1
        ku = unique * b
        if ku > 0:
            eQB = _relmax(Q[:, :ku] @ B[:ku], Qo[:, :ku] @ o.B[:ku])
            amp = np.sqrt(o.normA2 / max(E[unique - 1], 1e-300))
            assert eQB <= 10 * bar * max(1.0, amp), (eQB, amp)
        # what is unique whatever the blocks were sampled from: the residual the basis leaves
        res_g = np.linalg.norm(A64 - Q @ B)
        res_o = np.sqrt(max(o.E_dir[k // b - 1], 0.0))
        assert abs(res_g - res_o) <= floor * np.linalg.norm(A64) + 0.05 * res_o, (res_g, res_o)
    finally:
        rrf.rrf_destroy(h)
