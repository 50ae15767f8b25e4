"""Pins for the CPU oracle: each test ties oracle/rrf_oracle.py to something
other than itself (LAPACK's dense Householder QR, an SVD, closed forms and the
invariants the paper states), so that a dropped term, a wrong sign, index or
transpose in the oracle fails at least one of them."""
import numpy as np
import pytest
import scipy.linalg as sla

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import workloads as wl


def _case(m=96, n=80, b=8, max_rank=48, seed=3, decay=3.0):
    rng = np.random.default_rng(seed)
    p = min(m, n)
    u, _ = np.linalg.qr(rng.standard_normal((m, p)))
    v, _ = np.linalg.qr(rng.standard_normal((n, p)))
    s = np.exp(-np.arange(p) / decay)
    A = (u * s) @ v.T
    Om = rng.standard_normal((n, max_rank))
    return A, Om, s, b, max_rank


def _lapack_vtau(Y):
    (h, tau), _ = sla.qr(Y, mode="raw")
    V = np.tril(h, -1)[:, :Y.shape[1]]
    V[np.arange(Y.shape[1]), np.arange(Y.shape[1])] = 1.0
    return V, tau, np.triu(h[:Y.shape[1], :])


# ---- P2 / Theorem 3.1: concatenated reflectors == dense Householder QR of A*Omega


@pytest.mark.parametrize("b", [1, 4, 8])
def test_reflectors_equal_dense_householder_qr(b):
    A, Om, _, _, max_rank = _case(b=b, max_rank=48)
    r = orc.rrf(A, Om, b, 0.0, max_rank)            # tol 0: runs to the cap
    assert r.k == max_rank and r.status == orc.RRF_MAX_RANK_REACHED
    V_ref, tau_ref, _ = _lapack_vtau(A @ Om[:, :r.k])
    tau = np.concatenate([np.diag(r.T[:, i * b:(i + 1) * b]) for i in range(r.k // b)])
    # block 0 agrees to round-off; block i is sampled from a residual of relative size
    # sqrt(E_{i-1}/E_0) and loses digits in that proportion, hence the graded tolerance
    prev = [r.normA2] + r.E_dir[:-1]
    for i in range(r.k // b):
        amp = np.sqrt(r.normA2 / prev[i])
        blk = slice(i * b, (i + 1) * b)
        assert np.max(np.abs(r.V[:, blk] - V_ref[:, blk])) < 2e-13 * amp, i
        assert np.max(np.abs(tau[blk] - tau_ref[blk])) < 2e-13 * amp, i


def test_panel_qr_matches_lapack():
    rng = np.random.default_rng(0)
    Y = rng.standard_normal((50, 7))
    V, tau, T, R = orc.panel_qr(Y)
    V_ref, tau_ref, R_ref = _lapack_vtau(Y)
    assert np.allclose(V, V_ref, atol=1e-14)
    assert np.allclose(tau, tau_ref, atol=1e-14)
    assert np.allclose(R, R_ref, atol=1e-13)          # sign convention: R_jj = beta


def test_house_closed_form():
    v, tau, beta = orc.house(np.array([3.0, 4.0]))
    assert beta == -5.0 and np.isclose(tau, 1.6) and np.allclose(v, [1.0, 0.5])
    v, tau, beta = orc.house(np.array([-3.0, 4.0]))
    assert beta == 5.0 and np.isclose(tau, 1.6) and np.allclose(v, [1.0, -0.5])
    v, tau, beta = orc.house(np.array([2.0, 0.0, 0.0]))   # nothing to annihilate: H = I
    assert tau == 0.0 and beta == 2.0 and np.allclose(v, [1, 0, 0])


def test_house_at_a_zero_pivot():
    # alpha = +0.0: beta = -||x||, tau = 1, v = [1, x_1/||x||, ...]; alpha = -0.0 takes the other sign
    # (LAPACK's SIGN(., alpha) honours the sign of a zero, and "geqrt" is LAPACK's routine)
    v, tau, beta = orc.house(np.array([0.0, 3.0, 4.0]))
    assert beta == -5.0 and tau == 1.0 and np.allclose(v, [1.0, 0.6, 0.8], atol=1e-16)
    v, tau, beta = orc.house(np.array([-0.0, 3.0, 4.0]))
    assert beta == 5.0 and tau == 1.0 and np.allclose(v, [1.0, -0.6, -0.8], atol=1e-16)


@pytest.mark.parametrize("zero", [0.0, -0.0])
def test_panel_qr_with_a_zero_pivot_matches_lapack(zero):
    rng = np.random.default_rng(5)
    Y = rng.standard_normal((30, 5))
    Y[0, 0] = zero                       # the first pivot is an exact (signed) zero
    V, tau, T, R = orc.panel_qr(Y)
    V_ref, tau_ref, R_ref = _lapack_vtau(Y)
    assert np.allclose(V, V_ref, atol=1e-14) and np.allclose(tau, tau_ref, atol=1e-14)
    assert np.allclose(R, R_ref, atol=1e-13)
    assert np.sign(R[0, 0]) == (-1.0 if np.copysign(1.0, zero) > 0 else 1.0)


# ---- P5: compact WY factor


def test_compact_wy_identities():
    rng = np.random.default_rng(1)
    Y = rng.standard_normal((40, 6))
    V, tau, T, R = orc.panel_qr(Y)
    H = np.eye(40)
    for j in range(6):
        H = H @ (np.eye(40) - tau[j] * np.outer(V[:, j], V[:, j]))
    Q = np.eye(40) - V @ T @ V.T
    assert np.allclose(Q, H, atol=1e-14)
    assert np.allclose(np.diag(T), tau)
    assert np.allclose(np.tril(T, -1), 0.0)
    Tinv = np.linalg.inv(T)
    assert np.allclose(Tinv + Tinv.T, V.T @ V, atol=1e-12)
    assert np.allclose((Q.T @ Y)[:6], R, atol=1e-13)
    assert np.allclose((Q.T @ Y)[6:], 0.0, atol=1e-13)


# ---- P1, P3, P4: triangularity, orthogonality, Frobenius identity, B = Q^T A


def test_invariants_of_a_run():
    A, Om, s, b, max_rank = _case()
    r = orc.rrf(A, Om, b, 1e-3, max_rank, keep_w=True)
    assert r.status == orc.RRF_OK and 0 < r.k < max_rank
    Q = orc.form_q(r.V, r.T, b)
    k = r.k
    assert np.linalg.norm(Q.T @ Q - np.eye(k)) < 1e-13
    R = Q.T @ (A @ Om[:, :k])
    assert np.max(np.abs(np.tril(R, -1))) < 1e-13 * np.linalg.norm(R)
    assert np.allclose(r.B, Q.T @ A, atol=1e-14)
    res2 = np.linalg.norm(A - Q @ r.B) ** 2
    assert np.isclose(res2, r.normA2 - np.linalg.norm(r.B) ** 2, rtol=1e-9)
    assert np.isclose(res2, r.E_dir[-1], rtol=1e-10)
    assert np.isclose(r.E_sub[-1], r.E_dir[-1], rtol=1e-6)
    assert np.sqrt(res2) <= 1e-3 * np.sqrt(r.normA2)
    # apply_qt reproduces the working matrix; its top k rows are B
    assert np.allclose(orc.apply_qt(r.V, r.T, b, A), r.W, atol=1e-14)


# ---- brute force on tiny inputs: k is the first multiple of b meeting the tolerance


@pytest.mark.parametrize("tol", [3e-1, 1e-2, 1e-4])
def test_k_is_first_block_count_meeting_tolerance(tol):
    A, Om, s, b, max_rank = _case(m=60, n=50, b=5, max_rank=40, seed=11, decay=3.0)
    r = orc.rrf(A, Om, b, tol, max_rank)
    nrm = np.linalg.norm(A)
    expected = None
    for k in range(0, max_rank + 1, b):
        if k == 0:
            err = nrm
        else:
            Qk, _ = np.linalg.qr(A @ Om[:, :k])
            err = np.linalg.norm(A - Qk @ (Qk.T @ A))
        if err <= tol * nrm:
            expected = k
            break
    assert expected is not None
    assert r.k == expected and r.status == orc.RRF_OK


# ---- P6: Eckart-Young lower bound with the known singular values


def test_eckart_young_bound():
    A, Om, s, b, max_rank = _case()
    for tol in (1e-1, 1e-2, 1e-4):
        r = orc.rrf(A, Om, b, tol, max_rank)
        tail = np.sqrt(np.sum(s[r.k:] ** 2))
        err = np.sqrt(r.E_dir[-1])
        assert err >= tail * (1 - 1e-10)
        assert err <= tol * np.sqrt(r.normA2)
        if r.k > b:   # and the block before did not meet it
            assert np.sqrt(r.E_dir[-2]) > tol * np.sqrt(r.normA2)


# ---- P7: run to completion


def test_run_to_completion_tall():
    A, Om, s, b, _ = _case(m=72, n=40, b=8, max_rank=40)
    r = orc.rrf(A, Om, b, 0.0, 40, keep_w=True)
    assert r.k == 40
    Q = orc.form_q(r.V, r.T, b)
    assert np.linalg.norm(A - Q @ r.B) < 1e-13 * np.linalg.norm(A)
    assert np.linalg.norm(r.W[40:, :]) < 1e-13 * np.linalg.norm(A)


# ---- P8: exact rank, zero matrix, b = 1


def test_exact_rank_stops_at_rank():
    rng = np.random.default_rng(5)
    A = rng.standard_normal((64, 12)) @ rng.standard_normal((12, 48))
    Om = rng.standard_normal((48, 32))
    r = orc.rrf(A, Om, 4, 1e-10, 32)
    assert r.k == 12 and r.status == orc.RRF_OK
    assert r.E_dir[-1] <= 1e-24 * r.normA2


def test_zero_matrix_gives_rank_zero():
    Om = np.random.default_rng(0).standard_normal((10, 8))
    r = orc.rrf(np.zeros((12, 10)), Om, 4, 1e-3, 8)
    assert r.k == 0 and r.steps == 0 and r.status == orc.RRF_OK and r.B.shape == (0, 10)


def test_absolute_tolerance_and_subtractive_estimator():
    A, Om, s, b, max_rank = _case()
    nrm = np.linalg.norm(A)
    r_rel = orc.rrf(A, Om, b, 1e-2, max_rank)
    r_abs = orc.rrf(A, Om, b, 1e-2 * nrm, max_rank, relative=False)
    r_sub = orc.rrf(A, Om, b, 1e-2, max_rank, estimator="subtractive")
    assert r_rel.k == r_abs.k == r_sub.k
    assert np.array_equal(r_rel.B, r_sub.B)


def test_permuted_rerun_is_the_same_problem():
    A, Om, s, b, max_rank = _case()
    r = orc.rrf(A, Om, b, 1e-3, max_rank)
    rp = orc.permuted_rerun(A, Om, b, 1e-3, max_rank, seed=1)
    assert r.k == rp.k
    assert np.max(np.abs(r.B - rp.B)) < 1e-12 * np.max(np.abs(r.B))
    assert np.max(np.abs(r.V - rp.V)) < 1e-8


# ---- P9: the law of k does not depend on the singular vectors (diag stand-in)


def test_diag_standin_predicts_same_rank():
    w = wl.CONFIGS["cfg1"].scaled(256, 192, max_rank=128)
    A, s = wl.make_matrix(w)
    Om = wl.make_omega(w)
    r = orc.rrf(A, Om, w.b, 1e-4, w.max_rank)
    rd = orc.rrf(wl.diag_matrix(s, w.m, w.n), Om, w.b, 1e-4, w.max_rank)
    assert abs(r.k - rd.k) <= w.b
    assert np.isclose(np.linalg.svd(A, compute_uv=False)[:20], s[:20], rtol=1e-10).all()


# ---- P10: the one numerical behaviour the paper prints (section "Numerical Stability and
# Performance"): single precision, 1024 x 1024, singular values log-spaced from 1 to 1e-14,
# b = 64: the subtractive stopping quantity stops tracking the residual near k = 384 through
# cancellation, while orthogonality and the residual stay at single-precision round-off.


def test_fp32_subtractive_estimator_stops_tracking_near_384():
    rng = np.random.default_rng(10)
    n, b = 1024, 64
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    Vv, _ = np.linalg.qr(rng.standard_normal((n, n)))
    s = 10.0 ** (-14 * np.arange(n) / (n - 1))
    A = ((U * s) @ Vv.T).astype(np.float32)
    Om = rng.standard_normal((n, 640)).astype(np.float32)
    r = orc.rrf(A, Om, b, 0.0, 640, dtype=np.float32)
    e_sub, e_dir = np.array(r.E_sub), np.array(r.E_dir)
    assert np.all(np.abs(e_sub[:3] - e_dir[:3]) <= 1e-2 * e_dir[:3])        # k <= 192: tracks
    assert e_sub[5] > 10 * e_dir[5] or e_sub[5] <= 0                        # k = 384: lost
    assert np.all(np.abs(e_sub[6:]) > 100 * e_dir[6:])                      # and never recovers
    Q = orc.form_q(r.V.astype(np.float64), r.T.astype(np.float64), b)
    assert np.linalg.norm(Q.T @ Q - np.eye(640), 2) < 5e-6
    assert np.linalg.norm(A - Q @ (Q.T @ A), 2) < 2e-6


def test_subspace_transfer_pins():
    """Q_new^T Q_old M: identity when the bases coincide, an isometry that pads with zeros when the new
    basis extends the old one, and equal to the same product with bases taken from LAPACK's QR."""
    import scipy.linalg as sla
    rng = np.random.default_rng(77)
    m, n, b = 240, 150, 16
    A = rng.standard_normal((m, 40)) @ rng.standard_normal((40, n))
    Om = rng.standard_normal((n, 64))
    small = orc.rrf(A, Om, b, 0.0, 32)
    large = orc.rrf(A, Om, b, 0.0, 64)
    M = rng.standard_normal((32, 70))
    same = orc.subspace_transfer(small.V, small.T, small.V, small.T, b, M)
    assert np.max(np.abs(same - M)) < 1e-13
    # the first 32 basis vectors of the longer run are the basis of the shorter one
    ext = orc.subspace_transfer(small.V, small.T, large.V, large.T, b, M)
    assert ext.shape == (64, 70)
    assert np.max(np.abs(ext[:32] - M)) < 1e-12 and np.max(np.abs(ext[32:])) < 1e-12
    # unrelated bases: against thin Q factors from LAPACK (sign-fixed to the Householder convention)
    A2 = rng.standard_normal((m, n))
    other = orc.rrf(A2, Om, b, 0.0, 48)

    def lapack_basis(Amat, k):
        Q, R = sla.qr(Amat @ Om[:, :k], mode="economic")
        return Q

    Qo, Qn = lapack_basis(A, 32), lapack_basis(A2, 48)
    # geqrf and the blocked run span the same subspaces and agree column by column up to sign
    So = np.sign(np.sum(Qo * orc.form_q(small.V, small.T, b), axis=0))
    Sn = np.sign(np.sum(Qn * orc.form_q(other.V, other.T, b), axis=0))
    want = (Qn * Sn).T @ ((Qo * So) @ M)
    got = orc.subspace_transfer(small.V, small.T, other.V, other.T, b, M)
    assert got.shape == (48, 70)
    assert np.max(np.abs(got - want)) < 1e-9 * np.max(np.abs(want))


def test_householder_keeps_orthogonality_where_block_gram_schmidt_loses_it():
    """The paper's stability experiment (1024 x 1024, singular values 1 ... 1e-14, b = 64, single precision),
    qualitatively: without reorthogonalisation the Gram-Schmidt range finder loses orthogonality while its own
    stopping quantity keeps falling; with it, and for the Householder method, Q stays orthonormal to single
    precision and the projection residual follows the singular values down to the fp32 floor."""
    from oracle import bcgs_foil
    rng = np.random.default_rng(2024)
    n, b, passes = 1024, 64, 10
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    Vv, _ = np.linalg.qr(rng.standard_normal((n, n)))
    s = np.logspace(0, -14, n)
    A = ((U * s) @ Vv.T).astype(np.float32)
    Om = rng.standard_normal((n, passes * b)).astype(np.float32)
    A64 = A.astype(np.float64)

    def orth_loss(Q):
        Q = Q.astype(np.float64)
        return np.linalg.norm(Q.T @ Q - np.eye(Q.shape[1]), 2)

    def proj_res(Q):
        Q = Q.astype(np.float64)
        return np.linalg.norm(A64 - Q @ (Q.T @ A64), 2)

    Q_plain, _, tracked_plain = bcgs_foil.bcgs_range_finder(A, Om, b, passes, reorth=False)
    Q_re, _, _ = bcgs_foil.bcgs_range_finder(A, Om, b, passes, reorth=True)
    hh = orc.rrf(A, Om, b, 0.0, passes * b, dtype=np.float32)
    Q_hh = orc.form_q(hh.V.astype(np.float64), hh.T.astype(np.float64), b)
    u32 = 6e-8
    assert orth_loss(Q_hh) < 100 * u32 and orth_loss(Q_re) < 100 * u32
    assert orth_loss(Q_plain) > 1e4 * u32                          # orthogonality gone ...
    assert proj_res(Q_plain) > 30 * proj_res(Q_hh)                 # ... and with it the approximation,
    assert tracked_plain[-1] < 0.1 * proj_res(Q_plain)             # which its stopping quantity does not see
    # Householder and reorthogonalised Gram-Schmidt both reach the single-precision floor of this matrix
    floor = np.linalg.svd(A64, compute_uv=False)[passes * b]
    assert proj_res(Q_hh) < 50 * max(floor, u32) and proj_res(Q_re) < 50 * max(floor, u32)


# ---- sampled stopping estimators and the schedule that leaves A unchanged


def test_sampled_frobenius_estimate_is_exact_for_an_orthogonal_probe():
    # closed form: with Omega_i = sqrt(b) O, O orthogonal n x n (b = n), ||W Omega_i||_F^2 / b = ||W||_F^2
    rng = np.random.default_rng(21)
    W = rng.standard_normal((30, 12))
    O, _ = np.linalg.qr(rng.standard_normal((12, 12)))
    est = orc.sampled_estimate(W @ (np.sqrt(12.0) * O), "sampled_fro")
    assert np.isclose(est, np.linalg.norm(W) ** 2, rtol=1e-13)


def test_sampled_estimates_are_unbiased_and_bound_the_spectral_norm():
    rng = np.random.default_rng(22)
    W = rng.standard_normal((60, 40)) * np.exp(-np.arange(40) / 6.0)
    fro2, two2 = np.linalg.norm(W) ** 2, np.linalg.norm(W, 2) ** 2
    b, draws = 8, 400
    est_f = np.array([orc.sampled_estimate(W @ rng.standard_normal((40, b)), "sampled_fro") for _ in range(draws)])
    # E[est] = ||W||_F^2; Var[est] = 2 ||W^T W||_F^2 / b
    std = np.sqrt(2.0 * np.linalg.norm(W.T @ W) ** 2 / b / draws)
    assert abs(est_f.mean() - fro2) < 5 * std
    est_s = np.array([orc.sampled_estimate(W @ rng.standard_normal((40, b)), "sampled_spectral") for _ in range(draws)])
    assert np.all(est_s >= two2)                      # fails with probability 10^-b per draw
    assert np.median(est_s) < 64 * 40 * two2          # and it is not vacuous


@pytest.mark.parametrize("estimator", ["sampled_fro", "sampled_spectral"])
def test_sampled_rules_stop_on_the_panel_before_it_is_factored(estimator):
    A, Om, s, b, max_rank = _case(m=120, n=100, b=10, max_rank=80, seed=5, decay=4.0)
    tol = 1e-3
    r = orc.rrf(A, Om, b, tol, max_rank, estimator=estimator, keep_w=True)
    assert r.status == orc.RRF_OK and 0 < r.k < max_rank
    assert len(r.E_est) == r.steps + 1                # the estimate that stopped the loop has no block
    # brute force from the recorded residuals: entry i was computed from the residual after i blocks
    sigma2 = tol * tol * r.normA2
    assert all(e > sigma2 for e in r.E_est[:-1]) and r.E_est[-1] <= sigma2
    Q = orc.form_q(r.V, r.T, b)
    res2 = np.linalg.norm(A - Q @ (Q.T @ A)) ** 2
    if estimator == "sampled_spectral":               # certifies the 2-norm of the residual
        assert np.linalg.norm(A - Q @ (Q.T @ A), 2) ** 2 <= r.E_est[-1] <= sigma2
    else:                                             # tracks the Frobenius residual within its spread
        assert 0.3 * res2 <= r.E_est[-1] <= 3.0 * res2
    # the first estimate probes A itself
    assert np.isclose(r.E_est[0], orc.sampled_estimate(A @ Om[:, :b], estimator), rtol=1e-12)


def test_schedule_that_leaves_a_unchanged_gives_the_same_reflectors():
    # Theorem 3.1: the panel sampled from A and pulled through the reflectors found so far is the panel the
    # in-place schedule samples from the updated matrix, so V, T (and k under a sampled rule) agree
    A, Om, s, b, max_rank = _case(m=90, n=70, b=6, max_rank=36, seed=8, decay=5.0)
    r1 = orc.rrf(A, Om, b, 0.0, max_rank, fixed_rank=True)
    r2 = orc.rrf(A, Om, b, 0.0, max_rank, fixed_rank=True, schedule="a_unchanged")
    assert r2.k == r1.k == max_rank and r2.B is None
    prev = [r1.normA2] + r1.E_dir[:-1]
    for i in range(max_rank // b):
        amp = np.sqrt(r1.normA2 / prev[i])
        blk = slice(i * b, (i + 1) * b)
        assert np.max(np.abs(r1.V[:, blk] - r2.V[:, blk])) < 1e-13 * amp, i
        assert np.max(np.abs(r1.T[:, blk] - r2.T[:, blk])) < 1e-12 * amp, i
    # against LAPACK directly: the reflectors are those of the dense QR of A Omega
    V_ref, tau_ref, _ = _lapack_vtau(A @ Om[:, :max_rank])
    assert np.max(np.abs(r2.V[:, :b] - V_ref[:, :b])) < 1e-13
    a = orc.rrf(A, Om, b, 5e-2, max_rank, estimator="sampled_fro")
    u = orc.rrf(A, Om, b, 5e-2, max_rank, estimator="sampled_fro", schedule="a_unchanged")
    assert 0 < a.k < max_rank and a.k == u.k and a.status == u.status == orc.RRF_OK
    assert np.allclose(a.E_est, u.E_est, rtol=1e-9)


def test_foil_on_the_stability_stress_configuration():
    """The third configuration's recipe (fifteen decades of singular values, then a 1e-16 floor) at 1024 x 1024 in
    double precision, b = 32: the regime where block Gram-Schmidt without reorthogonalisation loses orthogonality
    while the Householder range finder keeps it at round-off."""
    from oracle import bcgs_foil
    w = wl.CONFIGS["cfg3"].scaled(m=1024, n=1024, max_rank=384)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w)
    passes = w.max_rank // w.b
    Q_plain, _, _ = bcgs_foil.bcgs_range_finder(A, Om, w.b, passes, reorth=False, dtype=np.float64)
    Q_re, _, _ = bcgs_foil.bcgs_range_finder(A, Om, w.b, passes, reorth=True, dtype=np.float64)
    hh = orc.rrf(A, Om, w.b, 0.0, w.max_rank)
    Q_hh = orc.form_q(hh.V, hh.T, w.b)

    def loss(Q):
        return np.linalg.norm(Q.T @ Q - np.eye(Q.shape[1]))

    assert loss(Q_hh) < 1e-13                       # the bar the GPU path is held to is 1e-12
    assert loss(Q_re) < 1e-12
    assert loss(Q_plain) > 1e-6                     # orthogonality lost by ten orders of magnitude
