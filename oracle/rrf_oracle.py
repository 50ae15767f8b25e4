"""CPU oracle for the Householder blocked adaptive randomized range finder.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 restatement of the
paper's Algorithm 2 ("Householder Blocked Adaptive Randomized Range Finder")
written from the paper; it shares no code with the CUDA library and must only
be imported by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark.  Library matmuls (numpy `@`) serve as the GEMM steps; the panel
factorisation is written out column by column.

Readings of the paper taken here:
  * Algorithm 2 line 8 applies Q_i^T = I - V_i T_i^T V_i^T (Theorem 3.1 and
    step 3 of the recursive QB recipe say "A <- Q_1^T A").
  * "qr(.)" / geqrt: LAPACK's Householder convention, beta = -sign(alpha)*||x||,
    v[0] = 1, tau = (beta - alpha)/beta, H = I - tau v v^T.  The sign of a zero pivot is
    the sign of the zero, as in LAPACK (beta = -SIGN(||x||, alpha)): alpha = +0.0 gives
    beta = -||x||, alpha = -0.0 gives beta = +||x||.
  * tolerance: Frobenius norm, relative to ||A||_F when `relative` is set;
    the loop continues while E > sigma^2 (strict).
  * stopping quantity: `estimator="direct"` uses E = ||W[r0+b:, :]||_F^2, the
    residual itself (section 3, after the Frobenius identity: the rows below
    block row i of the updated matrix carry the whole remaining error);
    `estimator="subtractive"` is Algorithm 2 line 9 literally,
    E <- E - ||B_i||_F^2.  Both are always recorded.
  * rank cap: the loop also ends when another block would exceed `max_rank`
    (the paper's fixed-rank mode).
  * stopping rules that need neither B nor the updated matrix (the outlook's "alternative stopping
    criteria ... estimating the spectral norm of the remaining part", and its variant that leaves A
    unchanged): the sampled panel itself is a randomized probe of the residual.  With Omega_i
    standard Gaussian (n x b) and W the residual before block i,
        E[ ||W Omega_i||_F^2 ] = b ||W||_F^2,
    so `estimator="sampled_fro"` tests E = ||Y_i||_F^2 / b, and (Halko, Martinsson, Tropp 2011,
    Lemma 4.1) ||W||_2 <= 10 sqrt(2/pi) max_j ||W omega_j||_2 with probability 1 - 10^-b, so
    `estimator="sampled_spectral"` tests E = (200/pi) max_j ||Y_i[:, j]||_2^2, a bound on the squared
    SPECTRAL norm of the residual (the norm of Eq. "tolerance").  Both are evaluated when panel i has
    been sampled and before it is factored: the loop stops with k = i b if E <= sigma^2.  If the rank
    cap ends the loop instead, nothing certifies the last block and the status is "cap reached".
  * `schedule="a_unchanged"`: the outlook's variant that never updates A and returns no B.  The
    panel is sampled from A itself, Y_i = A Omega_i, and the reflector blocks found so far are applied
    to it, Y_i <- Q_{i-1}^T ... Q_0^T Y_i, before its rows i b.. are factored.  By Theorem 3.1 this is
    the same panel as the in-place schedule's.  Only the sampled estimators can stop this loop.

Parity status: every function below is pinned by tests/test_oracle_pins.py
(dense Householder QR of A*Omega via LAPACK, the compact-WY identities, the
Frobenius identity of section 3, Eckart-Young, exact-rank and run-to-completion
cases).  Element-wise agreement of late columns of Q between two correct
implementations is ill-conditioned: block i of Y is sampled from a residual
that carries absolute noise u*||A||, so V_i moves by about
u*||A||_F/||W_trail||_F times cond(Y_i).  That one comparison is therefore
graded against the oracle's own envelope (`permuted_rerun`): parity unpinned
for Q element-wise beyond that envelope.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

RRF_OK = 0
RRF_MAX_RANK_REACHED = 1


def house(x: np.ndarray):
    """Householder reflector of a vector (section 3, "factored form ... geqrf").

    Returns (v, tau, beta) with v[0] = 1 and (I - tau v v^T) x = beta e_1, in x's precision.
    """
    x = np.asarray(x)
    dt = x.dtype.type
    alpha = x[0]
    tail = x[1:]
    xnorm = np.sqrt(np.dot(tail, tail))
    v = np.zeros_like(x)
    v[0] = 1.0
    if xnorm == 0.0:
        return v, dt(0.0), alpha
    sign = dt(np.copysign(1.0, alpha))          # LAPACK's SIGN(., alpha): honours the sign of a zero
    beta = -sign * np.sqrt(alpha * alpha + xnorm * xnorm)
    tau = (beta - alpha) / beta
    v[1:] = tail / (alpha - beta)
    return v, tau, beta


def panel_qr(Y: np.ndarray):
    """Unblocked Householder QR of a tall panel with the compact-WY factor.

    Algorithm 2 line 7 (geqrt).  Returns (V, tau, T, R):
    V is rows x b unit lower trapezoidal (ones on the diagonal, zeros above),
    T is b x b upper triangular with H_0 H_1 ... H_{b-1} = I - V T V^T
    (Eq. "Q_i = I_m - V_i T_i V_i^T"), R is the b x b triangular factor.
    """
    Y = np.array(Y, copy=True)
    if Y.dtype not in (np.float32, np.float64):
        Y = Y.astype(np.float64)
    rows, b = Y.shape
    V = np.zeros((rows, b), dtype=Y.dtype)
    tau = np.zeros(b, dtype=Y.dtype)
    T = np.zeros((b, b), dtype=Y.dtype)
    for j in range(b):
        if j < rows:
            v, tau[j], beta = house(Y[j:, j])
            V[j:, j] = v
            Y[j, j] = beta
            Y[j + 1:, j] = 0.0
            if j + 1 < b and tau[j] != 0.0:
                wrow = v @ Y[j:, j + 1:]
                Y[j:, j + 1:] -= tau[j] * np.outer(v, wrow)
        # T[:, j]: forward accumulation of the product of reflectors
        T[j, j] = tau[j]
        if j > 0:
            T[:j, j] = -tau[j] * (T[:j, :j] @ (V[:, :j].T @ V[:, j]))
    return V, tau, T, np.triu(Y[:b, :])


@dataclass
class OracleResult:
    k: int
    status: int
    steps: int
    normA2: float
    sigma2: float
    V: np.ndarray            # m x k, unit lower trapezoidal
    T: np.ndarray            # b x k, T_i in columns i*b:(i+1)*b
    B: np.ndarray            # k x n
    E_sub: list = field(default_factory=list)   # after each block: Algorithm 2 line 9
    E_dir: list = field(default_factory=list)   # after each block: ||W[r0+b:, :]||_F^2
    E_est: list = field(default_factory=list)   # sampled estimators: per sampled panel, the estimate of the
                                                # residual BEFORE that block (one entry more than blocks if the
                                                # estimate stopped the loop)
    W: np.ndarray | None = None                 # final working matrix (m x n)


def _sumsq(X: np.ndarray) -> float:
    """Squared Frobenius norm, accumulated in float64 whatever X's precision."""
    X64 = X.astype(np.float64, copy=False)
    return float(np.sum(X64 * X64))


SPECTRAL_FACTOR = 200.0 / np.pi      # (10 sqrt(2/pi))^2


def sampled_estimate(Y: np.ndarray, estimator: str) -> float:
    """Randomized estimate of the squared residual norm from a sampled panel Y = W Omega_i."""
    colsq = np.sum(Y.astype(np.float64) ** 2, axis=0)
    if estimator == "sampled_fro":
        return float(np.sum(colsq)) / Y.shape[1]
    if estimator == "sampled_spectral":
        return SPECTRAL_FACTOR * float(np.max(colsq))
    raise ValueError(estimator)


def rrf(A: np.ndarray, Omega: np.ndarray, b: int, tol: float, max_rank: int,
        relative: bool = True, estimator: str = "direct", keep_w: bool = False,
        dtype=np.float64, schedule: str = "in_place", fixed_rank: bool = False) -> OracleResult:
    """Algorithm 2, in the paper's order.

    A: m x n; Omega: n x max_rank (block i uses columns i*b:(i+1)*b, i.e. the
    "fresh Gaussian" of line 6 is passed in); tol: sigma (relative to ||A||_F
    if `relative`).  `dtype` is the working precision: float64 is the oracle
    proper; float32 reruns the same steps in single precision (the paper's
    experiments are in single precision) and serves as the plain-fp32 yardstick.
    `estimator`: "direct", "subtractive", "sampled_fro", "sampled_spectral" (see the header).
    `schedule`: "in_place" (Algorithm 2) or "a_unchanged" (no update of A, no B; sampled estimators
    or `fixed_rank` only).  `fixed_rank`: ignore the tolerance and run to the cap.
    """
    W = np.array(A, dtype=dtype, copy=True)                 # line 2: B <- A
    Omega = np.asarray(Omega, dtype=dtype)
    m, n = W.shape
    assert b >= 1 and max_rank % b == 0 and max_rank <= min(m, n)
    assert Omega.shape[0] == n and Omega.shape[1] >= max_rank
    sampled = estimator in ("sampled_fro", "sampled_spectral")
    unchanged = schedule == "a_unchanged"
    assert schedule in ("in_place", "a_unchanged")
    assert not unchanged or sampled or fixed_rank
    normA2 = _sumsq(W)                                      # line 1: E <- ||A||_F^2
    sigma2 = (tol * tol * normA2) if relative else tol * tol
    V = np.zeros((m, max_rank), dtype=dtype)                # line 3
    T = np.zeros((b, max_rank), dtype=dtype)
    res = OracleResult(0, RRF_OK, 0, normA2, sigma2, V, T, W)
    E_sub = normA2
    E = normA2
    met = (not fixed_rank) and not (E > sigma2)
    i = 0                                                   # line 4
    while not met and (i + 1) * b <= max_rank:              # line 5 (+ rank cap)
        r0 = i * b
        Om = Omega[:, r0:r0 + b]                            # line 6
        if unchanged:
            Y = W @ Om                                      # W is A itself here: it is never updated
            for l in range(i):                              # Q_{i-1}^T ... Q_0^T, in the order Q_0^T first
                q0 = l * b
                Vl = V[q0:, q0:q0 + b]
                Tl = T[:, q0:q0 + b]
                Y[q0:, :] -= Vl @ (Tl.T @ (Vl.T @ Y[q0:, :]))
            Y = Y[r0:, :]
        else:
            Y = W[r0:, :] @ Om                              # line 7: sample ...
        if sampled:
            E = sampled_estimate(Y, estimator)
            res.E_est.append(E)
            if not fixed_rank and not (E > sigma2):
                met = True
                break
        Vi, _, Ti, _ = panel_qr(Y)                          # ... and factor
        V[r0:, r0:r0 + b] = Vi
        T[:, r0:r0 + b] = Ti
        if not unchanged:
            Z = Vi.T @ W[r0:, :]                            # line 8: W <- Q_i^T W
            Z = Ti.T @ Z
            W[r0:, :] -= Vi @ Z
            Bi = W[r0:r0 + b, :]
            E_sub = E_sub - _sumsq(Bi)                      # line 9
            trail = W[r0 + b:, :]
            E_dir = _sumsq(trail)
            res.E_sub.append(E_sub)
            res.E_dir.append(E_dir)
            if not sampled:
                E = E_dir if estimator == "direct" else E_sub
                met = (not fixed_rank) and not (E > sigma2)
        i += 1                                              # line 10
    k = i * b                                               # lines 12-14
    res.k = k
    res.steps = i
    if sampled or unchanged:
        res.status = RRF_OK if met else RRF_MAX_RANK_REACHED     # only an estimate that stopped the loop certifies
    else:
        res.status = RRF_OK if E <= sigma2 else RRF_MAX_RANK_REACHED
    res.V = V[:, :k]
    res.T = T[:, :k]
    res.B = None if unchanged else W[:k, :].copy()
    res.W = W if (keep_w and not unchanged) else None
    return res


def apply_qt(V: np.ndarray, T: np.ndarray, b: int, C: np.ndarray) -> np.ndarray:
    """C <- Q^T C with Q = Q_0 Q_1 ... Q_{i-1}, Q_l = I - V_l T_l V_l^T on rows l*b: ."""
    C = np.array(C, dtype=np.float64, copy=True)
    k = V.shape[1]
    for l in range(k // b):
        r0 = l * b
        Vl = V[r0:, r0:r0 + b]
        Tl = T[:, r0:r0 + b]
        C[r0:, :] -= Vl @ (Tl.T @ (Vl.T @ C[r0:, :]))
    return C


def apply_q(V: np.ndarray, T: np.ndarray, b: int, C: np.ndarray) -> np.ndarray:
    """C <- Q C (block reflectors applied from the last to the first)."""
    C = np.array(C, dtype=np.float64, copy=True)
    k = V.shape[1]
    for l in range(k // b - 1, -1, -1):
        r0 = l * b
        Vl = V[r0:, r0:r0 + b]
        Tl = T[:, r0:r0 + b]
        C[r0:, :] -= Vl @ (Tl @ (Vl.T @ C[r0:, :]))
    return C


def rrf_column_sharded(A_loc: np.ndarray, Omega_loc: np.ndarray, b: int, tol: float, max_rank: int, allreduce,
                       relative: bool = True, fixed_rank: bool = False) -> OracleResult:
    """One rank of the column-sharded variant (outlook: "extensions to distributed matrix layouts").

    The columns of A are split over the ranks, A = [A_1 ... A_P]; rank p holds A_p (m x n_p) and the matching
    ROWS of Omega (n_p x max_rank), since A Omega_i = sum_p A_p Omega_{i,p}.  `allreduce(x)` returns the sum of the
    ranks' arrays (or floats).  Per block there is exactly one exchange of data, the m_i x b panel:
        Y_i = allreduce(W_p[r0:, :] Omega_{i,p});  every rank factors the same Y_i;  the update is local;
    plus two scalars (||A||_F^2 once, the residual norm per block).  V, T, k and the traces come out identical on
    every rank; B is this rank's column block of B.  Stops on the residual norm (estimator "direct").
    """
    W = np.array(A_loc, dtype=np.float64, copy=True)
    Omega_loc = np.asarray(Omega_loc, dtype=np.float64)
    m = W.shape[0]
    normA2 = float(allreduce(_sumsq(W)))
    sigma2 = (tol * tol * normA2) if relative else tol * tol
    V = np.zeros((m, max_rank))
    T = np.zeros((b, max_rank))
    res = OracleResult(0, RRF_OK, 0, normA2, sigma2, V, T, None)
    E = normA2
    E_sub = normA2
    met = (not fixed_rank) and not (E > sigma2)
    i = 0
    while not met and (i + 1) * b <= max_rank:
        r0 = i * b
        Y = allreduce(W[r0:, :] @ Omega_loc[:, r0:r0 + b])           # the one exchange of a block step
        Vi, _, Ti, _ = panel_qr(Y)
        V[r0:, r0:r0 + b] = Vi
        T[:, r0:r0 + b] = Ti
        W[r0:, :] -= Vi @ (Ti.T @ (Vi.T @ W[r0:, :]))
        E_sub = E_sub - float(allreduce(_sumsq(W[r0:r0 + b, :])))
        E = float(allreduce(_sumsq(W[r0 + b:, :])))
        res.E_sub.append(E_sub)
        res.E_dir.append(E)
        met = (not fixed_rank) and not (E > sigma2)
        i += 1
    k = i * b
    res.k, res.steps = k, i
    res.status = RRF_OK if E <= sigma2 else RRF_MAX_RANK_REACHED
    res.V, res.T, res.B = V[:, :k], T[:, :k], W[:k, :].copy()
    return res


def permuted_rerun(A, Omega, b, tol, max_rank, seed=0, **kw) -> OracleResult:
    """The same problem with the columns of A and the rows of Omega permuted.

    A P (P^T Omega) = A Omega, so V, T, k are mathematically unchanged and B is
    column-permuted; only the summation order differs.  The distance between
    this run and the plain one is the envelope inside which two correct
    float64 implementations may disagree.  B is returned un-permuted.
    """
    perm = np.random.default_rng(seed).permutation(A.shape[1])
    res = rrf(np.ascontiguousarray(A[:, perm]), np.ascontiguousarray(Omega[perm, :]),
              b, tol, max_rank, **kw)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.size)
    res.B = res.B[:, inv]
    return res


def subspace_transfer(V_old, T_old, V_new, T_new, b: int, M: np.ndarray) -> np.ndarray:
    """Section "Towards Efficient Low-Rank Deep Learning": an optimiser state M (k_old x n) held in the
    basis Q_old is replaced by Q_new^T Q_old M (k_new x n).  Written out with the explicit bases."""
    Q_old = form_q(V_old, T_old, b)
    Q_new = form_q(V_new, T_new, b)
    return Q_new.T @ (Q_old @ np.asarray(M, dtype=np.float64))


def form_q(V: np.ndarray, T: np.ndarray, b: int) -> np.ndarray:
    """Explicit Q = (Q_0 ... Q_{i-1}) I[:, 0:k]  (Algorithm 2, Ensure line)."""
    m, k = V.shape
    return apply_q(V, T, b, np.eye(m, k))
