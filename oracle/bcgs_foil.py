"""Block classical Gram-Schmidt range finder (the paper's Algorithm 1), CPU only.

TEST INFRASTRUCTURE, like everything under oracle/: the comparison method of the paper's stability
experiment (Section "Numerical experiments", Figure "orthogonality loss"), restated so that the CPU tests
can show the behaviour the Householder formulation is built to avoid.  It is not part of the library
and nothing on the product path imports it.

One pass of Algorithm 1 with the block Omega_i passed in (so that both methods see the same samples):
    Q_new <- orth(A_res Omega_i)                     (line 3; orth = thin QR)
    Q_new <- orth((I - Q Q^T) Q_new)                 (line 4, only with `reorth`)
    Q <- [Q Q_new];  B_new <- Q_new^T A_res;  B <- [B; B_new];  A_res <- A_res - Q_new B_new   (lines 5-8)
A_res is the residual the method tracks in place of A; its norm is the method's stopping quantity.
"""
from __future__ import annotations

import numpy as np


def bcgs_range_finder(A: np.ndarray, Omega: np.ndarray, b: int, passes: int, reorth: bool, dtype=np.float32):
    """Runs `passes` passes; returns Q (m x passes*b), B, and per pass the tracked residual norm
    ||A_res||_2 (the stopping quantity of Algorithm 1)."""
    R = np.array(A, dtype=dtype, copy=True)
    Omega = np.asarray(Omega, dtype=dtype)
    m, n = R.shape
    Q = np.zeros((m, 0), dtype=dtype)
    B = np.zeros((0, n), dtype=dtype)
    tracked = []
    for i in range(passes):
        Y = R @ Omega[:, i * b:(i + 1) * b]
        Qn, _ = np.linalg.qr(Y)
        Qn = Qn.astype(dtype)
        if reorth and Q.shape[1] > 0:
            Qn, _ = np.linalg.qr(Qn - Q @ (Q.T @ Qn))
            Qn = Qn.astype(dtype)
        Bn = Qn.T @ R
        Q = np.concatenate([Q, Qn], axis=1)
        B = np.concatenate([B, Bn], axis=0)
        R = R - Qn @ Bn
        tracked.append(float(np.linalg.norm(R.astype(np.float64), 2)))
    return Q, B, tracked
