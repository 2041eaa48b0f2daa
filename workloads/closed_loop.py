"""Closed-loop toy problem: a quadratic whose gradient is computed from the CURRENT weights, so that
a delay of tau calls makes the applied gradient genuinely stale (the setting of the paper's toy
experiments, Sec. 2.2 and App. D.1: an aligned versus a misaligned quadratic under delay).

The loss is f(W) = 1/2 tr(W^T P W Q) for a weight matrix W (m x n), with P (m x m) and Q (n x n)
symmetric positive definite: its gradient is P W Q and its Hessian is the Kronecker product Q (x) P,
the structure the method assumes (Sec. 3.1).  `aligned=True` takes P and Q diagonal (the Hessian
eigenbasis is the coordinate basis); otherwise both are rotated by seeded random orthogonal matrices
and the starting point is rotated with them, so that both variants are the same problem in different
coordinates.  The paper does not print its matrix; spectra here are log-spaced over two (P) and one
and a half (Q) decades.  Inputs only: nothing of the optimizer lives here.
"""
from __future__ import annotations

import numpy as np


def kronecker_quadratic(m: int = 32, n: int = 16, aligned: bool = False, seed: int = 0):
    """Returns (P, Q, W0) as float64 arrays."""
    rng = np.random.default_rng(seed)
    dp = np.logspace(0.0, -2.0, m)
    dq = np.logspace(0.0, -1.5, n)
    w0 = np.random.default_rng(seed + 1).standard_normal((m, n))
    if aligned:
        return np.diag(dp), np.diag(dq), w0
    rp, _ = np.linalg.qr(rng.standard_normal((m, m)))
    rq, _ = np.linalg.qr(rng.standard_normal((n, n)))
    return (rp * dp) @ rp.T, (rq * dq) @ rq.T, rp @ w0 @ rq.T


def loss(P, Q, W) -> float:
    return 0.5 * float(np.sum(W * (P @ W @ Q)))
