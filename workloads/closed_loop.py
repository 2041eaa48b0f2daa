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


# ---------------------------------------------------------------------------------------------
# Spiral loss (Sec. 2.2, App. D.1): a two-parameter landscape whose Hessian eigenbasis turns along
# the valley, f(r, theta) = r^2 + (20 sin(4 r - theta) + 1)^2 in polar coordinates of p = (x, y).
# The paper runs plain Adam on it (learning rate 0.1, beta1 = 0, beta2 = 0.9) and switches a delay of
# tau = 1 on at some iteration.  Problem definition only: loss, gradient and a measure of how far the
# Hessian eigenbasis is from the coordinate axes.
# ---------------------------------------------------------------------------------------------
def spiral_loss(p) -> float:
    x, y = float(p[0]), float(p[1])
    r, th = np.hypot(x, y), np.arctan2(y, x)
    return r * r + (20.0 * np.sin(4.0 * r - th) + 1.0) ** 2


def spiral_grad(p) -> np.ndarray:
    """Gradient with respect to (x, y): chain rule through r = |p| and theta = atan2(y, x)."""
    x, y = float(p[0]), float(p[1])
    r, th = np.hypot(x, y), np.arctan2(y, x)
    s = 20.0 * np.sin(4.0 * r - th) + 1.0
    c = 20.0 * np.cos(4.0 * r - th)
    f_r = 2.0 * r + 8.0 * s * c
    f_th = -2.0 * s * c
    return np.array([f_r * x / r - f_th * y / (r * r), f_r * y / r + f_th * x / (r * r)])


def spiral_valley_excess(p) -> float:
    """Loss above the floor r^2 of the valley: how far the iterate sits up the valley walls."""
    return spiral_loss(p) - float(p[0]) ** 2 - float(p[1]) ** 2


def spiral_misalignment(p, h: float = 1e-6) -> float:
    """0 when the dominant Hessian eigenvector at p lies along a coordinate axis, 1 when it is at 45
    degrees to both (central differences of the gradient)."""
    p = np.asarray(p, dtype=np.float64)
    H = np.zeros((2, 2))
    for i in range(2):
        e = np.zeros(2)
        e[i] = h
        H[:, i] = (spiral_grad(p + e) - spiral_grad(p - e)) / (2.0 * h)
    w, v = np.linalg.eigh(0.5 * (H + H.T))
    d = v[:, int(np.argmax(np.abs(w)))]
    a = np.arctan2(abs(d[1]), abs(d[0]))
    return float(min(a, np.pi / 2.0 - a) / (np.pi / 4.0))
