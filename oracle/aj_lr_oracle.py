"""CPU oracle for the classifier fit (test infrastructure, not a product path).

The paper's classifier (Section 3.2 "Classifier model & training", Section 4.1 and the appendix on classifier
ablations) is a logistic regression with L2 regularisation fitted by scikit-learn with default settings,
regularisation coefficient C from a logarithmic grid (1e-4 for the 8B/70B pair).  In scikit-learn's
convention that is the unique minimiser of

    f(w, b) = 1/2 w.w  +  C * sum_i log(1 + exp(-s_i (x_i.w + b))),     s_i = +1 if row i is important, else -1,

with the intercept b not regularised.  This module finds that minimiser by Newton's method with the exact
Hessian in fp64 (plain numpy), to a gradient of 1e-10 or better: slow, obviously correct, and independent of
the CUDA library.  Only tests, the smoke check and the benchmark's CPU baseline may import it.
"""
from __future__ import annotations

import numpy as np


def objective(X, y, C, w, b):
    """f(w, b) and its gradient (dw, db) in fp64."""
    X = np.asarray(X, dtype=np.float64)
    s = np.where(np.asarray(y) != 0, 1.0, -1.0)
    t = s * (X @ w + b)
    f = 0.5 * float(w @ w) + C * float(np.sum(np.logaddexp(0.0, -t)))
    r = -s / (1.0 + np.exp(t))  # d/dz of log(1 + exp(-s z))
    return f, w + C * (X.T @ r), C * float(np.sum(r))


def fit(X, y, C, tol=1e-11, max_iter=200):
    """The minimiser (w [F] fp64, b) by damped Newton steps on f."""
    X = np.asarray(X, dtype=np.float64)
    n, F = X.shape
    s = np.where(np.asarray(y) != 0, 1.0, -1.0)
    A = np.hstack([X, np.ones((n, 1))])  # the intercept as a last, unregularised coordinate
    reg = np.ones(F + 1)
    reg[F] = 0.0
    v = np.zeros(F + 1)
    for _ in range(max_iter):
        t = s * (A @ v)
        p = 1.0 / (1.0 + np.exp(t))       # sigma(-t)
        g = reg * v + C * (A.T @ (-s * p))
        if np.max(np.abs(g)) <= tol:
            break
        h = p * (1.0 - p)
        H = np.diag(reg) + C * (A.T * h) @ A
        H[F, F] += 1e-300
        step = np.linalg.solve(H, g)
        f0 = 0.5 * float(v[:F] @ v[:F]) + C * float(np.sum(np.logaddexp(0.0, -t)))
        a = 1.0
        while True:  # halve the step until f decreases (Newton is monotone near the optimum)
            vn = v - a * step
            tn = s * (A @ vn)
            fn = 0.5 * float(vn[:F] @ vn[:F]) + C * float(np.sum(np.logaddexp(0.0, -tn)))
            if fn <= f0 or a < 1e-8:
                break
            a *= 0.5
        v = vn
    return v[:F].copy(), float(v[F])


def predict_proba(X, w, b):
    return 1.0 / (1.0 + np.exp(-(np.asarray(X, dtype=np.float64) @ w + b)))
