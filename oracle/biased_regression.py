"""CPU checker for the biased-regression study (Appendix E of arXiv 2310.05674).

TEST INFRASTRUCTURE ONLY, like the rest of ``oracle/``: plain numpy in float64, called by ``tests/`` and by
the benchmark's validation stage; the CUDA package never imports it and shares no code with it.

The bilevel problem of Appendix E:

    lambda* = argmin_lambda  L_meta(w*(lambda)),   L_meta(w)         = || X' w - y' ||^2
    w*(lambda) = argmin_w    L_base(w, lambda),    L_base(w, lambda) = || X w - y ||^2 + beta || w - lambda ||^2

Closed forms (Appendix E, items 1-3), written out from the normal equations:

    base Jacobian (item 1)   H = X^T X + beta I              (half the Hessian of L_base in w)
    base solution            w*(lambda) = H^-1 (X^T y + beta lambda)
    meta gradient (item 2)   dL_meta/dlambda = 2 beta H^-1 (X'^T X' w* - X'^T y')
    optimum (item 3)         lambda* = (A^T A)^-1 A^T b,  A = beta X' H^-1,  b = y' - X' H^-1 X^T y

Reading: the paper prints item 2 without the factor 2 (it is the gradient of half the printed objective); the
functions below differentiate the objective as printed, and ``printed_meta_grad`` returns the printed expression.
The study's measures (a cosine and the distance to lambda*) do not depend on that factor.

SAMA on this problem, in the paper's order (Eq. 3-5, Sec. 3.2), at base parameters w:
    g_meta   = dL_meta/dw = 2 X'^T (X' w - y')                         direct gradient (Eq. 1)
    p        = (du/dg_base) * g_meta                                   Eq. 4 (identity for an SGD base optimiser)
    eps_fd   = alpha / ||p||_2,   w+- = w +- eps_fd p                  Sec. 3.2
    g_lambda(w) = dL_base/dlambda = -2 beta (w - lambda)
    metagrad = -[ g_lambda(w+) - g_lambda(w-) ] / (2 eps_fd)           Eq. 5
L_base is quadratic, so the central difference is exact: metagrad = 2 beta p.
"""
from __future__ import annotations

import numpy as np

import oracle as _o


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def base_jacobian(X, beta: float) -> np.ndarray:
    """Item 1: X^T X + beta I."""
    X = _f64(X)
    return X.T @ X + beta * np.eye(X.shape[1])


def base_solution(X, y, beta: float, lam) -> np.ndarray:
    """w*(lambda) = H^-1 (X^T y + beta lambda)."""
    X, y, lam = _f64(X), _f64(y), _f64(lam)
    return np.linalg.solve(base_jacobian(X, beta), X.T @ y + beta * lam)


def meta_loss(Xv, yv, w) -> float:
    r = _f64(Xv) @ _f64(w) - _f64(yv)
    return float(r @ r)


def base_loss(X, y, beta: float, w, lam) -> float:
    r = _f64(X) @ _f64(w) - _f64(y)
    d = _f64(w) - _f64(lam)
    return float(r @ r + beta * (d @ d))


def direct_grad(Xv, yv, w) -> np.ndarray:
    """dL_meta/dw = 2 X'^T (X' w - y')."""
    Xv, yv, w = _f64(Xv), _f64(yv), _f64(w)
    return 2.0 * (Xv.T @ (Xv @ w - yv))


def true_meta_grad(X, y, Xv, yv, beta: float, lam) -> np.ndarray:
    """Item 2 for the objective as printed: 2 beta H^-1 (X'^T X' w* - X'^T y')."""
    X, Xv, yv = _f64(X), _f64(Xv), _f64(yv)
    w = base_solution(X, y, beta, lam)
    return 2.0 * beta * np.linalg.solve(base_jacobian(X, beta), Xv.T @ (Xv @ w) - Xv.T @ yv)


def printed_meta_grad(X, y, Xv, yv, beta: float, lam) -> np.ndarray:
    """Item 2 exactly as printed (no factor 2)."""
    return 0.5 * true_meta_grad(X, y, Xv, yv, beta, lam)


def lambda_star(X, y, Xv, yv, beta: float) -> np.ndarray:
    """Item 3: (A^T A)^-1 A^T b with A = beta X' H^-1 and b = y' - X' H^-1 X^T y."""
    X, y, Xv, yv = _f64(X), _f64(y), _f64(Xv), _f64(yv)
    H = base_jacobian(X, beta)
    A = beta * np.linalg.solve(H, Xv.T).T          # X' H^-1 (H is symmetric)
    b = yv - Xv @ np.linalg.solve(H, X.T @ y)
    return np.linalg.solve(A.T @ A, A.T @ b)


def base_grad_lambda(w, lam, beta: float) -> np.ndarray:
    """dL_base/dlambda = -2 beta (w - lambda)."""
    return -2.0 * beta * (_f64(w) - _f64(lam))


def sama_meta_grad(Xv, yv, w, lam, beta: float, alpha: float, adam: "_o.Adam" = None, m=None, s=None, g_base=None):
    """SAMA's meta gradient at base parameters w (fp32 inputs, as the library receives them), step by step.
    ``adam=None`` is the SGD base optimiser (identity adaptation).  Returns a dict of float64 arrays."""
    w32 = np.ascontiguousarray(w, dtype=np.float32)
    g_meta = direct_grad(Xv, yv, w32)
    g32 = g_meta.astype(np.float32)          # the direct gradient crosses to the adaptation as fp32 storage
    if adam is None:
        adam = _o.Adam(identity=True)
    zeros = np.zeros_like(g32)
    p = _o.adapt(zeros if m is None else m, zeros if s is None else s, g_base, g32, adam)
    w_plus, w_minus, eps_fd, bad = _o.perturb(w32, p, alpha)
    if bad:
        mg = np.zeros_like(p)
    else:
        mg = -(base_grad_lambda(w_plus, lam, beta) - base_grad_lambda(w_minus, lam, beta)) / (2.0 * eps_fd)
    return {"g_meta": g_meta, "p": p, "w_plus": w_plus, "w_minus": w_minus, "eps_fd": eps_fd, "degenerate": bad,
            "metagrad": mg}


def cosine(a, b) -> float:
    a, b = _f64(a), _f64(b)
    return float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))
