"""ctypes front end of the CPU checker (``sama_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
shares no code with it.  ``build()`` compiles the C++ file with g++ (-O2, one
thread, no fast-math) into ``oracle/libsama_oracle.so``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sama_oracle.cpp")
_LIB = os.path.join(_HERE, "libsama_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Adam(C.Structure):
    _fields_ = [("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("step", C.c_int64), ("bias_correction", C.c_int32), ("drop_eps_term", C.c_int32),
                ("identity", C.c_int32)]


@dataclass
class Adam:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    step: int = 100
    bias_correction: bool = True
    drop_eps_term: bool = False
    identity: bool = False

    def _c(self) -> _Adam:
        return _Adam(self.lr, self.beta1, self.beta2, self.eps, self.step, int(self.bias_correction),
                     int(self.drop_eps_term), int(self.identity))


def _bind(lib):
    fp, dp, ip = C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int32)
    ap = C.POINTER(_Adam)
    lib.sama_oracle_adapt.argtypes = [C.c_int64, fp, fp, fp, fp, ap, dp]
    lib.sama_oracle_adapt.restype = None
    lib.sama_oracle_sumsq.argtypes = [C.c_int64, dp]
    lib.sama_oracle_sumsq.restype = C.c_double
    lib.sama_oracle_perturb.argtypes = [C.c_int64, fp, dp, C.c_double, dp, dp, dp]
    lib.sama_oracle_perturb.restype = C.c_int
    lib.sama_oracle_perturb_given_sumsq.argtypes = [C.c_int64, fp, dp, C.c_double, C.c_double, dp, dp, dp]
    lib.sama_oracle_perturb_given_sumsq.restype = C.c_int
    lib.sama_oracle_losses.argtypes = [C.c_int32, ip, dp, fp, ip, C.c_int32, dp, dp]
    lib.sama_oracle_losses.restype = None
    lib.sama_oracle_fd.argtypes = [C.c_int32, dp, dp, fp, C.c_double, C.c_int32, dp]
    lib.sama_oracle_fd.restype = None
    lib.sama_oracle_meta_grad.argtypes = [C.c_int32, ip, fp, fp, ip, C.c_int32, dp]
    lib.sama_oracle_meta_grad.restype = C.c_double
    lib.sama_oracle_reweight_grad.argtypes = [C.c_int32, dp, C.c_int32, fp, C.c_int32, dp, dp]
    lib.sama_oracle_reweight_grad.restype = None
    lib.sama_oracle_fd_reweight.argtypes = [C.c_int32, dp, dp, C.c_int32, fp, C.c_double, C.c_int32, dp]
    lib.sama_oracle_fd_reweight.restype = None
    lib.sama_oracle_step.argtypes = [C.c_int32, ip, C.c_int64, fp, fp, fp, fp, fp, ap, C.c_double,
                                     fp, ip, fp, C.c_int32, C.c_int32, dp, dp, dp, dp, dp, dp, dp]
    lib.sama_oracle_step.restype = C.c_int
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(C.CDLL(build()))
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def adapt(m, s, g_base, g_meta, adam: Adam) -> np.ndarray:
    """S1: p = (du_adam/dg_base) * g_meta, in double.  ``g_base=None`` uses g := m."""
    m, s, g_meta = _f32(m), _f32(s), _f32(g_meta)
    gb = None if g_base is None else _f32(g_base)
    n = g_meta.size
    p = np.empty(n, dtype=np.float64)
    h = adam._c()
    _load().sama_oracle_adapt(n, _p(m, C.c_float), _p(s, C.c_float), _p(gb, C.c_float),
                              _p(g_meta, C.c_float), C.byref(h), _p(p, C.c_double))
    return p


def sumsq(p) -> float:
    p = _f64(p)
    return float(_load().sama_oracle_sumsq(p.size, _p(p, C.c_double)))


def perturb(theta, p, alpha: float):
    """S2+S3: returns (theta_plus, theta_minus, eps_fd, degenerate) in double."""
    theta, p = _f32(theta), _f64(p)
    n = theta.size
    tp, tm = np.empty(n, dtype=np.float64), np.empty(n, dtype=np.float64)
    eps = C.c_double(0.0)
    bad = _load().sama_oracle_perturb(n, _p(theta, C.c_float), _p(p, C.c_double), float(alpha),
                                      _p(tp, C.c_double), _p(tm, C.c_double), C.byref(eps))
    return tp, tm, eps.value, bool(bad)


def perturb_given_sumsq(theta, p, sumsq_all: float, alpha: float):
    """S3 on a slice, with the sum of squares of the whole vector supplied."""
    theta, p = _f32(theta), _f64(p)
    n = theta.size
    tp, tm = np.empty(n, dtype=np.float64), np.empty(n, dtype=np.float64)
    eps = C.c_double(0.0)
    bad = _load().sama_oracle_perturb_given_sumsq(n, _p(theta, C.c_float), _p(p, C.c_double), float(sumsq_all),
                                                  float(alpha), _p(tp, C.c_double), _p(tm, C.c_double),
                                                  C.byref(eps))
    return tp, tm, eps.value, bool(bad)


def losses(dims: Sequence[int], theta, X, y, want_logits: bool = False):
    """S4: per-sample cross-entropy (and optionally logits) at parameters ``theta``."""
    dims_a = _i32(dims)
    theta, X, y = _f64(theta), _f32(X), _i32(y)
    B = y.size
    out = np.empty(B, dtype=np.float64)
    logits = np.empty((B, int(dims_a[-1])), dtype=np.float64) if want_logits else None
    _load().sama_oracle_losses(len(dims_a) - 1, _p(dims_a, C.c_int32), _p(theta, C.c_double),
                               _p(X, C.c_float), _p(y, C.c_int32), B, _p(out, C.c_double),
                               _p(logits, C.c_double))
    return (out, logits) if want_logits else out


def meta_grad(dims: Sequence[int], theta, X, y):
    """Direct gradient (Eq. 1): (L_meta, dL_meta/dtheta) of the mean cross-entropy on a clean batch, in double."""
    dims_a = _i32(dims)
    theta, X, y = _f32(theta), _f32(X), _i32(y)
    g = np.empty(theta.size, dtype=np.float64)
    loss = _load().sama_oracle_meta_grad(len(dims_a) - 1, _p(dims_a, C.c_int32), _p(theta, C.c_float),
                                         _p(X, C.c_float), _p(y, C.c_int32), y.size, _p(g, C.c_double))
    return float(loss), g


def fd(loss_plus, loss_minus, lam, eps_fd: float, B_norm: int) -> np.ndarray:
    """S5: central-difference meta-gradient w.r.t. the weight logits."""
    lp, lm, lam = _f64(loss_plus), _f64(loss_minus), _f32(lam)
    out = np.empty(lp.size, dtype=np.float64)
    _load().sama_oracle_fd(lp.size, _p(lp, C.c_double), _p(lm, C.c_double), _p(lam, C.c_float),
                           float(eps_fd), int(B_norm), _p(out, C.c_double))
    return out


def reweight_grad(loss, lambda_r, B_norm: Optional[int] = None):
    """dL_base/dlambda_r at fixed theta for the shared reweighting network of Sec. 4.1
    (lambda_r = v1[H], c1[H], v2[H], c2); returns (gradient [3H + 1], per-sample weights)."""
    loss, lambda_r = _f64(loss), _f32(lambda_r)
    H = (lambda_r.size - 1) // 3
    assert lambda_r.size == 3 * H + 1
    g, wts = np.empty(3 * H + 1, dtype=np.float64), np.empty(loss.size, dtype=np.float64)
    _load().sama_oracle_reweight_grad(loss.size, _p(loss, C.c_double), H, _p(lambda_r, C.c_float),
                                      int(loss.size if B_norm is None else B_norm), _p(g, C.c_double),
                                      _p(wts, C.c_double))
    return g, wts


def fd_reweight(loss_plus, loss_minus, lambda_r, eps_fd: float, B_norm: Optional[int] = None) -> np.ndarray:
    """Eq. 5 with the shared reweighting network: central difference of dL_base/dlambda_r between theta+ and theta-."""
    lp, lm, lambda_r = _f64(loss_plus), _f64(loss_minus), _f32(lambda_r)
    H = (lambda_r.size - 1) // 3
    assert lambda_r.size == 3 * H + 1
    out = np.empty(3 * H + 1, dtype=np.float64)
    _load().sama_oracle_fd_reweight(lp.size, _p(lp, C.c_double), _p(lm, C.c_double), H, _p(lambda_r, C.c_float),
                                    float(eps_fd), int(lp.size if B_norm is None else B_norm), _p(out, C.c_double))
    return out


def step(dims: Sequence[int], theta, m, s, g_base, g_meta, adam: Adam, alpha: float, X, y, lam,
         B_norm: Optional[int] = None):
    """S1..S5 chained on the rows of X given; returns a dict of double arrays."""
    dims_a = _i32(dims)
    theta, m, s, g_meta = _f32(theta), _f32(m), _f32(s), _f32(g_meta)
    gb = None if g_base is None else _f32(g_base)
    X, y, lam = _f32(X), _i32(y), _f32(lam)
    n, cnt = theta.size, y.size
    B_norm = cnt if B_norm is None else int(B_norm)
    p, tp, tm = (np.empty(n, dtype=np.float64) for _ in range(3))
    lp, lm, mg = (np.empty(cnt, dtype=np.float64) for _ in range(3))
    eps = C.c_double(0.0)
    h = adam._c()
    bad = _load().sama_oracle_step(len(dims_a) - 1, _p(dims_a, C.c_int32), n, _p(theta, C.c_float),
                                   _p(m, C.c_float), _p(s, C.c_float), _p(gb, C.c_float),
                                   _p(g_meta, C.c_float), C.byref(h), float(alpha),
                                   _p(X, C.c_float), _p(y, C.c_int32), _p(lam, C.c_float), cnt, B_norm,
                                   _p(p, C.c_double), _p(tp, C.c_double), _p(tm, C.c_double), C.byref(eps),
                                   _p(lp, C.c_double), _p(lm, C.c_double), _p(mg, C.c_double))
    return {"p": p, "theta_plus": tp, "theta_minus": tm, "eps_fd": eps.value, "degenerate": bool(bad),
            "loss_plus": lp, "loss_minus": lm, "metagrad": mg}
