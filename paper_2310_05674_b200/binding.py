"""Thin ctypes binding of ``libsama.so`` (declared in ``include/sama.h``).

Argument marshalling only: every function here has the name and the argument
order of the C entry point it calls, takes torch tensors (device memory, or
pinned host memory for ``sama_step_host``) or raw integer addresses, and returns
the C status code after raising ``SamaError`` for a negative one.  Nothing is
computed in Python, and there is no fallback: if the shared library has not
been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsama.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libsama.so is missing: build it with `python -m paper_2310_05674_b200.build` "
        "(needs nvcc; there is no CPU or PyTorch fallback)")

lib = C.CDLL(LIB_PATH)

SAMA_OK = 0
SAMA_ERR_NULL, SAMA_ERR_ALIGN, SAMA_ERR_SIZE, SAMA_ERR_PARAM = -1, -2, -3, -4
SAMA_ERR_OVERLAP, SAMA_ERR_CUDA, SAMA_ERR_NOMEM, SAMA_ERR_UNSUPPORTED = -5, -6, -7, -8
SAMA_DEV_DEGENERATE_NORM, SAMA_DEV_BAD_LABEL, SAMA_DEV_TIMEOUT = 1, 2, 4


class SamaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, sama_status_string(status), status))


class sama_adam_t(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("step", C.c_int64), ("bias_correction", C.c_int32), ("drop_eps_term", C.c_int32),
                ("identity", C.c_int32)]


class sama_kernel_time_t(C.Structure):
    _fields_ = [("kind", C.c_int32), ("layer", C.c_int32), ("ms", C.c_float), ("launches", C.c_int32)]


KERNEL_KINDS = {0: "adapt_sumsq", 1: "sumsq", 2: "perturb", 3: "gemm_ffma", 4: "ce_fd", 5: "split_tf32",
                6: "gemm_tf32x3", 7: "head_ce_fd", 8: "perturb_split", 9: "meta_gemm", 10: "meta_aux",
                11: "reweight_fd", 12: "biasreg_grad", 13: "biasreg_fd", 14: "fused_sweep"}


class sama_mlp_t(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("dims", C.POINTER(C.c_int32))]


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

    def c(self) -> sama_adam_t:
        return sama_adam_t(self.lr, self.beta1, self.beta2, self.eps, int(self.step), int(self.bias_correction),
                           int(self.drop_eps_term), int(self.identity))


class MLP:
    """Host description of the base model: dims = (d_0, ..., d_L)."""

    def __init__(self, dims: Sequence[int]):
        self.dims = tuple(int(d) for d in dims)
        self._arr = (C.c_int32 * len(self.dims))(*self.dims)
        self._c = sama_mlp_t(len(self.dims) - 1, C.cast(self._arr, C.POINTER(C.c_int32)))

    def c(self):
        return C.byref(self._c)


_vp = C.c_void_p
lib.sama_create.argtypes = [C.POINTER(_vp), C.c_int, C.c_int64, C.c_int32, C.POINTER(sama_mlp_t)]
lib.sama_destroy.argtypes = [_vp]
lib.sama_adapt.argtypes = [_vp, C.c_int64, _vp, _vp, _vp, _vp, C.POINTER(sama_adam_t), _vp, _vp, _vp]
lib.sama_adapt_noalloc.argtypes = [C.c_int64, _vp, _vp, _vp, _vp, C.POINTER(sama_adam_t), _vp, _vp, _vp]
lib.sama_perturb.argtypes = [_vp, C.c_int64, _vp, _vp, _vp, C.c_float, _vp, _vp, _vp, _vp]
lib.sama_fd_metagrad.argtypes = [_vp, C.POINTER(sama_mlp_t), _vp, _vp, _vp, _vp, _vp, C.c_int32, _vp, _vp, _vp,
                                 _vp, _vp]
lib.sama_step.argtypes = [_vp, C.POINTER(sama_mlp_t), C.c_int64, _vp, _vp, _vp, _vp, _vp, C.POINTER(sama_adam_t),
                          C.c_float, _vp, _vp, _vp, C.c_int32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.sama_fd_metagrad_reweight.argtypes = [_vp, C.c_int32, _vp, _vp, _vp, C.c_int32, _vp, _vp, C.c_int32, _vp, _vp]
lib.sama_ctx_loss_diff.argtypes = [_vp]
lib.sama_ctx_loss_diff.restype = _vp
lib.sama_step_reweight.argtypes = [_vp, C.POINTER(sama_mlp_t), C.c_int64, _vp, _vp, _vp, _vp, _vp,
                                   C.POINTER(sama_adam_t), C.c_float, _vp, _vp, C.c_int32, C.c_int32, _vp, _vp, _vp,
                                   _vp, _vp, _vp, _vp, _vp]
lib.sama_biasreg_direct_grad.argtypes = [_vp, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, _vp, _vp]
lib.sama_biasreg_fd_metagrad.argtypes = [_vp, C.c_int64, _vp, _vp, _vp, C.c_float, _vp, _vp, _vp]
lib.sama_biasreg_step.argtypes = [_vp, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, C.c_float, _vp, _vp, _vp,
                                  C.POINTER(sama_adam_t), C.c_float, _vp, _vp, _vp, _vp, _vp, _vp]
lib.sama_meta_grad.argtypes = [_vp, C.POINTER(sama_mlp_t), _vp, _vp, _vp, C.c_int32, _vp, _vp, _vp]
lib.sama_step_host.argtypes = [_vp, C.POINTER(sama_mlp_t), C.c_int64, _vp, _vp, _vp, _vp, _vp,
                               C.POINTER(sama_adam_t), C.c_float, _vp, _vp, _vp, C.c_int32, _vp, _vp, _vp, _vp]
lib.sama_ctx_sumsq.argtypes = [_vp]
lib.sama_ctx_sumsq.restype = _vp
lib.sama_ctx_eps_fd.argtypes = [_vp]
lib.sama_ctx_eps_fd.restype = _vp
lib.sama_device_status.argtypes = [_vp, _vp, C.POINTER(C.c_int32)]
lib.sama_selftest_wait_expiry.argtypes = [_vp, C.c_int64, _vp, _vp]
lib.sama_last_cuda_error.argtypes = [_vp]
lib.sama_mlp_param_count.argtypes = [C.POINTER(sama_mlp_t)]
lib.sama_mlp_param_count.restype = C.c_int64
lib.sama_status_string.argtypes = [C.c_int]
lib.sama_status_string.restype = C.c_char_p
lib.sama_set_gemm_mode.argtypes = [_vp, C.c_int]
lib.sama_launch_count.argtypes = [_vp]
lib.sama_last_forward_path.argtypes = [_vp]
lib.sama_launch_count.restype = C.c_int64
lib.sama_profile_enable.argtypes = [_vp, C.c_int32]
lib.sama_profile_collect.argtypes = [_vp, C.POINTER(sama_kernel_time_t), C.c_int32, C.POINTER(C.c_int32)]


def _ptr(x) -> Optional[int]:
    """Address of a tensor's first element; ints and None pass through."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(rc: int, where: str) -> int:
    if rc < 0:
        raise SamaError(rc, where)
    return rc


def sama_status_string(status: int) -> str:
    return lib.sama_status_string(int(status)).decode()


def sama_mlp_param_count(mlp: MLP) -> int:
    return int(lib.sama_mlp_param_count(mlp.c()))


def sama_create(device: int, max_n: int, max_batch: int, mlp: Optional[MLP]) -> int:
    out = _vp()
    _check(lib.sama_create(C.byref(out), int(device), int(max_n), int(max_batch), mlp.c() if mlp else None),
           "sama_create")
    return out.value


def sama_destroy(ctx: int) -> int:
    return _check(lib.sama_destroy(ctx), "sama_destroy")


def sama_adapt(ctx, n, m, s, g_base, g_meta, adam: Adam, p_out, sumsq_out=None, stream=None) -> int:
    a = adam.c()
    return _check(lib.sama_adapt(ctx, int(n), _ptr(m), _ptr(s), _ptr(g_base), _ptr(g_meta), C.byref(a),
                                 _ptr(p_out), _ptr(sumsq_out), _stream(stream)), "sama_adapt")


SAMA_NOALLOC_MAX_N = 1 << 30


def sama_adapt_noalloc(n, m, s, g_base, g_meta, adam: Adam, p_out, sumsq_out, stream=None) -> int:
    """sama_adapt for callers that must not allocate: no context, static device scratch, current device."""
    a = adam.c()
    return _check(lib.sama_adapt_noalloc(int(n), _ptr(m), _ptr(s), _ptr(g_base), _ptr(g_meta), C.byref(a),
                                         _ptr(p_out), _ptr(sumsq_out), _stream(stream)), "sama_adapt_noalloc")


def sama_perturb(ctx, n, theta, p, p_sumsq, alpha, theta_plus, theta_minus, eps_fd_out=None, stream=None) -> int:
    return _check(lib.sama_perturb(ctx, int(n), _ptr(theta), _ptr(p), _ptr(p_sumsq), float(alpha),
                                   _ptr(theta_plus), _ptr(theta_minus), _ptr(eps_fd_out), _stream(stream)),
                  "sama_perturb")


def sama_fd_metagrad(ctx, mlp: MLP, theta_plus, theta_minus, X, y, lam, B, eps_fd, metagrad_out,
                     loss_plus_out=None, loss_minus_out=None, stream=None) -> int:
    return _check(lib.sama_fd_metagrad(ctx, mlp.c(), _ptr(theta_plus), _ptr(theta_minus), _ptr(X), _ptr(y),
                                       _ptr(lam), int(B), _ptr(eps_fd), _ptr(metagrad_out), _ptr(loss_plus_out),
                                       _ptr(loss_minus_out), _stream(stream)), "sama_fd_metagrad")


def sama_step(ctx, mlp: MLP, n, theta, m, s, g_base, g_meta, adam: Adam, alpha, X, y, lam, B, p_out, theta_plus,
              theta_minus, metagrad_out, loss_plus_out=None, loss_minus_out=None, stream=None) -> int:
    a = adam.c()
    return _check(lib.sama_step(ctx, mlp.c(), int(n), _ptr(theta), _ptr(m), _ptr(s), _ptr(g_base), _ptr(g_meta),
                                C.byref(a), float(alpha), _ptr(X), _ptr(y), _ptr(lam), int(B), _ptr(p_out),
                                _ptr(theta_plus), _ptr(theta_minus), _ptr(metagrad_out), _ptr(loss_plus_out),
                                _ptr(loss_minus_out), _stream(stream)), "sama_step")


def sama_ctx_loss_diff(ctx) -> int:
    return lib.sama_ctx_loss_diff(ctx)


def sama_fd_metagrad_reweight(ctx, B, loss_plus, loss_minus, loss_diff, hidden, lambda_r, eps_fd, B_norm,
                              metagrad_r_out, stream=None) -> int:
    return _check(lib.sama_fd_metagrad_reweight(ctx, int(B), _ptr(loss_plus), _ptr(loss_minus), _ptr(loss_diff),
                                                int(hidden),
                                                _ptr(lambda_r), _ptr(eps_fd), int(B_norm), _ptr(metagrad_r_out),
                                                _stream(stream)), "sama_fd_metagrad_reweight")


def sama_step_reweight(ctx, mlp: MLP, n, theta, m, s, g_base, g_meta, adam: Adam, alpha, X, y, B, hidden, lambda_r,
                       p_out, theta_plus, theta_minus, metagrad_r_out, loss_plus_out=None, loss_minus_out=None,
                       stream=None) -> int:
    a = adam.c()
    return _check(lib.sama_step_reweight(ctx, mlp.c(), int(n), _ptr(theta), _ptr(m), _ptr(s), _ptr(g_base),
                                         _ptr(g_meta), C.byref(a), float(alpha), _ptr(X), _ptr(y), int(B),
                                         int(hidden), _ptr(lambda_r), _ptr(p_out), _ptr(theta_plus),
                                         _ptr(theta_minus), _ptr(metagrad_r_out), _ptr(loss_plus_out),
                                         _ptr(loss_minus_out), _stream(stream)), "sama_step_reweight")


def sama_biasreg_direct_grad(ctx, d, n_val, Xv, yv, w, g_meta_out, meta_loss_out=None, stream=None) -> int:
    return _check(lib.sama_biasreg_direct_grad(ctx, int(d), int(n_val), _ptr(Xv), _ptr(yv), _ptr(w),
                                               _ptr(g_meta_out), _ptr(meta_loss_out), _stream(stream)),
                  "sama_biasreg_direct_grad")


def sama_biasreg_fd_metagrad(ctx, d, w_plus, w_minus, lam, beta, eps_fd, metagrad_out, stream=None) -> int:
    return _check(lib.sama_biasreg_fd_metagrad(ctx, int(d), _ptr(w_plus), _ptr(w_minus), _ptr(lam), float(beta),
                                               _ptr(eps_fd), _ptr(metagrad_out), _stream(stream)),
                  "sama_biasreg_fd_metagrad")


def sama_biasreg_step(ctx, d, n_val, Xv, yv, w, lam, beta, m, s, g_base, adam: Adam, alpha, g_meta_out, p_out,
                      w_plus, w_minus, metagrad_out, stream=None) -> int:
    a = adam.c()
    return _check(lib.sama_biasreg_step(ctx, int(d), int(n_val), _ptr(Xv), _ptr(yv), _ptr(w), _ptr(lam), float(beta),
                                        _ptr(m), _ptr(s), _ptr(g_base), C.byref(a), float(alpha), _ptr(g_meta_out),
                                        _ptr(p_out), _ptr(w_plus), _ptr(w_minus), _ptr(metagrad_out),
                                        _stream(stream)), "sama_biasreg_step")


def sama_meta_grad(ctx, mlp: MLP, theta, X_meta, y_meta, B, g_meta_out, loss_out=None, stream=None) -> int:
    return _check(lib.sama_meta_grad(ctx, mlp.c(), _ptr(theta), _ptr(X_meta), _ptr(y_meta), int(B),
                                     _ptr(g_meta_out), _ptr(loss_out), _stream(stream)), "sama_meta_grad")


def sama_step_host(ctx, mlp: MLP, n, theta_host, m_host, s_host, g_base_host, g_meta_host, adam: Adam, alpha,
                   X_host, y_host, lam_host, B, metagrad_out_host, eps_fd_out_host=None,
                   theta_minus_out_host=None, stream=None) -> int:
    a = adam.c()
    return _check(lib.sama_step_host(ctx, mlp.c(), int(n), _ptr(theta_host), _ptr(m_host), _ptr(s_host),
                                     _ptr(g_base_host), _ptr(g_meta_host), C.byref(a), float(alpha),
                                     _ptr(X_host), _ptr(y_host), _ptr(lam_host), int(B),
                                     _ptr(metagrad_out_host), _ptr(eps_fd_out_host),
                                     _ptr(theta_minus_out_host), _stream(stream)), "sama_step_host")


def sama_ctx_sumsq(ctx) -> int:
    return lib.sama_ctx_sumsq(ctx)


def sama_ctx_eps_fd(ctx) -> int:
    return lib.sama_ctx_eps_fd(ctx)


def sama_device_status(ctx, stream=None) -> int:
    out = C.c_int32(0)
    _check(lib.sama_device_status(ctx, _stream(stream), C.byref(out)), "sama_device_status")
    return out.value


def sama_selftest_wait_expiry(ctx, limit_cycles, waited_cycles_out=None, stream=None) -> int:
    return _check(lib.sama_selftest_wait_expiry(ctx, int(limit_cycles), _ptr(waited_cycles_out), _stream(stream)),
                  "sama_selftest_wait_expiry")


def sama_last_cuda_error(ctx) -> int:
    return int(lib.sama_last_cuda_error(ctx))


def sama_set_gemm_mode(ctx, mode: int) -> int:
    return _check(lib.sama_set_gemm_mode(ctx, int(mode)), "sama_set_gemm_mode")


def sama_launch_count(ctx) -> int:
    return int(lib.sama_launch_count(ctx))


def sama_last_forward_path(ctx) -> int:
    return int(lib.sama_last_forward_path(ctx))


def sama_profile_enable(ctx, on) -> int:
    """on: 0 / False = off, 1 / True = one event pair per launch, 2 = one pair per run of same-kind launches."""
    return _check(lib.sama_profile_enable(ctx, int(on)), "sama_profile_enable")


def sama_profile_collect(ctx, capacity: int = 65536, with_launches: bool = False):
    """Returns [(kind, layer, ms), ...] in launch order ((kind, layer, ms, launches) with ``with_launches``)."""
    buf = (sama_kernel_time_t * capacity)()
    cnt = C.c_int32(0)
    _check(lib.sama_profile_collect(ctx, buf, capacity, C.byref(cnt)), "sama_profile_collect")
    if with_launches:
        return [(buf[i].kind, buf[i].layer, buf[i].ms, buf[i].launches) for i in range(cnt.value)]
    return [(buf[i].kind, buf[i].layer, buf[i].ms) for i in range(cnt.value)]
