"""Helpers for the GPU parity tests: run the C-ABI path on seeded inputs and
bring results back as numpy arrays, plus the tolerance checks the tests share."""
from __future__ import annotations

import numpy as np
import torch

from paper_2310_05674_b200 import binding as B

DEV = "cuda:0"


def dev(a):
    """Device copy; an empty array still gets a valid (4-element) allocation so that n = 0 calls have pointers."""
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.size == 0:
        return torch.zeros(4, dtype=torch.from_numpy(a).dtype, device=DEV)
    return torch.from_numpy(a).to(DEV)


def unaligned(a: np.ndarray, shift: int = 1) -> torch.Tensor:
    """Device copy of ``a`` whose first element sits ``shift`` floats past a 16-byte boundary."""
    buf = torch.empty(a.size + 8, dtype=torch.float32, device=DEV)
    view = buf[shift:shift + a.size]
    view.copy_(torch.from_numpy(np.ascontiguousarray(a)))
    assert view.data_ptr() % 16 == 4 * shift
    return view


class Ctx:
    def __init__(self, max_n, max_batch=0, dims=None, gemm_mode=0):
        self.mlp = B.MLP(dims) if dims is not None else None
        self.h = B.sama_create(0, max_n, max_batch, self.mlp)
        if gemm_mode:
            B.sama_set_gemm_mode(self.h, gemm_mode)

    def close(self):
        if self.h:
            torch.cuda.synchronize()
            B.sama_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def run_adapt(ctx, w, adam, use_gbase=True, inplace=False, shift=0):
    mk = (lambda a: unaligned(a, shift)) if shift else dev
    m, s, gm = mk(w["m"]), mk(w["s"]), mk(w["g_meta"])
    gb = mk(w["g_base"]) if use_gbase else None
    n = w["g_meta"].size
    if inplace:
        p = gm
    elif shift:
        p = unaligned(np.zeros(n, np.float32), shift)
    else:
        p = torch.empty(max(n, 4), dtype=torch.float32, device=DEV)
    ss = torch.zeros(1, dtype=torch.float64, device=DEV)
    B.sama_adapt(ctx.h, n, m, s, gb, gm, adam, p, ss)
    torch.cuda.synchronize()
    return p.cpu().numpy()[:n], float(ss.item()), p, ss


def run_step(ctx, cfg, w, adam, alpha, use_gbase=True, want_losses=True, want_plus=True, want_minus=True):
    n, Bsz = w["theta"].size, cfg.batch
    t = {k: dev(w[k]) for k in ["theta", "m", "s", "g_meta", "X", "y", "lam"]}
    gb = dev(w["g_base"]) if use_gbase else None
    f = lambda k: torch.full((k,), float("nan"), dtype=torch.float32, device=DEV)
    p, tp, tm, mg, lp, lm = f(n), f(n), f(n), f(Bsz), f(Bsz), f(Bsz)
    B.sama_step(ctx.h, ctx.mlp, n, t["theta"], t["m"], t["s"], gb, t["g_meta"], adam, alpha, t["X"], t["y"],
                t["lam"], Bsz, p, tp if want_plus else None, tm if want_minus else None, mg,
                lp if want_losses else None, lm if want_losses else None)
    torch.cuda.synchronize()
    out = {"p": p.cpu().numpy(), "theta_plus": tp.cpu().numpy(), "theta_minus": tm.cpu().numpy(),
           "metagrad": mg.cpu().numpy(), "loss_plus": lp.cpu().numpy(), "loss_minus": lm.cpu().numpy(),
           "eps_fd": read_f32(B.sama_ctx_eps_fd(ctx.h)), "sumsq": read_f64(B.sama_ctx_sumsq(ctx.h)),
           "status": B.sama_device_status(ctx.h)}
    return out


def read_f32(addr: int) -> float:
    t = torch.empty(1, dtype=torch.float32, device=DEV)
    _memcpy_d2d(t.data_ptr(), addr, 4)
    return float(t.item())


def read_f64(addr: int) -> float:
    t = torch.empty(1, dtype=torch.float64, device=DEV)
    _memcpy_d2d(t.data_ptr(), addr, 8)
    return float(t.item())


_rt = None


def _cudart():
    """The CUDA runtime torch has already loaded (found again by its soname)."""
    global _rt
    if _rt is None:
        import ctypes
        for name in ("libcudart.so.12", "libcudart.so.13", "libcudart.so"):
            try:
                _rt = ctypes.CDLL(name)
                break
            except OSError:
                continue
        assert _rt is not None, "libcudart not found"
        _rt.cudaMemcpy.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
    return _rt


def _memcpy_d2d(dst: int, src: int, nbytes: int):
    torch.cuda.synchronize()
    err = _cudart().cudaMemcpy(dst, src, nbytes, 3)  # cudaMemcpyDeviceToDevice
    assert int(err) == 0, err
    torch.cuda.synchronize()


# ---- tolerances -----------------------------------------------------------

def rel_err_elementwise(got, ref):
    """max over elements of |got-ref| / max(|ref|, 1e-3 max|ref|)."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    scale = np.maximum(np.abs(ref), 1e-3 * np.abs(ref).max())
    scale = np.where(scale > 0, scale, 1.0)
    return float((np.abs(got - ref) / scale).max())


def assert_adapt_close(got, ref, what="p"):
    """Relative 1e-5 for adaptation / perturbation outputs (elements below
    1e-3 of the largest magnitude are held to 1e-5 of that floor)."""
    e = rel_err_elementwise(got, ref)
    assert e <= 1e-5, "%s: max rel err %.3e" % (what, e)
    return e


def fd_errors(got, ref):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    diff = np.abs(got - ref)
    viol = diff > np.maximum(2e-3 * np.abs(ref), 1e-6)
    nrm = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    rel = diff / np.maximum(np.abs(ref), 1e-300)
    return {"violations": int(viol.sum()), "norm_rel": nrm, "max_abs": float(diff.max()),
            "max_rel": float(rel.max()), "p999_rel": float(np.quantile(rel, 0.999)),
            "median_rel": float(np.median(rel))}


def assert_fd_close(got, ref, what="metagrad", norm_tol=2e-3):
    """FD meta-gradient: |a-b| <= max(2e-3 |b|, 1e-6) elementwise (the stated
    bar), and the same relative 2e-3 on the whole vector in the 2-norm, which is
    scale-free and so still bites when the 1/B factor pushes every entry under
    the absolute floor.  Callers pass a looser norm bound only for the fp32 FMA
    forward at alpha = 1e-2 (its chain of K sequential roundings per logit is
    amplified by 1/(2 eps_fd))."""
    e = fd_errors(got, ref)
    assert e["violations"] == 0, (what, e)
    assert e["norm_rel"] <= norm_tol, (what, e)
    return e
