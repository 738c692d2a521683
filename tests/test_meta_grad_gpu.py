"""GPU parity of the direct gradient dL_meta/dtheta (Eq. 1) against the CPU checker.

Inputs are conditioned so that no hidden pre-activation lies within max(1e-3, 1e-4 max|z|) of the
ReLU kink (see away_from_kinks).  Tolerance: every entry within 5e-5 of the largest magnitude in its
own layer block (weights or biases): three chained fp32 contractions of length up to K = 4096, each
with about sqrt(K) 2^-24 = 4e-6 of relative rounding, times a margin of 4.  Each entry is an fp32 sum
of B products (and the dz it is built from went through the fp32 forward pass), so its error scales
with the block's magnitude, not with the entry's own.  Both GEMM modes (fp32 FMA and the three-product
TF32 tensor-core path) are held to the same bound."""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_05674_b200 import workloads as W

pytestmark = pytest.mark.gpu

from gpu_util import B, Ctx, DEV, assert_fd_close, dev, run_step  # noqa: E402


def blocks(dims):
    out = []
    o = 0
    for l in range(len(dims) - 1):
        out.append((o, o + dims[l] * dims[l + 1]))
        o += dims[l] * dims[l + 1]
        out.append((o, o + dims[l + 1]))
        o += dims[l + 1]
    return out


def away_from_kinks(dims, theta, X, tau_abs=1e-3, tau_rel=1e-4):
    """Deterministically nudges hidden-layer biases until no hidden pre-activation lies within
    tau = max(tau_abs, tau_rel * max|z|) of zero.  At a ReLU kink the derivative is not determined
    within the rounding of the forward pass (both 0 and 1 are right; the rounding scales with the
    size of the pre-activations), so a well-posed comparison needs inputs that stay clear of it."""
    theta = theta.copy()
    L = len(dims) - 1
    h = X.astype(np.float64)
    o = 0
    for l in range(L - 1):
        nw = dims[l] * dims[l + 1]
        Wl = theta[o:o + nw].astype(np.float64).reshape(dims[l + 1], dims[l])
        bias = theta[o + nw:o + nw + dims[l + 1]]
        zw = h @ Wl.T
        tau = max(tau_abs, tau_rel * float(np.abs(zw).max()))
        for it in range(50):
            z = zw + bias.astype(np.float64)
            bad = np.unique(np.argwhere(np.abs(z) < tau)[:, 1])
            if bad.size == 0:
                break
            bias[bad] += np.float32(2.5 * tau * (1 + it))
        else:
            raise AssertionError("could not move the pre-activations off the kink")
        h = np.maximum(zw + bias.astype(np.float64), 0.0)
        o += nw + dims[l + 1]
    return theta


def check(dims, batch, seed, clean=True, gemm_mode=0):
    cfg, w = W.custom_mlp(dims, batch, seed=seed)
    theta = (w["theta"] + 0.05 * W.normal(seed, 99, cfg.n_params).astype(np.float32)).astype(np.float32)
    theta = away_from_kinks(dims, theta, w["X"])
    y = w["y_clean"] if clean else w["y"]
    loss_ref, g_ref = oracle.meta_grad(dims, theta, w["X"], y)
    with Ctx(cfg.n_params, batch, dims, gemm_mode) as ctx:
        g = torch.full((cfg.n_params,), float("nan"), dtype=torch.float32, device=DEV)
        loss = torch.zeros(1, dtype=torch.float32, device=DEV)
        th, X, yd = dev(theta), dev(w["X"]), dev(y)
        B.sama_meta_grad(ctx.h, ctx.mlp, th, X, yd, batch, g, loss)
        torch.cuda.synchronize()
        g1 = g.cpu().numpy()
        B.sama_meta_grad(ctx.h, ctx.mlp, th, X, yd, batch, g, None)
        torch.cuda.synchronize()
        assert np.array_equal(g.cpu().numpy(), g1)          # bitwise reproducible
        assert B.sama_device_status(ctx.h) == 0
    # the mean loss is a by-product; with the weight noise added above the logits reach ~100, so fp32 rounding of
    # the logits (sqrt(K) 2^-24 of their magnitude) shows up at a few 1e-6 of the loss.  A tensor-core
    # accumulator left to drift over the whole contraction (it rounds toward zero) would miss this by 4x.
    assert float(loss.item()) == pytest.approx(loss_ref, rel=2e-5)
    worst = 0.0
    for a, b in blocks(dims):
        scale = np.abs(g_ref[a:b]).max()
        if scale == 0:
            assert np.all(g1[a:b] == 0)
            continue
        worst = max(worst, float(np.abs(g1[a:b] - g_ref[a:b]).max() / scale))
    print("\n[meta_grad] dims=%s B=%d gemm_mode=%d: worst block-relative error %.2e" % (dims, batch, gemm_mode, worst))
    assert worst <= 5e-5, worst
    return theta, w, g1, g_ref


@pytest.mark.parametrize("dims,batch", [((12, 5), 1), ((33, 17, 12, 6), 7), ((100, 50, 3), 129), ((257, 130, 66, 11), 65),
                                        ((40, 200, 72, 24), 257)])
@pytest.mark.parametrize("gemm_mode", [1, 2])
def test_meta_grad_parity_ragged(dims, batch, gemm_mode):
    check(dims, batch, seed=sum(dims), gemm_mode=gemm_mode)


@pytest.mark.parametrize("gemm_mode", [1, 2])
def test_meta_grad_parity_tiny_and_mlp3072(gemm_mode):
    check(W.CONFIGS["tiny"].dims, W.CONFIGS["tiny"].batch, 0, gemm_mode=gemm_mode)
    check(W.CONFIGS["mlp3072"].dims, W.CONFIGS["mlp3072"].batch, 0, clean=False, gemm_mode=gemm_mode)


@pytest.mark.parametrize("gemm_mode", [1, 2])
def test_meta_grad_parity_head1024(gemm_mode):
    check(W.CONFIGS["head1024"].dims, 1024, 0, gemm_mode=gemm_mode)


@pytest.mark.parametrize("gemm_mode", [1, 2])
def test_meta_grad_parity_wide_dims_small_batch(gemm_mode):
    check(W.CONFIGS["wide4096"].dims, 48, 0, gemm_mode=gemm_mode)


def test_meta_grad_parity_on_the_paths_full_size_models_take():
    """A shape that takes what the 4096-wide model takes at its full batch, at a cost the CPU checker pays in
    seconds: batch x widest layer = 6 Mi elements, so the chain's small kernels run without dependent-launch
    overlap, and the first layer's forward product (1536 x 4096 x 512) is 96 CTA-pair tiles on 74 resident
    pairs, so its last 22 tiles are each shared by two pairs.  Both forward modes against one checker run."""
    dims, batch = (512, 4096, 32), 1536
    cached = {}
    for gemm_mode in (2, 1):
        cfg, w = W.custom_mlp(dims, batch, seed=17)
        if not cached:
            theta = (w["theta"] + 0.05 * W.normal(17, 99, cfg.n_params).astype(np.float32)).astype(np.float32)
            cached["theta"] = away_from_kinks(dims, theta, w["X"])
            cached["ref"] = oracle.meta_grad(dims, cached["theta"], w["X"], w["y_clean"])
        theta, (loss_ref, g_ref) = cached["theta"], cached["ref"]
        with Ctx(cfg.n_params, batch, dims, gemm_mode) as ctx:
            g = torch.full((cfg.n_params,), float("nan"), dtype=torch.float32, device=DEV)
            loss = torch.zeros(1, dtype=torch.float32, device=DEV)
            B.sama_meta_grad(ctx.h, ctx.mlp, dev(theta), dev(w["X"]), dev(w["y_clean"]), batch, g, loss)
            torch.cuda.synchronize()
            assert B.sama_device_status(ctx.h) == 0
            g1 = g.cpu().numpy()
        assert float(loss.item()) == pytest.approx(loss_ref, rel=2e-5)
        worst = 0.0
        for a, b in blocks(dims):
            scale = np.abs(g_ref[a:b]).max()
            worst = max(worst, float(np.abs(g1[a:b] - g_ref[a:b]).max() / scale))
        print("\n[meta_grad] dims=%s B=%d gemm_mode=%d: worst block-relative error %.2e" % (dims, batch, gemm_mode, worst))
        assert worst <= 5e-5, worst


def test_meta_grad_feeds_the_step():
    """The whole chain on the device: g_meta from a clean batch, then the SAMA step on the noisy batch."""
    cfg = W.CONFIGS["tiny"]
    w = W.mlp_workload(cfg, 3)
    _, wm = W.custom_mlp(cfg.dims, 64, seed=4)       # the clean meta batch
    _, g_ref = oracle.meta_grad(cfg.dims, w["theta"], wm["X"], wm["y_clean"])
    with Ctx(cfg.n_params, cfg.batch, cfg.dims) as ctx:
        g = torch.empty(cfg.n_params, dtype=torch.float32, device=DEV)
        B.sama_meta_grad(ctx.h, ctx.mlp, dev(w["theta"]), dev(wm["X"]), dev(wm["y_clean"]), 64, g, None)
        torch.cuda.synchronize()
        w2 = dict(w)
        w2["g_meta"] = g.cpu().numpy()
        got = run_step(ctx, cfg, w2, B.Adam(), 1.0)
    f = lambda x: float(np.float32(x))
    ref = oracle.step(cfg.dims, w["theta"], w["m"], w["s"], w["g_base"], g_ref.astype(np.float32),
                      oracle.Adam(f(1e-3), f(0.9), f(0.999), f(1e-8), 100), 1.0, w["X"], w["y"], w["lam"])
    assert_fd_close(got["metagrad"], ref["metagrad"], norm_tol=2e-3)


def test_meta_grad_argument_errors():
    cfg, w = W.custom_mlp((8, 4, 3), 5, seed=1)
    with Ctx(cfg.n_params, 5, (8, 4, 3)) as ctx:
        th, X, y = dev(w["theta"]), dev(w["X"]), dev(w["y"])
        g = torch.empty(cfg.n_params, dtype=torch.float32, device=DEV)

        def status(*a):
            with pytest.raises(B.SamaError) as e:
                B.sama_meta_grad(*a)
            return e.value.status

        assert status(ctx.h, ctx.mlp, None, X, y, 5, g) == B.SAMA_ERR_NULL
        assert status(ctx.h, ctx.mlp, th, X, y, 6, g) == B.SAMA_ERR_SIZE
        assert status(ctx.h, ctx.mlp, th, X, y, 0, g) == B.SAMA_ERR_SIZE
        assert status(ctx.h, ctx.mlp, th, X, y, 5, th) == B.SAMA_ERR_OVERLAP
        assert status(ctx.h, B.MLP((8, 64, 3)), th, X, y, 5, g) == B.SAMA_ERR_SIZE
        ybad = w["y"].copy()
        ybad[2] = 7
        B.sama_meta_grad(ctx.h, ctx.mlp, th, X, dev(ybad), 5, g)
        assert B.sama_device_status(ctx.h) == B.SAMA_DEV_BAD_LABEL
    with Ctx(cfg.n_params) as ctx:   # no model in the context: no workspace
        assert status(ctx.h, B.MLP((8, 4, 3)), th, X, y, 5, g) == B.SAMA_ERR_SIZE
