"""GPU parity of Eq. 5 with the shared reweighting network of Sec. 4.1 against the CPU checker.

Tolerance.  On given losses (no forward pass involved) the kernel is held to the stated finite-difference bar,
relative 2e-3, on the whole vector in the 2-norm and elementwise with a floor of 2e-3 of the largest entry.
Through the whole step, every entry of the result is a SUM over the batch of signed per-sample terms
t_ki = -[f_k(l+_i) - f_k(l-_i)] / (2 eps_fd B); the stated bar is a bar on each sample's finite difference, so a sum
of them is held to 2e-3 sum_i |t_ki| (the forward-error bound of a sum whose terms are each good to 2e-3), not
to 2e-3 of the sum's own size: the terms cancel (on the 3072-wide workload ||sum_i |t_i||| is 24 times
||sum_i t_i||), and rounding theta+- to fp32 storage alone moves the sum by 1e-3 of its size there."""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_05674_b200 import workloads as W

pytestmark = pytest.mark.gpu

from gpu_util import B, Ctx, DEV, dev, run_step  # noqa: E402


def lambda_r(hidden, seed, scale=0.6):
    rng = np.random.default_rng(seed)
    lam = (scale * rng.normal(size=3 * hidden + 1)).astype(np.float32)
    lam[hidden:2 * hidden] += 0.3          # most units active somewhere in the range of the losses
    return lam


def close(got, ref, what):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    nrm = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert nrm <= 2e-3, (what, nrm)
    assert np.all(np.abs(got - ref) <= 2e-3 * np.maximum(np.abs(ref), np.abs(ref).max())), what
    return nrm


@pytest.mark.parametrize("batch,hidden", [(1, 1), (7, 3), (129, 100), (2048, 256), (4096, 33)])
def test_fd_reweight_on_given_losses(batch, hidden):
    rng = np.random.default_rng(batch + hidden)
    lp = (np.abs(rng.normal(size=batch)) * 2 + 0.05).astype(np.float32)
    lm = (lp.astype(np.float64) * (1 + 1e-3 * rng.normal(size=batch))).astype(np.float32)
    lam = lambda_r(hidden, 3 * batch + hidden)
    eps = np.float32(0.03)
    ref = oracle.fd_reweight(lp, lm, lam, float(eps), batch)
    with Ctx(16, batch, (4, 2)) as ctx:
        out = torch.full((3 * hidden + 1,), float("nan"), dtype=torch.float32, device=DEV)
        args = (ctx.h, batch, dev(lp), dev(lm), None, hidden, dev(lam), dev(np.array([eps])), batch, out)
        B.sama_fd_metagrad_reweight(*args)
        torch.cuda.synchronize()
        a = out.cpu().numpy()
        close(a, ref, (batch, hidden))
        B.sama_fd_metagrad_reweight(*args)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), a)      # fixed reduction order
        # a zero step size gives a zero meta gradient, not a division by zero
        B.sama_fd_metagrad_reweight(ctx.h, batch, dev(lp), dev(lm), None, hidden, dev(lam), dev(np.float32([0.0])), batch, out)
        torch.cuda.synchronize()
        assert np.all(out.cpu().numpy() == 0.0)
        # the difference given separately (here exactly lp - lm) and loss_plus left out: same result to rounding
        diff = (lp.astype(np.float64) - lm.astype(np.float64)).astype(np.float32)
        B.sama_fd_metagrad_reweight(ctx.h, batch, None, dev(lm), dev(diff), hidden, dev(lam), dev(np.array([eps])), batch, out)
        torch.cuda.synchronize()
        close(out.cpu().numpy(), oracle.fd_reweight(lm.astype(np.float64) + diff.astype(np.float64), lm, lam, float(eps), batch),
              (batch, hidden, "diff"))
        assert B.sama_device_status(ctx.h) == 0


@pytest.mark.parametrize("name,alpha", [("tiny", 1e-2), ("tiny", 1.0), ("mlp3072", 1e-2)])
def test_step_reweight_parity(name, alpha):
    cfg = W.CONFIGS[name]
    w = W.mlp_workload(cfg, 0)
    n, Bsz, hidden = cfg.n_params, cfg.batch, 100
    lam = lambda_r(hidden, 5)
    f = lambda x: float(np.float32(x))
    ref = oracle.step(cfg.dims, w["theta"], w["m"], w["s"], w["g_base"], w["g_meta"],
                      oracle.Adam(f(1e-3), f(0.9), f(0.999), f(1e-8), 100), f(alpha), w["X"], w["y"], w["lam"])
    ref_r = oracle.fd_reweight(ref["loss_plus"], ref["loss_minus"], lam, ref["eps_fd"], Bsz)
    with Ctx(n, Bsz, cfg.dims) as ctx:
        t = {k: dev(w[k]) for k in ["theta", "m", "s", "g_base", "g_meta", "X", "y"]}
        fl = lambda k: torch.empty(k, dtype=torch.float32, device=DEV)
        p, tp, tm, lp, lm, out = fl(n), fl(n), fl(n), fl(Bsz), fl(Bsz), fl(3 * hidden + 1)
        B.sama_step_reweight(ctx.h, ctx.mlp, n, t["theta"], t["m"], t["s"], t["g_base"], t["g_meta"], B.Adam(), alpha,
                             t["X"], t["y"], Bsz, hidden, dev(lam), p, tp, tm, out, lp, lm)
        torch.cuda.synchronize()
        assert B.sama_device_status(ctx.h) == 0
        a = out.cpu().numpy().astype(np.float64)
        # per-sample terms from the checker, one row at a time
        terms = np.stack([oracle.fd_reweight(ref["loss_plus"][i:i + 1], ref["loss_minus"][i:i + 1], lam, ref["eps_fd"], Bsz)
                          for i in range(Bsz)])
        np.testing.assert_allclose(terms.sum(axis=0), ref_r, rtol=1e-9, atol=1e-18)
        scale = np.abs(terms).sum(axis=0)
        assert np.all(np.abs(a - ref_r) <= 2e-3 * scale + 1e-12), (name, alpha, float((np.abs(a - ref_r) / (scale + 1e-300)).max()))
        nrm = float(np.linalg.norm(a - ref_r) / np.linalg.norm(scale))
        assert nrm <= 2e-3
        cancel = float(np.linalg.norm(scale) / np.linalg.norm(ref_r))
        np.testing.assert_allclose(lp.cpu().numpy(), ref["loss_plus"], rtol=1e-4, atol=1e-4)
        # without the optional loss outputs the result is the same
        out2 = fl(3 * hidden + 1)
        B.sama_step_reweight(ctx.h, ctx.mlp, n, t["theta"], t["m"], t["s"], t["g_base"], t["g_meta"], B.Adam(), alpha,
                             t["X"], t["y"], Bsz, hidden, dev(lam), p, tp, tm, out2)
        torch.cuda.synchronize()
        assert torch.equal(out2, out)
        # the modular route: per-sample step, then the shared-network difference from its losses and the
        # context's loss difference
        got = run_step(ctx, cfg, w, B.Adam(), alpha)
        assert np.array_equal(got["loss_plus"], lp.cpu().numpy())
        out3 = fl(3 * hidden + 1)
        B.sama_fd_metagrad_reweight(ctx.h, Bsz, None, dev(got["loss_minus"]), B.sama_ctx_loss_diff(ctx.h), hidden, dev(lam),
                                    None, Bsz, out3)
        torch.cuda.synchronize()
        assert torch.equal(out3, out)
    print("\n[reweight] %s alpha=%g: error %.2e of ||sum |terms||| (= %.1f x ||sum terms||), %.2e of the result's norm" %
          (name, alpha, nrm, cancel, nrm * cancel))


def test_reweight_argument_errors():
    with Ctx(16, 8, (4, 2)) as ctx:
        x = torch.ones(8, dtype=torch.float32, device=DEV)
        lam = torch.zeros(3 * 4 + 1, dtype=torch.float32, device=DEV)
        out = torch.zeros(3 * 4 + 1, dtype=torch.float32, device=DEV)
        eps = torch.ones(1, dtype=torch.float32, device=DEV)

        def status(*a):
            with pytest.raises(B.SamaError) as e:
                B.sama_fd_metagrad_reweight(*a)
            return e.value.status

        assert status(ctx.h, 9, x, x, None, 4, lam, eps, 9, out) == B.SAMA_ERR_SIZE
        assert status(ctx.h, 8, x, x, None, 0, lam, eps, 8, out) == B.SAMA_ERR_SIZE
        assert status(ctx.h, 8, x, x, None, 257, lam, eps, 8, out) == B.SAMA_ERR_SIZE
        assert status(ctx.h, 8, x, None, None, 4, lam, eps, 8, out) == B.SAMA_ERR_NULL
        assert status(ctx.h, 8, None, x, None, 4, lam, eps, 8, out) == B.SAMA_ERR_NULL
        assert status(ctx.h, 8, x, x, None, 4, lam, eps, 8, lam) == B.SAMA_ERR_OVERLAP
    with Ctx(16) as ctx:     # no model, no workspace
        assert status(ctx.h, 8, x, x, None, 4, lam, eps, 8, out) == B.SAMA_ERR_SIZE
