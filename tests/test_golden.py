"""Stored results of the CPU checker on small seeded workloads (tests/golden/step_small.json and
biasreg_small.json, written by tests/golden/make_golden.py from ``oracle/`` alone): the checker must still
reproduce them, and the CUDA path must match them within the parity tolerances."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = json.load(open(os.path.join(HERE, "golden", "step_small.json")))
GOLDEN_BIASREG = json.load(open(os.path.join(HERE, "golden", "biasreg_small.json")))


def _maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


@pytest.mark.parametrize("g", GOLDEN, ids=[g["case"]["name"] for g in GOLDEN])
def test_checker_reproduces_stored_values(g):
    r = _maker().run_case(g["case"])
    for k in ("eps_fd", "sumsq"):
        assert r[k] == pytest.approx(g[k], rel=1e-12)
    for k in ("p_head", "theta_plus_head", "loss_plus", "loss_minus", "metagrad", "metagrad_reweight"):
        np.testing.assert_allclose(r[k], g[k], rtol=1e-10, atol=1e-300)


def test_checker_reproduces_stored_biased_regression_values():
    g = GOLDEN_BIASREG
    r = _maker().run_biasreg(g["case"])
    assert r["eps_fd"] == pytest.approx(g["eps_fd"], rel=1e-12)
    for k in ("w_star", "g_meta", "metagrad", "true_meta_grad", "lambda_star"):
        np.testing.assert_allclose(r[k], g[k], rtol=1e-9, atol=1e-300)


@pytest.mark.gpu
@pytest.mark.parametrize("gemm_mode", [1, 2])
@pytest.mark.parametrize("g", GOLDEN, ids=[g["case"]["name"] for g in GOLDEN])
def test_cuda_path_matches_stored_values(g, gemm_mode):
    from gpu_util import B, Ctx, assert_fd_close, run_step
    from paper_2310_05674_b200 import workloads as W
    c = g["case"]
    cfg, w = W.custom_mlp(c["dims"], c["batch"], seed=c["seed"])
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, gemm_mode) as ctx:
        got = run_step(ctx, cfg, w, B.Adam(step=c["step"]), c["alpha"])
    assert got["eps_fd"] == pytest.approx(g["eps_fd"], rel=1e-6)
    np.testing.assert_allclose(got["p"][:8], g["p_head"], rtol=1e-5)
    np.testing.assert_allclose(got["theta_plus"][:8], g["theta_plus_head"], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(got["loss_plus"], g["loss_plus"], rtol=1e-4, atol=1e-5)
    assert_fd_close(got["metagrad"], np.array(g["metagrad"]), norm_tol=2e-2 if (gemm_mode == 1 and c["alpha"] < 1) else 2e-3)
    # the shared reweighting network on the same step: held to 2e-3 of the sum of its terms' magnitudes
    import torch
    from gpu_util import DEV, dev
    lam_r = _maker().reweight_lambda(c)
    lp, lm = np.array(g["loss_plus"]), np.array(g["loss_minus"])
    import oracle
    terms = np.stack([oracle.fd_reweight(lp[i:i + 1], lm[i:i + 1], lam_r, g["eps_fd"], c["batch"]) for i in range(c["batch"])])
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, gemm_mode) as ctx:
        t = {k: dev(w[k]) for k in ["theta", "m", "s", "g_base", "g_meta", "X", "y"]}
        fl = lambda k: torch.empty(k, dtype=torch.float32, device=DEV)
        out = fl(lam_r.size)
        B.sama_step_reweight(ctx.h, ctx.mlp, cfg.n_params, t["theta"], t["m"], t["s"], t["g_base"], t["g_meta"],
                             B.Adam(step=c["step"]), c["alpha"], t["X"], t["y"], cfg.batch, 3, dev(lam_r), fl(cfg.n_params),
                             fl(cfg.n_params), fl(cfg.n_params), out)
        torch.cuda.synchronize()
    tol = (2e-2 if (gemm_mode == 1 and c["alpha"] < 1) else 2e-3) * np.abs(terms).sum(axis=0) + 1e-12
    assert np.all(np.abs(out.cpu().numpy() - np.array(g["metagrad_reweight"])) <= tol)


@pytest.mark.gpu
def test_cuda_biased_regression_matches_stored_values():
    import torch
    from gpu_util import B, Ctx, DEV, dev
    from paper_2310_05674_b200 import workloads as W
    g = GOLDEN_BIASREG
    c = g["case"]
    w = W.biased_regression(W.BiasRegConfig(c["name"], c["d"], c["n"], c["n_val"], beta=c["beta"]), c["seed"])
    d = c["d"]
    with Ctx(d) as ctx:
        fl = lambda: torch.empty(d, dtype=torch.float32, device=DEV)
        gm, p, wp, wm, mg = fl(), fl(), fl(), fl(), fl()
        B.sama_biasreg_step(ctx.h, d, c["n_val"], dev(w["Xv"]), dev(w["yv"]), dev(np.float32(g["w_star"])), dev(w["lam0"]),
                            c["beta"], None, None, None, B.Adam(identity=True), c["alpha"], gm, p, wp, wm, mg)
        torch.cuda.synchronize()
    np.testing.assert_allclose(gm.cpu().numpy(), g["g_meta"], rtol=1e-5, atol=1e-5 * np.abs(g["g_meta"]).max())
    ref = np.array(g["metagrad"])
    assert np.linalg.norm(mg.cpu().numpy() - ref) <= 2e-3 * np.linalg.norm(ref)
