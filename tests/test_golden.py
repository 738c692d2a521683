"""Stored results of the CPU checker on two small seeded workloads (tests/golden/step_small.json,
written by tests/golden/make_golden.py from ``oracle/`` alone): the checker must still reproduce
them, and the CUDA path must match them within the parity tolerances."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = json.load(open(os.path.join(HERE, "golden", "step_small.json")))


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
    for k in ("p_head", "theta_plus_head", "loss_plus", "loss_minus", "metagrad"):
        np.testing.assert_allclose(r[k], g[k], rtol=1e-10, atol=1e-300)


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
    assert_fd_close(got["metagrad"], np.array(g["metagrad"]), norm_tol=2e-3 if c["alpha"] >= 1 else 2e-2)
