"""Writes tests/golden/step_small.json and tests/golden/biasreg_small.json: the CPU checker's results on small
seeded workloads (the step with per-sample weights and with the shared reweighting network of Sec. 4.1; SAMA on
the biased-regression problem of Appendix E).  Calls only ``oracle/`` and the seeded input generators (never the CUDA path).
The paper prints no worked numeric example, so these values pin nothing by themselves:
they detect drift of the checker (its arithmetic is pinned by tests/test_oracle_pins.py).

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from oracle import biased_regression as R  # noqa: E402
from paper_2310_05674_b200 import workloads as W  # noqa: E402

CASES = [
    {"name": "mlp_6_5_3", "dims": [6, 5, 3], "batch": 4, "seed": 41, "alpha": 1.0, "step": 100},
    {"name": "mlp_9_7_6_4", "dims": [9, 7, 6, 4], "batch": 6, "seed": 42, "alpha": 1e-2, "step": 1},
]


def f32(x):
    return float(np.float32(x))


def run_case(c):
    cfg, w = W.custom_mlp(c["dims"], c["batch"], seed=c["seed"])
    adam = oracle.Adam(f32(1e-3), f32(0.9), f32(0.999), f32(1e-8), c["step"])
    r = oracle.step(c["dims"], w["theta"], w["m"], w["s"], w["g_base"], w["g_meta"], adam, f32(c["alpha"]),
                    w["X"], w["y"], w["lam"])
    lam_r = reweight_lambda(c)
    return {"case": c, "eps_fd": r["eps_fd"], "sumsq": oracle.sumsq(r["p"]), "p_head": r["p"][:8].tolist(),
            "theta_plus_head": r["theta_plus"][:8].tolist(), "loss_plus": r["loss_plus"].tolist(),
            "loss_minus": r["loss_minus"].tolist(), "metagrad": r["metagrad"].tolist(),
            "metagrad_reweight": oracle.fd_reweight(r["loss_plus"], r["loss_minus"], lam_r, r["eps_fd"], c["batch"]).tolist()}


def reweight_lambda(c, hidden=3):
    """lambda_r = (v1, c1, v2, c2) of a width-3 reweighting network, drawn by the seeded generator."""
    lam = (0.5 * W.normal(c["seed"], 90, 3 * hidden + 1)).astype(np.float32)
    lam[hidden:2 * hidden] += np.float32(0.3)
    return lam


BIASREG_CASE = {"name": "biasreg_6", "d": 6, "n": 14, "n_val": 9, "seed": 43, "beta": 0.1, "alpha": 1.0}


def run_biasreg(c):
    cfg = W.BiasRegConfig(c["name"], c["d"], c["n"], c["n_val"], beta=c["beta"])
    w = W.biased_regression(cfg, c["seed"])
    w_cur = R.base_solution(w["X"], w["y"], c["beta"], w["lam0"]).astype(np.float32)
    r = R.sama_meta_grad(w["Xv"], w["yv"], w_cur, w["lam0"], f32(c["beta"]), f32(c["alpha"]))
    return {"case": c, "w_star": w_cur.astype(np.float64).tolist(), "g_meta": r["g_meta"].tolist(), "eps_fd": r["eps_fd"],
            "metagrad": r["metagrad"].tolist(),
            "true_meta_grad": R.true_meta_grad(w["X"], w["y"], w["Xv"], w["yv"], c["beta"], w["lam0"]).tolist(),
            "lambda_star": R.lambda_star(w["X"], w["y"], w["Xv"], w["yv"], c["beta"]).tolist()}


if __name__ == "__main__":
    out = [run_case(c) for c in CASES]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "step_small.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "biasreg_small.json")
    with open(path, "w") as f:
        json.dump(run_biasreg(BIASREG_CASE), f, indent=1)
    print("wrote", path)
