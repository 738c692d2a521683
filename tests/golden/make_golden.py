"""Writes tests/golden/step_small.json: the CPU checker's results on two small seeded
workloads.  Calls only ``oracle/`` and the seeded input generators (never the CUDA path).
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
    return {"case": c, "eps_fd": r["eps_fd"], "sumsq": oracle.sumsq(r["p"]), "p_head": r["p"][:8].tolist(),
            "theta_plus_head": r["theta_plus"][:8].tolist(), "loss_plus": r["loss_plus"].tolist(),
            "loss_minus": r["loss_minus"].tolist(), "metagrad": r["metagrad"].tolist()}


if __name__ == "__main__":
    out = [run_case(c) for c in CASES]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "step_small.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)
