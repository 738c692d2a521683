"""Pins the biased-regression part of the CPU checker (Appendix E) to things other than itself:
a different library route to the base solution, numerical differentiation of the bilevel objective,
optimality of lambda*, the exactness of the central difference on a quadratic, the orthogonal-design
case in which the identity approximation of Eq. 3 is exact, and Kantorovich's bound on the cosine."""
import importlib.util
import os

import numpy as np
import pytest

import oracle
from oracle import biased_regression as R
from paper_2310_05674_b200 import workloads as W


def problem(d=12, n=30, nv=20, seed=0):
    rng = np.random.default_rng(seed)
    X, Xv = rng.normal(size=(n, d)), rng.normal(size=(nv, d))
    wt = rng.normal(size=d)
    y, yv = X @ wt + 0.1 * rng.normal(size=n), Xv @ wt + 0.1 * rng.normal(size=nv)
    return X, y, Xv, yv, rng.normal(size=d)


def run_pins(mod):
    beta = 0.1
    X, y, Xv, yv, lam = problem()
    d = X.shape[1]
    # base solution: the same minimiser through a stacked least-squares problem (another library route)
    w = mod.base_solution(X, y, beta, lam)
    stacked_A = np.vstack([X, np.sqrt(beta) * np.eye(d)])
    stacked_b = np.concatenate([y, np.sqrt(beta) * lam])
    w_ls = np.linalg.lstsq(stacked_A, stacked_b, rcond=None)[0]
    np.testing.assert_allclose(w, w_ls, rtol=1e-9, atol=1e-12)
    # ... and it is a minimiser of the printed base objective
    f0 = mod.base_loss(X, y, beta, w, lam)
    rng = np.random.default_rng(5)
    for _ in range(20):
        assert mod.base_loss(X, y, beta, w + 1e-3 * rng.normal(size=d), lam) > f0
    # item 1
    np.testing.assert_allclose(mod.base_jacobian(X, beta), X.T @ X + beta * np.eye(d), rtol=0, atol=1e-12)
    # item 2: central differences of lambda -> L_meta(w*(lambda)) (a quadratic, so they are exact up to rounding)
    g = mod.true_meta_grad(X, y, Xv, yv, beta, lam)
    F = lambda l: mod.meta_loss(Xv, yv, mod.base_solution(X, y, beta, l))
    for k in range(d):
        e = np.zeros(d)
        e[k] = 1e-3
        assert (F(lam + e) - F(lam - e)) / 2e-3 == pytest.approx(g[k], rel=1e-7, abs=1e-9)
    np.testing.assert_allclose(mod.printed_meta_grad(X, y, Xv, yv, beta, lam), 0.5 * g, rtol=1e-12)
    # the direct gradient by differences of L_meta in w
    gw = mod.direct_grad(Xv, yv, w)
    for k in range(d):
        e = np.zeros(d)
        e[k] = 1e-3
        assert (mod.meta_loss(Xv, yv, w + e) - mod.meta_loss(Xv, yv, w - e)) / 2e-3 == pytest.approx(gw[k], rel=1e-7, abs=1e-9)
    # dL_base/dlambda by differences
    gl = mod.base_grad_lambda(w, lam, beta)
    for k in range(d):
        e = np.zeros(d)
        e[k] = 1e-3
        assert (mod.base_loss(X, y, beta, w, lam + e) - mod.base_loss(X, y, beta, w, lam - e)) / 2e-3 == \
            pytest.approx(gl[k], rel=1e-7, abs=1e-9)
    # item 3 (needs n' >= d): stationarity, optimality, and the least-squares route
    ls = mod.lambda_star(X, y, Xv, yv, beta)
    assert np.abs(mod.true_meta_grad(X, y, Xv, yv, beta, ls)).max() < 1e-9
    for _ in range(20):
        assert F(ls + 1e-2 * rng.normal(size=d)) > F(ls)
    H = X.T @ X + beta * np.eye(d)
    A = beta * Xv @ np.linalg.inv(H)
    b = yv - Xv @ np.linalg.inv(H) @ X.T @ y
    np.testing.assert_allclose(ls, np.linalg.lstsq(A, b, rcond=None)[0], rtol=1e-6, atol=1e-8)
    # SAMA on this problem: the central difference of a quadratic is exact, so metagrad = 2 beta p, and with an
    # SGD base optimiser p = g_meta, i.e. the true gradient with H^-1 replaced by (a multiple of) the identity
    w32 = w.astype(np.float32)
    for alpha in (1.0, 1e-2):
        out = mod.sama_meta_grad(Xv, yv, w32, lam, beta, alpha)
        assert not out["degenerate"]
        np.testing.assert_allclose(out["p"], mod.direct_grad(Xv, yv, w32).astype(np.float32), rtol=0, atol=0)
        np.testing.assert_allclose(out["metagrad"], 2 * beta * out["p"], rtol=1e-9 / alpha, atol=1e-12)
        assert np.linalg.norm(out["w_plus"] - w32) == pytest.approx(alpha, rel=1e-12)
        r = Xv.T @ (Xv @ w32.astype(np.float64) - yv)
        assert mod.cosine(out["metagrad"], r) == pytest.approx(1.0, abs=1e-6)   # only fp32 storage of g_meta between them
    # sign: a step against SAMA's meta gradient lowers the meta loss
    out = mod.sama_meta_grad(Xv, yv, w32, lam, beta, 1.0)
    assert F(lam - 1e-3 * out["metagrad"]) < F(lam)
    # Kantorovich: cos(r, H^-1 r) >= 2 sqrt(l_min l_max) / (l_min + l_max)
    ev = np.linalg.eigvalsh(H)
    bound = 2 * np.sqrt(ev[0] * ev[-1]) / (ev[0] + ev[-1])
    assert mod.cosine(out["metagrad"], mod.true_meta_grad(X, y, Xv, yv, beta, lam)) >= bound - 1e-6
    # Adam adaptation reuses S1: with zero moments it is the checker's adapt on the direct gradient
    adam = oracle.Adam(step=3)
    z = np.zeros(d, np.float32)
    gb = (0.01 * rng.normal(size=d)).astype(np.float32)
    out_a = mod.sama_meta_grad(Xv, yv, w32, lam, beta, 1.0, adam, z, z, gb)
    np.testing.assert_array_equal(out_a["p"], oracle.adapt(z, z, gb, mod.direct_grad(Xv, yv, w32).astype(np.float32), adam))
    np.testing.assert_allclose(out_a["metagrad"], 2 * beta * out_a["p"], rtol=1e-9, atol=1e-12)


def test_biased_regression_checker_passes_its_pins():
    run_pins(R)


def test_identity_approximation_is_exact_for_an_orthogonal_design():
    """X^T X = c I makes the base Jacobian a multiple of the identity (Eq. 3's assumption holds exactly), so
    SAMA's direction equals the true meta gradient's."""
    rng = np.random.default_rng(3)
    d, n = 10, 25
    Q, _ = np.linalg.qr(rng.normal(size=(n, d)))
    X = 3.0 * Q
    _, y, Xv, yv, lam = problem(d, n, 20, seed=4)
    w = R.base_solution(X, y, 0.1, lam)
    out = R.sama_meta_grad(Xv, yv, w, lam, 0.1, 1.0)
    assert R.cosine(out["metagrad"], R.true_meta_grad(X, y, Xv, yv, 0.1, lam)) == pytest.approx(1.0, abs=1e-6)


def test_meta_updates_approach_the_optimum_on_the_bench_workload():
    """The study itself on the small workload: 100 meta updates with SAMA's gradient (base level solved in closed
    form, plain gradient descent on lambda with step 1 / lambda_max of the update's linear map).  The figure in
    Appendix E prints no numbers, so this pins behaviour only: a high, stable cosine and a shrinking distance."""
    cfg = W.BIASREG["biasreg256"]
    w = W.biased_regression(cfg, 0)
    X, y, Xv, yv = (w[k].astype(np.float64) for k in ("X", "y", "Xv", "yv"))
    H = R.base_jacobian(X, cfg.beta)
    M = 4 * cfg.beta ** 2 * (Xv.T @ Xv) @ np.linalg.inv(H)
    eta = 1.0 / np.linalg.eigvals(M).real.max()
    lam = w["lam0"].astype(np.float64)
    ls = R.lambda_star(X, y, Xv, yv, cfg.beta)
    dist, cosv = [], []
    for _ in range(cfg.meta_updates):
        wst = R.base_solution(X, y, cfg.beta, lam)
        out = R.sama_meta_grad(Xv, yv, wst, lam, cfg.beta, 1.0)
        cosv.append(R.cosine(out["metagrad"], R.true_meta_grad(X, y, Xv, yv, cfg.beta, lam)))
        dist.append(float(np.linalg.norm(lam - ls)))
        lam = lam - eta * out["metagrad"]
    assert min(cosv) > 0.7
    assert all(b < a for a, b in zip(dist, dist[1:]))
    assert dist[-1] < 0.25 * dist[0]


MUTATIONS = {
    "fd_sign": ("mg = -(base_grad_lambda(w_plus", "mg = (base_grad_lambda(w_plus"),
    "fd_one_sided_scale": ("/ (2.0 * eps_fd)", "/ (eps_fd)"),
    "beta_missing_in_meta_grad": ("return 2.0 * beta * np.linalg.solve(base_jacobian(X, beta), Xv.T @ (Xv @ w) - Xv.T @ yv)",
                                  "return 2.0 * np.linalg.solve(base_jacobian(X, beta), Xv.T @ (Xv @ w) - Xv.T @ yv)"),
    "base_solution_without_beta_lambda": ("X.T @ y + beta * lam)", "X.T @ y + lam)"),
    "jacobian_without_ridge": ("return X.T @ X + beta * np.eye(X.shape[1])", "return X.T @ X + 0 * beta * np.eye(X.shape[1])"),
    "direct_grad_not_transposed": ("return 2.0 * (Xv.T @ (Xv @ w - yv))", "return 2.0 * ((Xv @ w - yv) @ Xv[:, ::-1])"),
    "grad_lambda_sign": ("return -2.0 * beta * (_f64(w) - _f64(lam))", "return 2.0 * beta * (_f64(w) - _f64(lam))"),
    "lambda_star_b_without_base_fit": ("b = yv - Xv @ np.linalg.solve(H, X.T @ y)", "b = yv"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_in_the_regression_checker_is_caught(name, tmp_path):
    old, new = MUTATIONS[name]
    src = open(os.path.join(os.path.dirname(oracle.__file__), "biased_regression.py")).read()
    assert src.count(old) == 1, "mutation site not found exactly once"
    path = tmp_path / "mutant_biasreg.py"
    path.write_text(src.replace(old, new))
    spec = importlib.util.spec_from_file_location("mutant_biasreg", str(path))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with pytest.raises(AssertionError):
        run_pins(mod)
