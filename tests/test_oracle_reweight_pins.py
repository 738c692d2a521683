"""Pins the shared-reweighting-network part of the CPU checker (Sec. 4.1, Eq. 5) to things other than itself:
numerical differentiation of the base objective in extended precision, special cases with a known answer,
and the mixed second derivative on tiny MLPs by nested differences."""
import numpy as np
import pytest

import oracle

LD = np.longdouble


def weight_ld(l, lam):
    """w(l; lambda_r) typed out in extended precision: the definition, not the checker's derivative code."""
    H = (len(lam) - 1) // 3
    v1, c1, v2, c2 = lam[:H], lam[H:2 * H], lam[2 * H:3 * H], lam[3 * H]
    z = LD(c2)
    for j in range(H):
        a = LD(v1[j]) * LD(l) + LD(c1[j])
        if a > 0:
            z += LD(v2[j]) * a
    return 1 / (1 + np.exp(-z))


def base_objective_ld(losses, lam, B_norm):
    return sum(weight_ld(l, lam) * LD(l) for l in losses) / LD(B_norm)


def rand_lambda(rng, H, scale=0.7):
    return (scale * rng.normal(size=3 * H + 1)).astype(np.float32)


def test_reweight_gradient_matches_brute_force_difference():
    rng = np.random.default_rng(0)
    for H, cnt in [(1, 1), (3, 5), (8, 17), (16, 4)]:
        for trial in range(6):
            lam = rand_lambda(rng, H)
            losses = np.abs(rng.normal(size=cnt)) * 2.0 + 0.05
            # keep hidden pre-activations off the ReLU kink, where the derivative is not defined
            a = np.outer(losses, lam[:H]) + lam[H:2 * H]
            if np.abs(a).min() < 1e-3:
                continue
            g, wts = oracle.reweight_grad(losses, lam, B_norm=cnt + 2)
            for i, l in enumerate(losses):
                assert wts[i] == pytest.approx(float(weight_ld(l, lam)), rel=1e-12)
            for k in range(3 * H + 1):
                h = LD(1e-5)
                lp, lm = lam.astype(LD), lam.astype(LD)
                lp[k] += h
                lm[k] -= h
                d = (base_objective_ld(losses, lp, cnt + 2) - base_objective_ld(losses, lm, cnt + 2)) / (2 * h)
                assert g[k] == pytest.approx(float(d), rel=1e-7, abs=1e-11), (H, cnt, k)


def test_reweight_special_cases():
    # no active hidden unit: only the output bias has a gradient, mean of l sigmoid'(c2)
    lam = np.float32([0.5, -0.3, -1.0, -2.0, 0.7, 0.9, 0.25])      # H = 2, c1 < 0 and v1 l + c1 < 0 for small l
    losses = np.array([0.1, 0.2, 0.3])
    g, wts = oracle.reweight_grad(losses, lam)
    s = 1 / (1 + np.exp(-0.25))
    np.testing.assert_allclose(wts, s, rtol=1e-12)
    assert np.all(g[:6] == 0.0)
    assert g[6] == pytest.approx(losses.mean() * s * (1 - s), rel=1e-12)
    # a saturated output: the gradient vanishes
    lam = np.float32([1.0, 0.0, 1.0, 60.0])                          # H = 1, z >= 60
    g, wts = oracle.reweight_grad(np.array([1.0, 2.0]), lam)
    assert np.all(np.abs(g) < 1e-20) and np.all(wts >= 1 - 1e-15)
    # one hidden unit, one sample, by hand: a = v1 l + c1, z = v2 a + c2, f = l w (1 - w)
    v1, c1, v2, c2, l = 0.5, 0.25, -0.75, 0.125, 2.0
    g, wts = oracle.reweight_grad(np.array([l]), np.float32([v1, c1, v2, c2]))
    a = v1 * l + c1
    w = 1 / (1 + np.exp(-(v2 * a + c2)))
    f = l * w * (1 - w)
    np.testing.assert_allclose(g, [f * v2 * l, f * v2, f * a, f], rtol=1e-12)
    # the batch normaliser is the whole batch, not the number of rows evaluated
    g2, _ = oracle.reweight_grad(np.array([l]), np.float32([v1, c1, v2, c2]), B_norm=4)
    np.testing.assert_allclose(g2, g / 4, rtol=1e-12)
    # rows add up
    rng = np.random.default_rng(1)
    lam = rand_lambda(rng, 5)
    L = np.abs(rng.normal(size=9)) + 0.1
    ga, _ = oracle.reweight_grad(L[:4], lam, B_norm=9)
    gb, _ = oracle.reweight_grad(L[4:], lam, B_norm=9)
    np.testing.assert_allclose(oracle.reweight_grad(L, lam)[0], ga + gb, rtol=1e-12, atol=1e-300)


def test_fd_reweight_structure():
    rng = np.random.default_rng(2)
    lam = rand_lambda(rng, 6)
    lp, lm = np.abs(rng.normal(size=11)) + 0.1, np.abs(rng.normal(size=11)) + 0.1
    out = oracle.fd_reweight(lp, lm, lam, 0.05)
    gp, gm = oracle.reweight_grad(lp, lam)[0], oracle.reweight_grad(lm, lam)[0]
    np.testing.assert_allclose(out, -(gp - gm) / 0.1, rtol=1e-12, atol=1e-300)        # Eq. 5, minus sign included
    np.testing.assert_array_equal(oracle.fd_reweight(lm, lp, lam, 0.05), -out)          # antisymmetry
    assert np.all(oracle.fd_reweight(lp, lp, lam, 0.05) == 0.0)
    assert np.all(oracle.fd_reweight(lp, lm, lam, 0.0) == 0.0)                          # degenerate step


@pytest.mark.parametrize("dims,B", [((3, 4, 2), 5), ((4, 3), 6)])
def test_fd_reweight_against_nested_differences_on_a_tiny_mlp(dims, B):
    """Eq. 4/5: the meta gradient SAMA returns is -d/d(eps) [dL_base(theta + eps p)/dlambda_r] at 0, i.e. minus the
    mixed second derivative of L_base contracted with p.  Brute force: nested central differences of
    L_base(theta, lambda_r) = (1/B) sum_i w(l_i(theta)) l_i(theta), losses from the checker's forward (pinned
    elsewhere), weights typed out above."""
    rng = np.random.default_rng(sum(dims))
    n = sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))
    theta = (0.5 * rng.normal(size=n)).astype(np.float32)
    X = rng.normal(size=(B, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=B).astype(np.int32)
    lam = rand_lambda(rng, 3, 0.5)
    p = rng.normal(size=n)
    p /= np.linalg.norm(p)

    def L_base(th, lam_ld):
        return base_objective_ld(oracle.losses(dims, th, X, y), lam_ld, B)

    eps = 1e-3
    tp, tm = theta.astype(np.float64) + eps * p, theta.astype(np.float64) - eps * p
    got = oracle.fd_reweight(oracle.losses(dims, tp, X, y), oracle.losses(dims, tm, X, y), lam, eps)
    for k in range(lam.size):
        h = LD(1e-4)
        lp_, lm_ = lam.astype(LD), lam.astype(LD)
        lp_[k] += h
        lm_[k] -= h
        d_plus = (L_base(tp, lp_) - L_base(tp, lm_)) / (2 * h)
        d_minus = (L_base(tm, lp_) - L_base(tm, lm_)) / (2 * h)
        ref = -float((d_plus - d_minus) / (2 * LD(eps)))
        assert got[k] == pytest.approx(ref, rel=2e-4, abs=1e-7), k
