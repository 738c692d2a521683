"""Pins the CPU checker to things other than itself.

Each test fixes one part of ``oracle/`` against what the paper or plain
calculus determines: numerical differentiation of the Adam update (Appendix C),
the paper's printed numerator in the special case where it is exact, textbook
limits, the closed-form mixed second derivative of a linear-softmax model
(Eq. 4/5), nested numerical differentiation on tiny MLPs, a library matmul
forward pass, and the invariants of Sec. 3.2.  A dropped term, a wrong sign, a
swapped beta or a transposed weight in the checker fails at least one of them.
"""
import numpy as np
import pytest

import oracle
from paper_2310_05674_b200 import workloads as W

LD = np.longdouble


# ----------------------------------------------------------------------------
# S1: Adam adaptation matrix (Appendix C)
# ----------------------------------------------------------------------------

def adam_update_ld(g, m, s, lr, b1, b2, eps, step, bias_correction=True):
    """The Adam update u(g) itself (first line of Appendix C, bias-corrected
    as in the Adam paper), in extended precision.  Independent of the checker,
    which only ever evaluates the derivative."""
    g, m, s = LD(g), LD(m), LD(s)
    b1, b2, lr, eps = LD(b1), LD(b2), LD(lr), LD(eps)
    m_new = b1 * m + (1 - b1) * g
    s_new = b2 * s + (1 - b2) * g * g
    c1 = 1 - b1 ** LD(step) if bias_correction else LD(1)
    c2 = 1 - b2 ** LD(step) if bias_correction else LD(1)
    return lr * (m_new / c1) / (np.sqrt(s_new / c2) + eps)


def jac(m, s, g, adam):
    one = np.ones(1, dtype=np.float32)
    return oracle.adapt(np.float32([m]), np.float32([s]), None if g is None else np.float32([g]), one, adam)[0]


@pytest.mark.parametrize("bias_correction", [True, False])
def test_adam_jacobian_matches_brute_force_difference(bias_correction):
    rng = np.random.default_rng(1)
    worst = 0.0
    for trial in range(4000):
        step = int(rng.choice([1, 2, 100, 1000]))
        b1 = float(rng.choice([0.9, 0.8, 0.0, 0.95]))
        b2 = float(rng.choice([0.999, 0.99, 0.9]))
        lr = float(10 ** rng.uniform(-4, -1))
        eps = float(10 ** rng.uniform(-10, -4))
        m = np.float32(rng.normal() * 1e-3)
        s = np.float32(float(m) ** 2 + abs(rng.normal()) * 10 ** rng.uniform(-8, -4))
        g = np.float32(rng.normal() * 10 ** rng.uniform(-4, -2))
        adam = oracle.Adam(lr, b1, b2, eps, step, bias_correction)
        J = jac(m, s, g, adam)
        # 4th-order central difference in extended precision
        h = LD(1e-4) * max(abs(LD(g)), np.sqrt(LD(s)), LD(1e-12))
        f = lambda x: adam_update_ld(x, m, s, lr, b1, b2, eps, step, bias_correction)
        d = (-f(LD(g) + 2 * h) + 8 * f(LD(g) + h) - 8 * f(LD(g) - h) + f(LD(g) - 2 * h)) / (12 * h)
        scale = max(abs(float(d)), 1e-3 * lr / (np.sqrt(float(s)) + eps))
        worst = max(worst, abs(J - float(d)) / scale)
    assert worst < 1e-6, worst


def test_adam_jacobian_null_gbase_uses_m():
    adam = oracle.Adam()
    for m, s in [(1e-3, 2e-6), (-5e-4, 1e-6)]:
        assert jac(m, s, None, adam) == jac(m, s, m, adam)


def test_printed_numerator_in_equal_beta_case():
    """With beta1 == beta2 and no bias correction the exact derivative has the
    numerator the paper prints in Appendix C:
    (1-b) b s - (1-b) b m g + (1-b) eps r over r (r + eps)^2."""
    rng = np.random.default_rng(2)
    for _ in range(200):
        b = float(rng.uniform(0.5, 0.99))
        lr, eps = 3e-3, float(10 ** rng.uniform(-8, -5))
        m, g = np.float32(rng.normal() * 1e-3), np.float32(rng.normal() * 1e-3)
        s = np.float32(float(m) ** 2 + abs(rng.normal()) * 1e-6)
        md, gd, sd = float(m), float(g), float(s)
        r = np.sqrt(b * sd + (1 - b) * gd * gd)
        printed = lr * ((1 - b) * b * sd - (1 - b) * b * md * gd + (1 - b) * eps * r) / (r * (r + eps) ** 2)
        approx = lr * ((1 - b) * b * sd - (1 - b) * b * md * gd) / (r * (r + eps) ** 2)
        J = jac(m, s, g, oracle.Adam(lr, b, b, eps, 1, bias_correction=False))
        Jd = jac(m, s, g, oracle.Adam(lr, b, b, eps, 1, bias_correction=False, drop_eps_term=True))
        assert J == pytest.approx(printed, rel=1e-12)
        assert Jd == pytest.approx(approx, rel=1e-12, abs=1e-18)


def test_rms_normalised_limit():
    """beta1 = 0, beta2 -> 1, eps = 0: the update is lr g / sqrt(s), so dJ = lr / sqrt(s)."""
    for s in [1e-6, 4e-4, 2.5]:
        J = jac(0.123, s, 0.5e-3, oracle.Adam(lr=2e-3, beta1=0.0, beta2=1.0 - 1e-15, eps=0.0, step=1,
                                               bias_correction=False))
        assert J == pytest.approx(2e-3 / np.sqrt(float(np.float32(s))), rel=1e-9)


def test_zero_state_limit():
    """s = 0 and g = 0: u = (lr/c1)(1-b1) g / ((sqrt(1-b2)/sqrt(c2)) |g| + eps) has slope (lr/c1)(1-b1)/eps at 0."""
    adam = oracle.Adam(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=10)
    c1 = 1 - 0.9 ** 10
    assert jac(0.0, 0.0, 0.0, adam) == pytest.approx(1e-3 / c1 * 0.1 / 1e-8, rel=1e-12)
    # agrees with the difference quotient of the update over a step far below eps
    h = LD(1e-14)
    d = (adam_update_ld(h, 0, 0, 1e-3, 0.9, 0.999, 1e-8, 10) - adam_update_ld(-h, 0, 0, 1e-3, 0.9, 0.999, 1e-8, 10)) / (2 * h)
    assert jac(0.0, 0.0, 0.0, adam) == pytest.approx(float(d), rel=1e-4)


def test_zero_state_value_of_the_printed_approximation():
    """drop_eps_term at s = 0 and g = 0 (r = 0), where the printed approximate form (Appendix C, last
    line) is 0/0.  The checker returns 0 there.  That is what the form itself fixes: along g = 0 it is
    lr (1-b1) r / (c1 sqrt(c2) D^2) with r^2 = b2 s, which goes to 0 with s; along s = 0 it tends to
    -+ lr b1 sqrt(1-b2) m / (c1 sqrt(c2) eps^2) for g -> 0+-, two one-sided limits whose mean is 0 (the same
    symmetric-derivative convention that gives the exact form its value (lr/c1)(1-b1)/eps at this point).
    Both statements are evaluated from the formula typed out here, and against the checker just off the point."""
    lr, b1, b2, eps, step = 1e-3, 0.9, 0.999, 1e-8, 10
    c1, c2 = 1 - b1 ** step, 1 - b2 ** step
    adam = oracle.Adam(lr, b1, b2, eps, step, drop_eps_term=True)
    for m in (0.0, 3e-4, -2e-3):
        assert jac(m, 0.0, 0.0, adam) == 0.0
        # along g = 0, once r is below eps: monotone to 0 with s, and equal to the typed-out expression
        prev = None
        for s in (1e-18, 1e-22, 1e-26, 1e-32, 1e-37):
            sd = float(np.float32(s))
            r = np.sqrt(b2 * sd)
            D = r / np.sqrt(c2) + eps
            expect = (lr / c1) * (1 - b1) * b2 * sd / (np.sqrt(c2) * r * D * D)
            J = jac(m, s, 0.0, adam)
            assert J == pytest.approx(expect, rel=1e-12)
            assert prev is None or abs(J) < abs(prev)
            prev = J
        assert abs(prev) < 1e-8 * (lr / c1) * (1 - b1) / eps
        # along s = 0: odd in g, with the one-sided limits typed out
        for g in (1e-20, 1e-24):
            Jp, Jm = jac(m, 0.0, g, adam), jac(m, 0.0, -g, adam)
            md = float(np.float32(m))
            lim = -(lr / c1) * b1 * np.sqrt(1 - b2) * md / (np.sqrt(c2) * eps ** 2)
            assert Jp == pytest.approx(lim, rel=1e-6, abs=1e-12)
            assert Jm == pytest.approx(-lim, rel=1e-6, abs=1e-12)
            assert Jp + Jm == pytest.approx(0.0, abs=1e-6 * max(abs(lim), 1e-12))


def test_other_optimisers_are_arguments_of_the_same_matrix():
    """Appendix C's last sentence (other optimisers' matrices "can be similarly derived"), checked by differentiating
    their updates numerically.  RMSprop, u = lr g / (sqrt(b s + (1-b) g^2) + eps), is the Adam matrix with beta1 = 0
    and no bias correction.  SGD with momentum, u = lr (mu buf + g), has du/dg = lr: a multiple of the identity,
    which the norm-scaled step of Sec. 3.2 cannot tell from identity = 1 (same theta+-, same direction)."""
    rng = np.random.default_rng(7)
    for _ in range(300):
        b, lr, eps = float(rng.uniform(0.8, 0.999)), float(10 ** rng.uniform(-4, -2)), float(10 ** rng.uniform(-10, -6))
        s, g = np.float32(abs(rng.normal()) * 1e-5 + 1e-8), np.float32(rng.normal() * 3e-3)
        u = lambda x: LD(lr) * x / (np.sqrt(LD(b) * LD(s) + (1 - LD(b)) * x * x) + LD(eps))
        h = LD(1e-4) * max(abs(LD(g)), np.sqrt(LD(s)))
        d = (-u(LD(g) + 2 * h) + 8 * u(LD(g) + h) - 8 * u(LD(g) - h) + u(LD(g) - 2 * h)) / (12 * h)
        J = jac(0.123, s, g, oracle.Adam(lr, 0.0, b, eps, 1, bias_correction=False))
        assert J == pytest.approx(float(d), rel=1e-6)
    w = W.flat_vector(500, 8)
    lr, mu = 0.05, 0.9
    p_sgd = lr * w["g_meta"].astype(np.float64)                 # (d/dg)[lr (mu buf + g)] * g_meta
    tp_a, tm_a, _, _ = oracle.perturb(w["theta"], p_sgd, 1e-2)
    tp_b, tm_b, _, _ = oracle.perturb(w["theta"], oracle.adapt(w["m"], w["s"], None, w["g_meta"], oracle.Adam(identity=True)), 1e-2)
    np.testing.assert_allclose(tp_a, tp_b, rtol=0, atol=1e-15)
    np.testing.assert_allclose(tm_a, tm_b, rtol=0, atol=1e-15)


def test_identity_mode_is_bit_exact_and_sgd_reduction():
    w = W.adam_state(1000, 3)
    p = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], oracle.Adam(identity=True))
    assert np.array_equal(p, w["g_meta"].astype(np.float64))


def test_adaptation_is_elementwise():
    w = W.adam_state(64, 4)
    adam = oracle.Adam()
    p0 = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], adam)
    for name in ["m", "s", "g_base", "g_meta"]:
        w2 = {k: v.copy() for k, v in w.items()}
        w2[name][17] *= np.float32(1.5)
        p1 = oracle.adapt(w2["m"], w2["s"], w2["g_base"], w2["g_meta"], adam)
        changed = np.nonzero(p1 != p0)[0]
        assert list(changed) == [17], (name, changed)


def test_adapt_is_linear_in_lr_and_gmeta():
    w = W.adam_state(257, 5)
    a, b = oracle.Adam(lr=1e-3), oracle.Adam(lr=4e-3)
    pa = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], a)
    pb = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], b)
    np.testing.assert_allclose(pb, 4 * pa, rtol=1e-6)  # 4e-3 and 1e-3 differ from 4:1 by double rounding of the literals
    pc = oracle.adapt(w["m"], w["s"], w["g_base"], 2 * w["g_meta"], a)
    np.testing.assert_array_equal(pc, 2 * pa)


# ----------------------------------------------------------------------------
# S2, S3: norm and perturbation (Sec. 3.2)
# ----------------------------------------------------------------------------

def test_perturbation_invariants():
    w = W.flat_vector(5001, 6)
    p = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], oracle.Adam())
    alpha = 0.37
    tp, tm, eps, bad = oracle.perturb(w["theta"], p, alpha)
    assert not bad
    th = w["theta"].astype(np.float64)
    assert eps == pytest.approx(alpha / np.linalg.norm(p), rel=1e-12)
    assert np.linalg.norm(tp - th) == pytest.approx(alpha, rel=1e-9)
    np.testing.assert_allclose((tp + tm) / 2, th, rtol=0, atol=1e-17)
    # flipping the direction swaps the branches; rescaling it changes nothing
    tp2, tm2, eps2, _ = oracle.perturb(w["theta"], -p, alpha)
    np.testing.assert_array_equal(tp2, tm)
    np.testing.assert_array_equal(tm2, tp)
    tp3, tm3, eps3, _ = oracle.perturb(w["theta"], 8.0 * p, alpha)
    np.testing.assert_allclose(tp3, tp, rtol=1e-14)
    assert eps3 == pytest.approx(eps / 8, rel=1e-12)
    assert oracle.sumsq(p) == pytest.approx(float(np.dot(p, p)), rel=1e-12)


def test_degenerate_norm_is_flagged():
    th = np.float32([1.0, -2.0, 3.0])
    tp, tm, eps, bad = oracle.perturb(th, np.zeros(3), 1.0)
    assert bad and eps == 0.0
    np.testing.assert_array_equal(tp, th.astype(np.float64))
    np.testing.assert_array_equal(tm, th.astype(np.float64))
    _, _, _, bad = oracle.perturb(th, np.array([1.0, np.inf, 0.0]), 1.0)
    assert bad
    _, _, _, bad = oracle.perturb(th, np.array([1.0, np.nan, 0.0]), 1.0)
    assert bad


# ----------------------------------------------------------------------------
# S4: forward pass and cross-entropy
# ----------------------------------------------------------------------------

def numpy_losses(dims, theta, X, y, dtype=np.float64):
    """Library-matmul statement of the same MLP (row-major [out][in] weights)."""
    theta = np.asarray(theta, dtype=dtype)
    h = np.asarray(X, dtype=dtype)
    o = 0
    L = len(dims) - 1
    for l in range(L):
        Wl = theta[o:o + dims[l] * dims[l + 1]].reshape(dims[l + 1], dims[l])
        o += dims[l] * dims[l + 1]
        b = theta[o:o + dims[l + 1]]
        o += dims[l + 1]
        h = h @ Wl.T + b
        if l + 1 < L:
            h = np.maximum(h, 0)
    zmax = h.max(axis=1, keepdims=True)
    lse = np.log(np.exp(h - zmax).sum(axis=1)) + zmax[:, 0]
    return lse - h[np.arange(len(y)), y], h


@pytest.mark.parametrize("dims,B", [((7, 5, 3), 9), ((33, 17, 12, 6), 20), ((10, 4), 11)])
def test_forward_matches_library_matmul(dims, B):
    cfg, w = W.custom_mlp(dims, B, seed=7)
    theta = w["theta"].astype(np.float64)
    theta += 0.05 * W.normal(7, 99, theta.size)  # non-zero biases
    got, logits = oracle.losses(dims, theta, w["X"], w["y"], want_logits=True)
    ref, ref_logits = numpy_losses(dims, theta, w["X"], w["y"])
    np.testing.assert_allclose(logits, ref_logits, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_cross_entropy_known_values():
    # single linear layer with W = 0: logits are the bias, loss = log C for zero bias
    dims = (3, 4)
    theta = np.zeros(3 * 4 + 4)
    X = np.float32([[1, 2, 3], [4, 5, 6]])
    y = np.int32([0, 3])
    np.testing.assert_allclose(oracle.losses(dims, theta, X, y), np.log(4.0), rtol=1e-15)
    theta[12:] = [0.0, np.log(2.0), 0.0, np.log(5.0)]      # softmax = (1,2,1,5)/9
    np.testing.assert_allclose(oracle.losses(dims, theta, X, y), [np.log(9.0), np.log(9.0 / 5.0)], rtol=1e-14)
    # huge logits do not overflow
    theta[12:] = [1000.0, 0.0, 0.0, 999.0]
    l = oracle.losses(dims, theta, X, y)
    assert l[0] == pytest.approx(np.log1p(np.exp(-1.0)), rel=1e-12)
    assert l[1] == pytest.approx(1.0 + np.log1p(np.exp(-1.0)), rel=1e-12)


def test_relu_applies_to_hidden_layers_only():
    dims = (1, 1, 2)
    # hidden = relu(-x) = 0 for x > 0; logits = b2 = (-3, 1): a ReLU on the last layer would give (0, 1)
    theta = np.array([-1.0, 0.0, 5.0, 7.0, -3.0, 1.0])
    l, z = oracle.losses(dims, theta, np.float32([[2.0]]), np.int32([0]), want_logits=True)
    np.testing.assert_allclose(z, [[-3.0, 1.0]])
    assert l[0] == pytest.approx(np.log(np.exp(-3.0) + np.exp(1.0)) + 3.0, rel=1e-13)


# ----------------------------------------------------------------------------
# S5 / whole step: finite-difference meta-gradient (Eq. 5)
# ----------------------------------------------------------------------------

def small_step(dims, B, seed, alpha, adam=None, flip=False, scale_gmeta=1.0, lam=None):
    cfg, w = W.custom_mlp(dims, B, seed=seed)
    gm = w["g_meta"] * np.float32(-scale_gmeta if flip else scale_gmeta)
    lam = w["lam"] if lam is None else lam
    out = oracle.step(dims, w["theta"], w["m"], w["s"], w["g_base"], gm, adam or oracle.Adam(), alpha,
                      w["X"], w["y"], lam)
    return w, out


def test_fd_matches_closed_form_on_linear_softmax():
    """One linear layer: d^2 L_base / dlambda_i dtheta . p =
    sigmoid'(lambda_i)/B * (softmax(W x_i + b) - e_{y_i})^T (P_W x_i + p_b).
    The central difference must agree up to O(eps_fd^2), i.e. the error must
    fall about 100x when alpha falls 10x."""
    dims, B = (12, 5), 16
    errs = []
    for alpha in [1e-1, 1e-2]:
        w, out = small_step(dims, B, seed=11, alpha=alpha)
        p = out["p"]
        PW, pb = p[:60].reshape(5, 12), p[60:]
        Wm, b = w["theta"][:60].astype(np.float64).reshape(5, 12), w["theta"][60:].astype(np.float64)
        X = w["X"].astype(np.float64)
        z = X @ Wm.T + b
        sm = np.exp(z - z.max(1, keepdims=True))
        sm /= sm.sum(1, keepdims=True)
        sm[np.arange(B), w["y"]] -= 1.0
        dz = X @ PW.T + pb
        sg = 1 / (1 + np.exp(-w["lam"].astype(np.float64)))
        exact = -(sg * (1 - sg)) / B * (sm * dz).sum(1)
        errs.append(np.abs(out["metagrad"] - exact).max() / np.abs(exact).max())
    assert errs[0] < 5e-2 and errs[1] < 5e-4, errs
    assert 30 < errs[0] / errs[1] < 300, errs


def l_base_ld(dims, theta, X, y, lam):
    """L_base(theta, lambda) = mean_i sigmoid(lambda_i) CE_i in extended precision."""
    losses, _ = numpy_losses(dims, np.asarray(theta, dtype=LD), np.asarray(X, dtype=LD), y, dtype=LD)
    sg = 1 / (1 + np.exp(-np.asarray(lam, dtype=LD)))
    return (sg * losses).mean()


@pytest.mark.parametrize("dims,B", [((3, 4, 2), 5), ((4, 3, 3, 2), 4)])
def test_fd_matches_nested_brute_force(dims, B):
    """-d/dlambda_i [ directional derivative of L_base along p ] by nested
    central differences of the scalar objective, against the checker's Eq. 5
    with a small alpha (so its own truncation error is negligible)."""
    w, out = small_step(dims, B, seed=13, alpha=1e-4)
    p = out["p"].astype(LD)
    theta, lam = w["theta"].astype(LD), w["lam"].astype(LD)
    ht, hl = LD(1e-5) / np.sqrt((p * p).sum()), LD(1e-5)
    ref = np.zeros(B)
    for i in range(B):
        e = np.zeros(B, dtype=LD)
        e[i] = hl
        f = lambda st, sl: l_base_ld(dims, theta + st * ht * p, w["X"], w["y"], lam + sl * e)
        ref[i] = -float((f(1, 1) - f(1, -1) - f(-1, 1) + f(-1, -1)) / (4 * ht * hl))
    np.testing.assert_allclose(out["metagrad"], ref, rtol=2e-4, atol=1e-5 * np.abs(ref).max())


def test_fd_antisymmetry_and_scaling():
    dims, B = (9, 6, 4), 10
    _, a = small_step(dims, B, 17, 1e-2)
    _, b = small_step(dims, B, 17, 1e-2, flip=True)
    np.testing.assert_array_equal(b["metagrad"], -a["metagrad"])
    np.testing.assert_array_equal(b["theta_plus"], a["theta_minus"])
    # g_meta -> c g_meta: same theta+-, eps_fd / c, metagrad * c
    _, c = small_step(dims, B, 17, 1e-2, scale_gmeta=4.0)
    np.testing.assert_allclose(c["theta_plus"], a["theta_plus"], rtol=1e-14)
    np.testing.assert_allclose(c["metagrad"], 4 * a["metagrad"], rtol=1e-9)
    # lr only rescales p: theta+- unchanged
    _, d = small_step(dims, B, 17, 1e-2, adam=oracle.Adam(lr=8e-3))
    np.testing.assert_allclose(d["theta_plus"], a["theta_plus"], rtol=1e-13)


def test_fd_saturated_weights_and_permutation():
    dims, B = (6, 5, 3), 8
    w, a = small_step(dims, B, 19, 1e-2)
    lam = w["lam"].copy()
    lam[2], lam[5] = 80.0, -80.0
    _, b = small_step(dims, B, 19, 1e-2, lam=lam)
    assert abs(b["metagrad"][2]) < 1e-30 and abs(b["metagrad"][5]) < 1e-30
    keep = [i for i in range(B) if i not in (2, 5)]
    np.testing.assert_array_equal(b["metagrad"][keep], a["metagrad"][keep])
    perm = np.array([3, 0, 7, 1, 6, 2, 5, 4])
    c = oracle.step(dims, w["theta"], w["m"], w["s"], w["g_base"], w["g_meta"], oracle.Adam(), 1e-2,
                    w["X"][perm], w["y"][perm], w["lam"][perm])
    np.testing.assert_array_equal(c["metagrad"], a["metagrad"][perm])


def test_batch_normaliser_and_subset():
    dims, B = (6, 5, 3), 8
    w, a = small_step(dims, B, 23, 1e-2)
    sub = oracle.step(dims, w["theta"], w["m"], w["s"], w["g_base"], w["g_meta"], oracle.Adam(), 1e-2,
                      w["X"][:3], w["y"][:3], w["lam"][:3], B_norm=B)
    np.testing.assert_array_equal(sub["metagrad"], a["metagrad"][:3])
    lp = oracle.losses(dims, a["theta_plus"], w["X"], w["y"])
    lm = oracle.losses(dims, a["theta_minus"], w["X"], w["y"])
    np.testing.assert_array_equal(oracle.fd(lp, lm, w["lam"], a["eps_fd"], B), a["metagrad"])
    np.testing.assert_allclose(oracle.fd(lp, lm, w["lam"], a["eps_fd"], 2 * B), a["metagrad"] / 2, rtol=1e-15)


def test_fd_sign_descends_meta_loss_direction():
    """Sign convention of Eq. 2/Eq. 5 on a case with a known answer: SGD base
    (identity adaptation), g_meta = gradient of sample j's own loss.  Raising
    sample j's weight makes the base step reduce that loss, so the meta
    gradient w.r.t. lambda_j must be negative (it equals
    -sigmoid'(lambda_j)/B * |grad loss_j|^2 up to the 1/||p|| scale and O(eps^2))."""
    dims, B = (5, 3), 6
    cfg, w = W.custom_mlp(dims, B, seed=29)
    j = 2
    Wm, b = w["theta"][:15].astype(np.float64).reshape(3, 5), w["theta"][15:].astype(np.float64)
    x = w["X"][j].astype(np.float64)
    z = Wm @ x + b
    sm = np.exp(z - z.max())
    sm /= sm.sum()
    sm[w["y"][j]] -= 1
    grad = np.concatenate([np.outer(sm, x).ravel(), sm]).astype(np.float32)
    out = oracle.step(dims, w["theta"], w["m"], w["s"], None, grad, oracle.Adam(identity=True), 1e-3,
                      w["X"], w["y"], w["lam"])
    sg = 1 / (1 + np.exp(-float(w["lam"][j])))
    gd = grad.astype(np.float64)
    expect = -sg * (1 - sg) / B * np.dot(gd, gd)
    assert out["metagrad"][j] < 0
    assert out["metagrad"][j] == pytest.approx(expect, rel=1e-4)


# ----------------------------------------------------------------------------
# Direct gradient dL_meta/dtheta (first factor of Eq. 1)
# ----------------------------------------------------------------------------

@pytest.mark.parametrize("dims,B", [((5, 3), 4), ((6, 5, 3), 7), ((4, 6, 5, 3), 5)])
def test_meta_grad_matches_brute_force_differences(dims, B):
    """Every component against a central difference of the mean cross-entropy (computed by the
    forward pass, which has its own pins) in extended precision."""
    cfg, w = W.custom_mlp(dims, B, seed=31)
    theta = (w["theta"] + 0.1 * W.normal(31, 77, w["theta"].size).astype(np.float32)).astype(np.float32)
    loss, g = oracle.meta_grad(dims, theta, w["X"], w["y"])
    f = lambda t: numpy_losses(dims, t, np.asarray(w["X"], dtype=LD), w["y"], dtype=LD)[0].mean()
    assert loss == pytest.approx(float(f(theta.astype(LD))), rel=1e-12)
    ref = np.zeros(theta.size)
    for k in range(theta.size):
        e = np.zeros(theta.size, dtype=LD)
        e[k] = LD(1e-6)
        ref[k] = float((f(theta.astype(LD) + e) - f(theta.astype(LD) - e)) / LD(2e-6))
    np.testing.assert_allclose(g, ref, rtol=1e-6, atol=1e-9)


def test_meta_grad_single_layer_closed_form():
    dims, B = (7, 4), 9
    cfg, w = W.custom_mlp(dims, B, seed=33)
    theta = w["theta"]
    Wm, b = theta[:28].astype(np.float64).reshape(4, 7), theta[28:].astype(np.float64)
    X = w["X"].astype(np.float64)
    z = X @ Wm.T + b
    sm = np.exp(z - z.max(1, keepdims=True))
    sm /= sm.sum(1, keepdims=True)
    sm[np.arange(B), w["y"]] -= 1
    _, g = oracle.meta_grad(dims, theta, w["X"], w["y"])
    np.testing.assert_allclose(g[:28].reshape(4, 7), sm.T @ X / B, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(g[28:], sm.sum(0) / B, rtol=1e-12, atol=1e-15)
