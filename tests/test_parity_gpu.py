"""GPU parity: the C-ABI CUDA path against the CPU checker, element by element,
on the same seeded inputs.

Tolerances (the library's stated accuracy targets):
  adaptation / perturbation : relative 1e-5 elementwise, eps_fd relative 1e-6;
  FD meta-gradient          : |a-b| <= max(2e-3 |b|, 1e-6) elementwise, plus the
                              same 2e-3 on the whole vector in the 2-norm.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_05674_b200 import workloads as W

pytestmark = pytest.mark.gpu

from gpu_util import (B, Ctx, DEV, assert_adapt_close, assert_fd_close, dev, fd_errors, read_f32, read_f64,  # noqa: E402
                      run_adapt, run_step, unaligned)


def o_adam(a: "B.Adam") -> oracle.Adam:
    """The same hyper-parameters as the C ABI receives them: rounded to fp32."""
    f = lambda x: float(np.float32(x))
    return oracle.Adam(f(a.lr), f(a.beta1), f(a.beta2), f(a.eps), a.step, a.bias_correction, a.drop_eps_term,
                       a.identity)


ADAMS = {
    "default": B.Adam(),
    "step1": B.Adam(step=1),
    "step1000": B.Adam(step=1000),
    "nobias": B.Adam(bias_correction=False),
    "dropeps": B.Adam(drop_eps_term=True),
    "identity": B.Adam(identity=True),
    "odd": B.Adam(lr=3e-2, beta1=0.8, beta2=0.99, eps=1e-6, step=7),
    "rmsprop": B.Adam(lr=1e-2, beta1=0.0, beta2=0.99, eps=1e-8, bias_correction=False),   # RMSprop's matrix (Appendix C, last sentence)
}


# ---------------------------------------------------------------- adapt ----

@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 1023, 1025, 2 ** 20 + 1])
@pytest.mark.parametrize("mode", sorted(ADAMS))
def test_adapt_parity(n, mode):
    adam = ADAMS[mode]
    w = W.flat_vector(n, seed=n + 1)
    ref = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], o_adam(adam))
    with Ctx(max(n, 1)) as ctx:
        p, ss, _, _ = run_adapt(ctx, w, adam)
        assert_adapt_close(p, ref)
        if mode == "identity":
            assert np.array_equal(p, w["g_meta"])
        assert ss == pytest.approx(float(np.dot(p.astype(np.float64), p.astype(np.float64))), rel=1e-12, abs=1e-300)
        assert ss == pytest.approx(oracle.sumsq(ref), rel=2e-6, abs=1e-300)
        assert read_f64(B.sama_ctx_sumsq(ctx.h)) == ss


@pytest.mark.parametrize("n", [5, 1025, 300001])
def test_adapt_variants(n):
    adam = B.Adam()
    w = W.flat_vector(n, seed=77)
    with Ctx(n) as ctx:
        base, ss0, _, _ = run_adapt(ctx, w, adam)
        # g_base = NULL means g := m
        ref = oracle.adapt(w["m"], w["s"], None, w["g_meta"], o_adam(adam))
        p, _, _, _ = run_adapt(ctx, w, adam, use_gbase=False)
        assert_adapt_close(p, ref)
        # unaligned pointers take the scalar kernels
        full = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], o_adam(adam))
        for shift in (1, 3):
            p, ss, _, _ = run_adapt(ctx, w, adam, shift=shift)
            assert_adapt_close(p, full)
            assert ss == pytest.approx(ss0, rel=1e-6)
        # in place over g_meta
        p, ss, _, _ = run_adapt(ctx, w, adam, inplace=True)
        assert np.array_equal(p, base) and ss == ss0
        # repeated calls are bit-identical (fixed reduction order)
        p2, ss2, _, _ = run_adapt(ctx, w, adam)
        assert np.array_equal(p2, base) and ss2 == ss0


def test_adapt_zero_state_corner():
    """Elements with s = 0 and g = 0 (r = 0): the exact form takes its limit (lr/c1)(1-b1)/eps, the printed
    approximation (drop_eps_term) is 0 there, whatever m is; neighbours are untouched."""
    n = 4099
    w = W.flat_vector(n, seed=21)
    zero = np.arange(0, n, 7)
    for k in ("s", "g_base"):
        w[k] = w[k].copy()
        w[k][zero] = 0.0
    w["m"] = w["m"].copy()
    w["m"][zero[::2]] = 0.0
    with Ctx(n) as ctx:
        for adam in (B.Adam(step=10), B.Adam(step=10, drop_eps_term=True), B.Adam(bias_correction=False, drop_eps_term=True)):
            ref = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], o_adam(adam))
            for shift in (0, 1):
                p, ss, _, _ = run_adapt(ctx, w, adam, shift=shift)
                assert np.all(np.isfinite(p))
                if adam.drop_eps_term:
                    assert np.all(p[zero] == 0.0) and np.all(ref[zero] == 0.0)
                # the limit is ~1e4 times a typical entry: compare it relative to itself, the rest as usual
                assert np.all(np.abs(p[zero] - ref[zero]) <= 1e-5 * np.abs(ref[zero]))
                rest = np.setdiff1d(np.arange(n), zero)
                assert_adapt_close(p[rest], ref[rest])
                assert ss == pytest.approx(oracle.sumsq(ref), rel=2e-6)


# -------------------------------------------------------------- perturb ----

@pytest.mark.parametrize("n", [1, 3, 4, 1023, 1025, 2 ** 20 + 1])
def test_perturb_parity(n):
    w = W.flat_vector(n, seed=n + 5)
    adam, alpha = B.Adam(), 0.37
    with Ctx(n) as ctx:
        p_np, ss, p_dev, ss_dev = run_adapt(ctx, w, adam)
        rtp, rtm, reps, bad = oracle.perturb(w["theta"], p_np, alpha)
        assert not bad
        theta = dev(w["theta"])
        tp, tm = torch.empty_like(theta), torch.empty_like(theta)
        eps = torch.zeros(1, dtype=torch.float32, device=DEV)
        B.sama_perturb(ctx.h, n, theta, p_dev, ss_dev, alpha, tp, tm, eps)
        torch.cuda.synchronize()
        assert float(eps.item()) == pytest.approx(reps, rel=1e-6)
        assert read_f32(B.sama_ctx_eps_fd(ctx.h)) == float(eps.item())
        assert_adapt_close(tp.cpu().numpy(), rtp, "theta_plus")
        assert_adapt_close(tm.cpu().numpy(), rtm, "theta_minus")
        # the displacement itself, not just theta + small: (theta+ - theta-)/2 = eps p to fp32 rounding of theta
        d = (tp.double() - tm.double()).cpu().numpy() / 2
        ulp = np.abs(w["theta"]).astype(np.float64) * 2.0 ** -23
        assert np.all(np.abs(d - reps * p_np.astype(np.float64)) <= 1e-5 * np.abs(reps * p_np) + ulp)
        # norm computed inside (p_sumsq = NULL) gives the same result
        tp2, tm2 = torch.empty_like(theta), torch.empty_like(theta)
        B.sama_perturb(ctx.h, n, theta, p_dev, None, alpha, tp2, tm2, None)
        torch.cuda.synchronize()
        assert read_f32(B.sama_ctx_eps_fd(ctx.h)) == pytest.approx(float(eps.item()), rel=1e-6)
        assert_adapt_close(tp2.cpu().numpy(), rtp)
        # theta_minus aliasing theta: the base-parameter nudge
        th2 = theta.clone()
        B.sama_perturb(ctx.h, n, th2, p_dev, ss_dev, alpha, tp2, th2, None)
        torch.cuda.synchronize()
        assert torch.equal(th2, tm) and torch.equal(tp2, tp)
        # unaligned
        thu, tpu, tmu = unaligned(w["theta"], 1), unaligned(np.zeros(n, np.float32), 1), unaligned(np.zeros(n, np.float32), 1)
        B.sama_perturb(ctx.h, n, thu, p_dev, ss_dev, alpha, tpu, tmu, None)
        torch.cuda.synchronize()
        assert torch.equal(tpu, tp) and torch.equal(tmu, tm)
        assert B.sama_device_status(ctx.h) == 0


def test_perturb_degenerate_norm_sets_status():
    n = 1000
    with Ctx(n) as ctx:
        theta = dev(W.flat_vector(n, 3)["theta"])
        for bad_p in (np.zeros(n, np.float32), np.full(n, np.nan, np.float32), np.full(n, 3e38, np.float32).astype(np.float32) * np.float32(1e30)):
            p = dev(bad_p.astype(np.float32))
            tp, tm = torch.empty_like(theta), torch.empty_like(theta)
            eps = torch.ones(1, dtype=torch.float32, device=DEV)
            B.sama_perturb(ctx.h, n, theta, p, None, 1.0, tp, tm, eps)
            assert B.sama_device_status(ctx.h) == B.SAMA_DEV_DEGENERATE_NORM
            assert float(eps.item()) == 0.0
            assert torch.equal(tp, theta) and torch.equal(tm, theta)
        assert B.sama_device_status(ctx.h) == 0  # reading clears


# ---------------------------------------------------- forward + FD alone ----

RAGGED = [((12, 5), 1), ((33, 17, 12, 6), 7), ((100, 50, 3), 129), ((257, 130, 66, 11), 65), ((64, 64, 64, 16), 300),
          ((40, 200, 72, 24), 257)]

# 1 = fp32 FMA on the CUDA cores, 2 = tensor cores (three TF32 products per fp32 product)
GEMM_MODES = [1, 2]
# sama_step also has mode 3: tensor cores, with the weights of both branches formed in the product kernel's
# operand stage from theta and p instead of being read as a pre-split copy
STEP_MODES = [1, 2, 3]


@pytest.mark.parametrize("gemm_mode", GEMM_MODES)
@pytest.mark.parametrize("dims,batch", RAGGED)
def test_fd_metagrad_parity_ragged(dims, batch, gemm_mode):
    cfg, w = W.custom_mlp(dims, batch, seed=sum(dims))
    n = cfg.n_params
    # non-zero biases and a realistic pair theta+-
    theta = (w["theta"] + 0.05 * W.normal(5, 99, n).astype(np.float32)).astype(np.float32)
    d = (1e-3 * W.normal(6, 98, n)).astype(np.float32)
    tp_np, tm_np = (theta + d).astype(np.float32), (theta - d).astype(np.float32)
    eps_val = np.float32(0.05)
    lp = oracle.losses(dims, tp_np, w["X"], w["y"])
    lm = oracle.losses(dims, tm_np, w["X"], w["y"])
    ref = oracle.fd(lp, lm, w["lam"], float(eps_val), batch)
    with Ctx(n, batch, dims, gemm_mode) as ctx:
        out = [torch.empty(batch, dtype=torch.float32, device=DEV) for _ in range(3)]
        B.sama_fd_metagrad(ctx.h, ctx.mlp, dev(tp_np), dev(tm_np), dev(w["X"]), dev(w["y"]), dev(w["lam"]), batch,
                           dev(np.array([eps_val])), out[0], out[1], out[2])
        torch.cuda.synchronize()
        np.testing.assert_allclose(out[1].cpu().numpy(), lp, rtol=2e-5, atol=2e-5)
        np.testing.assert_allclose(out[2].cpu().numpy(), lm, rtol=2e-5, atol=2e-5)
        assert_fd_close(out[0].cpu().numpy(), ref)
        # the loss outputs are optional
        mg2 = torch.empty(batch, dtype=torch.float32, device=DEV)
        B.sama_fd_metagrad(ctx.h, ctx.mlp, dev(tp_np), dev(tm_np), dev(w["X"]), dev(w["y"]), dev(w["lam"]), batch,
                           dev(np.array([eps_val])), mg2, None, None)
        torch.cuda.synchronize()
        assert torch.equal(mg2, out[0])
        assert B.sama_device_status(ctx.h) == 0


def test_bad_label_is_reported_not_faulted():
    dims, batch = (20, 9, 4), 10
    cfg, w = W.custom_mlp(dims, batch, seed=4)
    y = w["y"].copy()
    y[3], y[7] = 4, -1
    with Ctx(cfg.n_params, batch, dims) as ctx:
        mg = torch.empty(batch, dtype=torch.float32, device=DEV)
        th = dev(w["theta"])
        B.sama_fd_metagrad(ctx.h, ctx.mlp, th, dev(w["theta"] * np.float32(1.01)), dev(w["X"]), dev(y),
                           dev(w["lam"]), batch, dev(np.float32([0.1])), mg, None, None)
        assert B.sama_device_status(ctx.h) == B.SAMA_DEV_BAD_LABEL
        mg = mg.cpu().numpy()
        assert mg[3] == 0 and mg[7] == 0 and np.all(mg[[0, 1, 2, 4, 5, 6, 8, 9]] != 0)


@pytest.mark.parametrize("gemm_mode", GEMM_MODES)
@pytest.mark.parametrize("dims", [(160, 136, 72, 24), (160, 136, 10)])
def test_non_finite_input_is_not_hidden(dims, gemm_mode):
    """One NaN in X makes that sample's losses and meta-gradient NaN in both forward modes (a ReLU written as
    max(x, 0) would turn it into a finite number), and leaves every other sample untouched."""
    batch = 140
    cfg, w = W.custom_mlp(dims, batch, seed=31)
    theta = w["theta"]
    d = (1e-3 * W.normal(6, 97, cfg.n_params)).astype(np.float32)
    tp_np, tm_np = (theta + d).astype(np.float32), (theta - d).astype(np.float32)
    X = w["X"].copy()
    X[57, 11] = np.nan
    eps_val = np.float32(0.05)
    lp = oracle.losses(dims, tp_np, X, w["y"])
    lm = oracle.losses(dims, tm_np, X, w["y"])
    ref = oracle.fd(lp, lm, w["lam"], float(eps_val), batch)
    assert np.isnan(lp[57]) and np.isnan(ref[57]) and np.isfinite(np.delete(ref, 57)).all()
    with Ctx(cfg.n_params, batch, dims, gemm_mode) as ctx:
        out = [torch.empty(batch, dtype=torch.float32, device=DEV) for _ in range(3)]
        B.sama_fd_metagrad(ctx.h, ctx.mlp, dev(tp_np), dev(tm_np), dev(X), dev(w["y"]), dev(w["lam"]), batch,
                           dev(np.array([eps_val])), out[0], out[1], out[2])
        torch.cuda.synchronize()
        mg, glp, glm = (o.cpu().numpy() for o in out)
        assert np.isnan(mg[57]) and np.isnan(glp[57]) and np.isnan(glm[57])
        keep = np.arange(batch) != 57
        assert_fd_close(mg[keep], ref[keep])
        np.testing.assert_allclose(glp[keep], lp[keep], rtol=2e-5, atol=2e-5)
        assert B.sama_last_forward_path(ctx.h) == gemm_mode


# ------------------------------------------------------------ whole step ----

_REF_CACHE = {}


def check_step(cfg, w, adam, alpha, rows=None, use_gbase=True, gemm_mode=0, key=None):
    """Runs sama_step on the full batch; the checker runs on ``rows`` (all if None).
    ``key`` caches the checker's result across the gemm modes of one workload."""
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, gemm_mode) as ctx:
        got = run_step(ctx, cfg, w, adam, alpha, use_gbase=use_gbase)
    sel = slice(None) if rows is None else rows
    ref = _REF_CACHE.get(key) if key else None
    if ref is None:
        ref = oracle.step(cfg.dims, w["theta"], w["m"], w["s"], w["g_base"] if use_gbase else None, w["g_meta"],
                          o_adam(adam), alpha, w["X"][sel], w["y"][sel], w["lam"][sel], B_norm=cfg.batch)
        if key:
            _REF_CACHE[key] = ref
    assert got["status"] == 0 and not ref["degenerate"]
    assert_adapt_close(got["p"], ref["p"])
    assert got["eps_fd"] == pytest.approx(ref["eps_fd"], rel=1e-6)
    assert_adapt_close(got["theta_plus"], ref["theta_plus"], "theta_plus")
    assert_adapt_close(got["theta_minus"], ref["theta_minus"], "theta_minus")
    np.testing.assert_allclose(got["loss_plus"][sel], ref["loss_plus"], rtol=1e-4, atol=1e-4)
    # Norm-wise bound: 2e-3, the stated relative tolerance, on the default (tensor-core, three-product TF32) path
    # at every alpha.  The fp32 FMA path (gemm_mode 1) accumulates each logit in one chain of K roundings, which
    # the quotient amplifies by 1/(2 eps_fd): at alpha = 1e-2 it is held to 2e-2 (measured up to 1.0e-2 at K = 4096).
    norm_tol = 2e-2 if (gemm_mode == 1 and alpha < 1.0) else 2e-3
    e = assert_fd_close(got["metagrad"][sel], ref["metagrad"], norm_tol=norm_tol)
    # the per-sample difference quotient before the sigmoid'/B scaling, same bound in the 2-norm (the published
    # fp32 losses each carry half an ulp of rounding, which the difference of two of them inherits)
    dq = (got["loss_plus"].astype(np.float64) - got["loss_minus"].astype(np.float64))[sel]
    dr = ref["loss_plus"] - ref["loss_minus"]
    e["dq_norm_rel"] = float(np.linalg.norm(dq - dr) / np.linalg.norm(dr))
    ulp = 2.0 ** -24 * float(np.linalg.norm(np.abs(ref["loss_plus"]) + np.abs(ref["loss_minus"])))
    assert e["dq_norm_rel"] <= norm_tol + ulp / float(np.linalg.norm(dr)), e
    print("\n[parity] %s alpha=%g gemm_mode=%d: %s" % (cfg.name, alpha, gemm_mode, e))
    return e


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
@pytest.mark.parametrize("alpha", [1e-2, 1.0])
def test_step_parity_tiny(alpha, gemm_mode):
    cfg = W.CONFIGS["tiny"]
    check_step(cfg, W.mlp_workload(cfg, 0), B.Adam(), alpha, gemm_mode=gemm_mode, key=("tiny", alpha))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
def test_step_parity_tiny_variants(gemm_mode):
    cfg = W.CONFIGS["tiny"]
    w = W.mlp_workload(cfg, 0)
    check_step(cfg, w, B.Adam(), 1e-2, use_gbase=False, gemm_mode=gemm_mode, key=("tiny", "nog"))
    check_step(cfg, w, B.Adam(identity=True), 1.0, gemm_mode=gemm_mode, key=("tiny", "id"))
    if gemm_mode != 1:
        # SAMA-NA at the benchmark's alpha: entries are ~30x larger than with the Adam matrix, so the absolute
        # floor no longer absorbs rounding.  The tensor-core path holds the elementwise bar (worst entry at 0.99 of
        # it); the fp32 FMA path does not (11 of 128 entries over, up to 2.4x) and is tested at alpha = 1 only.
        check_step(cfg, w, B.Adam(identity=True), 1e-2, gemm_mode=gemm_mode, key=("tiny", "id-2"))
    check_step(cfg, w, B.Adam(step=1, drop_eps_term=True), 1e-2, gemm_mode=gemm_mode, key=("tiny", "drop"))
    check_step(cfg, w, B.Adam(bias_correction=False), 1.0, use_gbase=False, gemm_mode=gemm_mode, key=("tiny", "nobias"))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
@pytest.mark.parametrize("dims,batch", RAGGED[1:])
def test_step_parity_ragged(dims, batch, gemm_mode):
    cfg, w = W.custom_mlp(dims, batch, seed=3 + sum(dims))
    check_step(cfg, w, B.Adam(), 1e-2, gemm_mode=gemm_mode, key=("ragged", dims, batch))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
def test_step_parity_mlp3072(gemm_mode):
    cfg = W.CONFIGS["mlp3072"]
    w = W.mlp_workload(cfg, 0)
    check_step(cfg, w, B.Adam(), 1e-2, gemm_mode=gemm_mode, key=("mlp3072", 1e-2))
    check_step(cfg, w, B.Adam(), 1.0, rows=np.arange(0, cfg.batch, 8), gemm_mode=gemm_mode, key=("mlp3072", 1.0))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
def test_step_parity_head1024(gemm_mode):
    cfg = W.CONFIGS["head1024"]
    w = W.mlp_workload(cfg, 0)
    check_step(cfg, w, B.Adam(), 1e-2, gemm_mode=gemm_mode, key=("head1024", 1e-2))
    check_step(cfg, w, B.Adam(), 1.0, rows=np.arange(0, cfg.batch, 64), gemm_mode=gemm_mode, key=("head1024", 1.0))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
def test_step_parity_wide4096_sampled(gemm_mode):
    """Full-size launch; the checker evaluates a sample of the rows (each output
    depends only on its own row given theta+-, which are compared in full)."""
    cfg = W.CONFIGS["wide4096"]
    w = W.mlp_workload(cfg, 0)
    rows = np.unique(np.concatenate([np.arange(0, cfg.batch, 97), [cfg.batch - 1]]))
    check_step(cfg, w, B.Adam(), 1e-2, rows=rows, gemm_mode=gemm_mode, key=("wide4096", 1e-2))
    check_step(cfg, w, B.Adam(), 1.0, rows=rows[::2], gemm_mode=gemm_mode, key=("wide4096", 1.0))


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
def test_step_is_bitwise_reproducible(gemm_mode):
    """Fixed reduction orders everywhere (norm partials, split-K partial tiles): repeated steps agree bit for bit."""
    for cfg, w in [(W.CONFIGS["tiny"], W.mlp_workload(W.CONFIGS["tiny"], 0)), W.custom_mlp((40, 200, 72, 24), 257, seed=5),
                   W.custom_mlp((2048, 512, 40), 256, seed=6)]:
        with Ctx(cfg.n_params, cfg.batch, cfg.dims, gemm_mode) as ctx:
            runs = [run_step(ctx, cfg, w, B.Adam(), 1e-2) for _ in range(3)]
        for r in runs[1:]:
            for k in ("p", "theta_plus", "metagrad", "loss_plus", "loss_minus"):
                assert np.array_equal(r[k], runs[0][k]), (cfg.name, k)
            assert r["sumsq"] == runs[0]["sumsq"] and r["eps_fd"] == runs[0]["eps_fd"]


@pytest.mark.parametrize("pairs", ["1", "0"])
def test_several_tiles_per_cta(monkeypatch, pairs):
    """More output tiles than SMs: every CTA (or CTA pair; SAMA_TC_PAIR=0 forces single CTAs) of the
    persistent tensor-core kernel walks several tiles, with its copy pipeline and accumulators running
    across the tile boundary; the contraction (10 k-blocks) ends on a short chunk.  Same parity bar,
    bitwise repeatable."""
    monkeypatch.setenv("SAMA_TC_PAIR", pairs)
    cfg, w = W.custom_mlp((300, 2304, 40), 1200, seed=8)
    check_step(cfg, w, B.Adam(), 1.0, gemm_mode=2)
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, 2) as ctx:
        a = run_step(ctx, cfg, w, B.Adam(), 1.0)
        b = run_step(ctx, cfg, w, B.Adam(), 1.0)
    assert np.array_equal(a["metagrad"], b["metagrad"]) and np.array_equal(a["loss_plus"], b["loss_plus"])


def test_shared_tail_tiles_of_the_pair_kernel():
    """100 pair tiles on 74 resident CTA pairs: after one full round the 26 remaining tiles are each
    shared by two pairs (half of the 16 k-blocks each), which exchange partial sums through the
    workspace with arrival counters in global memory.  Same parity bar, bitwise repeatable, counters
    back at zero (the second and third call reuse them)."""
    cfg, w = W.custom_mlp((512, 2560, 40), 1280, seed=9)
    check_step(cfg, w, B.Adam(), 1.0, gemm_mode=2)
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, 2) as ctx:
        a = run_step(ctx, cfg, w, B.Adam(), 1.0)
        b = run_step(ctx, cfg, w, B.Adam(), 1.0)
        c = run_step(ctx, cfg, w, B.Adam(), 1.0)
    assert a["status"] == 0 and c["status"] == 0
    assert np.array_equal(a["metagrad"], b["metagrad"]) and np.array_equal(a["loss_plus"], c["loss_plus"])


@pytest.mark.parametrize("gemm_mode", STEP_MODES)
@pytest.mark.parametrize("dims,batch", [((784, 256, 10), 128), ((40, 200, 72, 24), 257), ((64, 64, 64, 16), 300),
                                        ((33, 17, 12, 6), 7)])
def test_step_without_theta_outputs(dims, batch, gemm_mode):
    """theta_plus and / or theta_minus = NULL: nothing else changes, bit for bit (the tensor-core forward reads
    its own operand copies and the compact bias slab; the fp32 FMA forward and shapes that cannot take the fused
    sweep read scratch copies), and the buffers not asked for are not written."""
    cfg, w = W.custom_mlp(dims, batch, seed=11 + batch)
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, gemm_mode) as ctx:
        full = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        for want_plus, want_minus in [(False, False), (False, True), (True, False)]:
            got = run_step(ctx, cfg, w, B.Adam(), 1e-2, want_plus=want_plus, want_minus=want_minus)
            for k in ("p", "metagrad", "loss_plus", "loss_minus"):
                assert np.array_equal(got[k], full[k]), (k, want_plus, want_minus)
            assert got["eps_fd"] == full["eps_fd"] and got["status"] == 0
            for k, want in (("theta_plus", want_plus), ("theta_minus", want_minus)):
                assert np.array_equal(got[k], full[k]) if want else np.all(np.isnan(got[k]))


@pytest.mark.parametrize("dims,batch", [((784, 256, 10), 128), ((40, 200, 72, 24), 257), ((3072, 1024, 1024, 10), 512),
                                        ((300, 2304, 40), 1200), ((512, 2560, 40), 1280)])
def test_weights_formed_in_the_operand_stage_match_the_presplit_copy(dims, batch):
    """Mode 3 forms hi / lo of theta +- eps_fd p inside the product kernel (theta and p tiles land in shared
    memory and are replaced in place); mode 2 reads the same numbers from the copy the perturbation sweep wrote.
    Same operands, same order of products: every output agrees bit for bit, on single-CTA tiles, clusters that
    split the contraction, CTA pairs with shared tail tiles, and contractions that end inside a k-block (columns
    beyond K read as zero).  A non-finite weight still shows."""
    cfg, w = W.custom_mlp(dims, batch, seed=21 + batch)
    out = {}
    for mode in (2, 3):
        with Ctx(cfg.n_params, cfg.batch, cfg.dims, mode) as ctx:
            out[mode] = run_step(ctx, cfg, w, B.Adam(), 1e-2)
            assert B.sama_last_forward_path(ctx.h) == mode and out[mode]["status"] == 0
            if mode == 3:
                again = run_step(ctx, cfg, w, B.Adam(), 1e-2, want_plus=False, want_minus=False)
                bad = dict(w)
                bad["theta"] = w["theta"].copy()
                bad["theta"][5] = np.nan
                poisoned = run_step(ctx, cfg, bad, B.Adam(), 1e-2)
                # the in-place nudge (theta- written over theta, Sec. 3.2): theta is gone by the time the products
                # run, so this call reads the pre-split copy after all
                t = {k: dev(w[k]) for k in ["theta", "m", "s", "g_base", "g_meta", "X", "y", "lam"]}
                fl = lambda k: torch.empty(k, dtype=torch.float32, device=DEV)
                p_o, mg_o = fl(cfg.n_params), fl(cfg.batch)
                B.sama_step(ctx.h, ctx.mlp, cfg.n_params, t["theta"], t["m"], t["s"], t["g_base"], t["g_meta"], B.Adam(),
                            1e-2, t["X"], t["y"], t["lam"], cfg.batch, p_o, None, t["theta"], mg_o, None, None)
                torch.cuda.synchronize()
                assert B.sama_last_forward_path(ctx.h) == 2
                nudged = {"theta_minus": t["theta"].cpu().numpy(), "metagrad": mg_o.cpu().numpy()}
    for k in ("p", "theta_plus", "theta_minus", "metagrad", "loss_plus", "loss_minus"):
        assert np.array_equal(out[2][k], out[3][k]), k
    for k in ("theta_minus", "metagrad"):
        assert np.array_equal(nudged[k], out[3][k]), k
    for k in ("metagrad", "loss_plus", "loss_minus"):
        assert np.array_equal(again[k], out[3][k]), k
    assert np.isnan(poisoned["loss_plus"]).all() and np.isnan(poisoned["loss_minus"]).all()


def test_two_contexts_keep_their_own_tensor_core_state():
    """The tensor-core path's launch state (shared-memory opt-in, resident CTA pairs, cached tensor maps,
    experiment switches) belongs to a context, not to the process: two contexts for different models, alive at
    once and used alternately, give what each gives alone, and destroying one leaves the other working."""
    cases = [W.custom_mlp((512, 2560, 40), 1280, seed=9), W.custom_mlp((40, 200, 72, 24), 257, seed=5)]
    alone = []
    for cfg, w in cases:
        with Ctx(cfg.n_params, cfg.batch, cfg.dims, 2) as ctx:
            alone.append(run_step(ctx, cfg, w, B.Adam(), 1e-2))
    a = Ctx(cases[0][0].n_params, cases[0][0].batch, cases[0][0].dims, 2)
    b = Ctx(cases[1][0].n_params, cases[1][0].batch, cases[1][0].dims, 2)
    try:
        for _ in range(2):
            for ctx, (cfg, w), ref in ((a, cases[0], alone[0]), (b, cases[1], alone[1])):
                got = run_step(ctx, cfg, w, B.Adam(), 1e-2)
                assert got["status"] == 0 and B.sama_last_forward_path(ctx.h) == 2
                for k in ("p", "metagrad", "loss_plus", "loss_minus"):
                    assert np.array_equal(got[k], ref[k]), k
        a.close()
        got = run_step(b, cases[1][0], cases[1][1], B.Adam(), 1e-2)
        assert np.array_equal(got["metagrad"], alone[1]["metagrad"]) and got["status"] == 0
    finally:
        a.close()
        b.close()


@pytest.mark.parametrize("name", ["tiny", "mlp3072"])
def test_one_launch_sweep_against_two_launches(monkeypatch, name):
    """Small models run adaptation, norm, perturbation and operand split as ONE cooperative launch (a grid-wide
    barrier between the halves); SAMA_NO_FUSED_SWEEP=1 keeps the two launches.  Same p bit for bit; the sum of
    squares is added up over a different grid, so it and what follows agree to rounding, and the status word
    shows no expired wait.  Repeated calls of the one-launch form are bit-identical (its counters return to zero)."""
    cfg = W.CONFIGS[name]
    w = W.mlp_workload(cfg, 0)
    monkeypatch.delenv("SAMA_NO_FUSED_SWEEP", raising=False)   # (the switch is read when a context is created)
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, 2) as ctx:
        a = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        a2 = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        kinds = None
        B.sama_profile_enable(ctx.h, 1)
        run_step(ctx, cfg, w, B.Adam(), 1e-2)
        kinds = [B.KERNEL_KINDS[k] for k, _, _ in B.sama_profile_collect(ctx.h)]
        B.sama_profile_enable(ctx.h, 0)
    assert kinds[0] == "fused_sweep" and "adapt_sumsq" not in kinds
    monkeypatch.setenv("SAMA_NO_FUSED_SWEEP", "1")
    with Ctx(cfg.n_params, cfg.batch, cfg.dims, 2) as ctx:
        b = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        B.sama_profile_enable(ctx.h, 1)
        run_step(ctx, cfg, w, B.Adam(), 1e-2)
        kinds_b = [B.KERNEL_KINDS[k] for k, _, _ in B.sama_profile_collect(ctx.h)]
    assert kinds_b[:2] == ["adapt_sumsq", "perturb_split"]
    assert a["status"] == 0 and b["status"] == 0
    for k in ("p", "theta_plus", "theta_minus", "metagrad", "loss_plus", "loss_minus"):
        assert np.array_equal(a[k], a2[k]), k
    assert a["sumsq"] == a2["sumsq"] and a["eps_fd"] == a2["eps_fd"]
    assert np.array_equal(a["p"], b["p"])
    assert a["sumsq"] == pytest.approx(b["sumsq"], rel=1e-12)
    assert a["eps_fd"] == pytest.approx(b["eps_fd"], rel=1e-6)
    np.testing.assert_allclose(a["theta_plus"], b["theta_plus"], rtol=1e-6, atol=0)
    np.testing.assert_allclose(a["loss_plus"], b["loss_plus"], rtol=1e-5, atol=1e-6)


def test_step_host_matches_step():
    cfg = W.CONFIGS["tiny"]
    w = W.mlp_workload(cfg, 0)
    adam, alpha = B.Adam(), 1e-2
    with Ctx(cfg.n_params, cfg.batch, cfg.dims) as ctx:
        got = run_step(ctx, cfg, w, adam, alpha)
        pin = {k: torch.from_numpy(np.ascontiguousarray(w[k])).pin_memory()
               for k in ["theta", "m", "s", "g_base", "g_meta", "X", "y", "lam"]}
        mg = torch.empty(cfg.batch, dtype=torch.float32).pin_memory()
        eps = torch.empty(1, dtype=torch.float32).pin_memory()
        tm = torch.empty(cfg.n_params, dtype=torch.float32).pin_memory()
        B.sama_step_host(ctx.h, ctx.mlp, cfg.n_params, pin["theta"], pin["m"], pin["s"], pin["g_base"],
                         pin["g_meta"], adam, alpha, pin["X"], pin["y"], pin["lam"], cfg.batch, mg, eps, tm)
        assert np.array_equal(mg.numpy(), got["metagrad"])
        assert float(eps.item()) == got["eps_fd"]
        assert np.array_equal(tm.numpy(), got["theta_minus"])


# ------------------------------------------------ flat vectors, full size ----

@pytest.mark.parametrize("name", ["flat110m", "flat355m"])
def test_flat_vector_full_size(name):
    """adapt + norm + perturb on BERT-base / RoBERTa-large sized vectors, every
    element compared; the checker runs in slices to bound host memory."""
    n = W.FLAT_SIZES[name]
    w = W.flat_vector(n, seed=0)
    alpha = 1.0
    t = {k: dev(w[k]) for k in ["theta", "m", "s", "g_base", "g_meta"]}
    p, tp, tm = (torch.empty(n, dtype=torch.float32, device=DEV) for _ in range(3))
    chunk = 1 << 24
    with Ctx(n) as ctx:
        for step in (1, 1000):
            adam = B.Adam(step=step)
            B.sama_adapt(ctx.h, n, t["m"], t["s"], t["g_base"], t["g_meta"], adam, p, None)
            B.sama_perturb(ctx.h, n, t["theta"], p, B.sama_ctx_sumsq(ctx.h), alpha, tp, tm, None)
            torch.cuda.synchronize()
            assert B.sama_device_status(ctx.h) == 0
            gp, gtp, gtm = p.cpu().numpy(), tp.cpu().numpy(), tm.cpu().numpy()
            refs, total = [], 0.0
            for a in range(0, n, chunk):
                b = min(n, a + chunk)
                rp = oracle.adapt(w["m"][a:b], w["s"][a:b], w["g_base"][a:b], w["g_meta"][a:b], o_adam(adam))
                total += oracle.sumsq(rp)
                refs.append(rp)
            assert read_f64(B.sama_ctx_sumsq(ctx.h)) == pytest.approx(total, rel=2e-6)
            pmax = max(float(np.abs(r).max()) for r in refs)
            worst = 0.0
            eps_ref = None
            for i, a in enumerate(range(0, n, chunk)):
                b = min(n, a + chunk)
                rp = refs[i]
                scale = np.maximum(np.abs(rp), 1e-3 * pmax)
                worst = max(worst, float((np.abs(gp[a:b] - rp) / scale).max()))
                rtp, rtm, eps_ref, bad = oracle.perturb_given_sumsq(w["theta"][a:b], rp, total, alpha)
                assert not bad
                # theta +- eps p can cancel: the rounding is relative to the larger of |result| and |theta|
                th = np.abs(w["theta"][a:b]).astype(np.float64)
                for g_, r_ in ((gtp[a:b], rtp), (gtm[a:b], rtm)):
                    assert float((np.abs(g_ - r_) / np.maximum(np.maximum(np.abs(r_), th), 1e-6)).max()) <= 1e-5
            assert worst <= 1e-5, worst
            assert read_f32(B.sama_ctx_eps_fd(ctx.h)) == pytest.approx(eps_ref, rel=1e-6)
            print("\n[parity] %s step=%d: max rel err p %.3e" % (name, step, worst))


# ---------------------------------------------------------- error paths ----

def test_argument_errors_are_caught_on_the_host():
    n = 64
    cfg, w = W.custom_mlp((8, 4, 3), 5, seed=1)
    with Ctx(n, 5, (8, 4, 3)) as ctx:
        buf = torch.zeros(8 * n, dtype=torch.float32, device=DEV)
        a = [buf[i * n:(i + 1) * n] for i in range(8)]
        adam = B.Adam()

        def status(fn, *args, **kw):
            with pytest.raises(B.SamaError) as e:
                fn(*args, **kw)
            return e.value.status

        assert status(B.sama_adapt, ctx.h, n, None, a[1], None, a[2], adam, a[3]) == B.SAMA_ERR_NULL
        assert status(B.sama_adapt, ctx.h, n, a[0], a[1], None, None, adam, a[3]) == B.SAMA_ERR_NULL
        assert status(B.sama_adapt, ctx.h, -1, a[0], a[1], None, a[2], adam, a[3]) == B.SAMA_ERR_SIZE
        assert status(B.sama_adapt, ctx.h, n + 1, a[0], a[1], None, a[2], adam, a[3]) == B.SAMA_ERR_SIZE
        assert status(B.sama_adapt, ctx.h, n, a[0].data_ptr() + 2, a[1], None, a[2], adam, a[3]) == B.SAMA_ERR_ALIGN
        assert status(B.sama_adapt, ctx.h, n, a[0], a[1], None, a[2], adam, a[0]) == B.SAMA_ERR_OVERLAP
        assert status(B.sama_adapt, ctx.h, n, a[0], a[1], None, a[2], adam, a[2].data_ptr() + 16) == B.SAMA_ERR_OVERLAP
        for bad in (B.Adam(step=0), B.Adam(beta1=1.0), B.Adam(beta2=-0.1), B.Adam(lr=float("nan")),
                    B.Adam(lr=0.0), B.Adam(eps=float("inf")), B.Adam(eps=-1e-8)):
            assert status(B.sama_adapt, ctx.h, n, a[0], a[1], None, a[2], bad, a[3]) == B.SAMA_ERR_PARAM
        # identity mode needs neither moments nor valid Adam scalars
        assert B.sama_adapt(ctx.h, n, None, None, None, a[2], B.Adam(identity=True, lr=float("nan")), a[3]) == 0

        assert status(B.sama_perturb, ctx.h, n, a[0], a[1], None, 0.0, a[2], a[3]) == B.SAMA_ERR_PARAM
        assert status(B.sama_perturb, ctx.h, n, a[0], a[1], None, float("inf"), a[2], a[3]) == B.SAMA_ERR_PARAM
        assert status(B.sama_perturb, ctx.h, n, a[0], a[1], None, 1.0, a[2], a[2]) == B.SAMA_ERR_OVERLAP
        assert status(B.sama_perturb, ctx.h, n, a[0], a[1], None, 1.0, a[0], a[3]) == B.SAMA_ERR_OVERLAP
        assert status(B.sama_perturb, ctx.h, n, a[0], a[1], None, 1.0, a[2], a[1]) == B.SAMA_ERR_OVERLAP
        assert status(B.sama_perturb, ctx.h, n, a[0], None, None, 1.0, a[2], a[3]) == B.SAMA_ERR_NULL

        mlp = ctx.mlp
        X, y, lam = dev(w["X"]), dev(w["y"]), dev(w["lam"])
        mg = torch.zeros(5, dtype=torch.float32, device=DEV)
        eps = torch.ones(1, dtype=torch.float32, device=DEV)
        assert status(B.sama_fd_metagrad, ctx.h, mlp, a[0], a[1], X, y, lam, 0, eps, mg) == B.SAMA_ERR_SIZE
        assert status(B.sama_fd_metagrad, ctx.h, mlp, a[0], a[1], X, y, lam, 6, eps, mg) == B.SAMA_ERR_SIZE
        assert status(B.sama_fd_metagrad, ctx.h, B.MLP((8, 5, 3)), a[0], a[1], X, y, lam, 5, eps, mg) == B.SAMA_ERR_SIZE
        assert status(B.sama_fd_metagrad, ctx.h, B.MLP((8, 4, 4)), a[0], a[1], X, y, lam, 5, eps, mg) == B.SAMA_ERR_SIZE
        assert status(B.sama_fd_metagrad, ctx.h, mlp, a[0], a[1], X, None, lam, 5, eps, mg) == B.SAMA_ERR_NULL
        assert status(B.sama_fd_metagrad, ctx.h, mlp, a[0], a[1], X, y, lam, 5, eps, lam) == B.SAMA_ERR_OVERLAP
        # n must be the model's parameter count
        assert status(B.sama_step, ctx.h, mlp, n, a[0], a[1], a[2], None, a[3], adam, 1.0, X, y, lam, 5,
                      a[4], a[5], a[6], mg) == B.SAMA_ERR_SIZE
        assert B.sama_last_cuda_error(ctx.h) == 0
        assert B.sama_device_status(ctx.h) == 0
    # a context without a model cannot run the forward pass
    with Ctx(n) as ctx:
        assert status(B.sama_fd_metagrad, ctx.h, B.MLP((8, 4, 3)), a[0], a[1], X, y, lam, 5, eps, mg) == B.SAMA_ERR_SIZE


def test_a_bounded_wait_that_runs_out_is_reported_not_hung():
    """The expiry path of the kernels' bounded waits, exercised without any fault: a wait on a barrier nothing
    arrives on, limited to about a millisecond, ends by itself, raises SAMA_DEV_TIMEOUT in the status word, and
    leaves the context and the device usable (a step right after gives the usual result)."""
    cfg = W.CONFIGS["tiny"]
    w = W.mlp_workload(cfg, 0)
    with Ctx(cfg.n_params, cfg.batch, cfg.dims) as ctx:
        before = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        waited = torch.zeros(1, dtype=torch.int64, device=DEV)
        limit = 2_000_000                       # ~1 ms at 2 GHz
        B.sama_selftest_wait_expiry(ctx.h, limit, waited)
        assert B.sama_device_status(ctx.h) == B.SAMA_DEV_TIMEOUT
        assert limit < int(waited.item()) < 50 * limit
        assert B.sama_device_status(ctx.h) == 0          # reading cleared it
        after = run_step(ctx, cfg, w, B.Adam(), 1e-2)
        assert after["status"] == 0 and np.array_equal(after["metagrad"], before["metagrad"])
        with pytest.raises(B.SamaError) as e:
            B.sama_selftest_wait_expiry(ctx.h, 0)
        assert e.value.status == B.SAMA_ERR_PARAM
        with pytest.raises(B.SamaError) as e:
            B.sama_selftest_wait_expiry(ctx.h, 10 ** 12)
        assert e.value.status == B.SAMA_ERR_PARAM
