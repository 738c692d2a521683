"""The allocation-free adaptation entry point against the regular one and against the CPU checker.

``sama_adapt_noalloc`` is for callers that are not allowed to call cudaMalloc
(code under a framework allocator that owns the device, plug-ins loaded after
memory pools were frozen): it keeps the reduction scratch in a static device
array instead of a context.  It must give what ``sama_adapt`` gives (and what the CPU
checker gives for Eq. 4 / Appendix C), and a call must leave the device's free memory where it was.  The file
name sorts last so that a run stopping at the first failure has already run
everything else; the test also passes on its own in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_05674_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_noalloc_adapt_matches_context_adapt_twice_in_a_row():
    from paper_2310_05674_b200 import binding as B
    dev = "cuda:0"
    torch.cuda.set_device(0)
    results = []
    # two calls in a row on different data and sizes: the second must not see the first one's leftovers
    for n, seed, adam, use_g in [(1_000_003, 11, B.Adam(), True), (262_145, 12, B.Adam(step=1, lr=5e-3), False)]:
        w = W.flat_vector(n, seed)
        t = {k: torch.from_numpy(w[k]).to(dev) for k in ["m", "s", "g_base", "g_meta"]}
        gb = t["g_base"] if use_g else None
        # every buffer is allocated BEFORE the call under test; the call itself allocates nothing
        p_new = torch.empty(n, dtype=torch.float32, device=dev)
        ss_new = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
        B.sama_adapt_noalloc(n, t["m"], t["s"], gb, t["g_meta"], adam, p_new, ss_new)
        torch.cuda.synchronize()
        # the name's promise: a further call (the set-up of the first one is done) moves no device memory
        free_before = torch.cuda.mem_get_info(0)[0]
        B.sama_adapt_noalloc(n, t["m"], t["s"], gb, t["g_meta"], adam, p_new, ss_new)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(0)[0] == free_before
        # against the CPU checker (same fp32-rounded hyper-parameters as the C ABI receives)
        f = lambda x: float(np.float32(x))
        ref = oracle.adapt(w["m"], w["s"], w["g_base"] if use_g else None, w["g_meta"],
                           oracle.Adam(f(adam.lr), f(adam.beta1), f(adam.beta2), f(adam.eps), adam.step))
        got = p_new.cpu().numpy().astype(np.float64)
        scale = np.maximum(np.abs(ref), 1e-3 * np.abs(ref).max())
        assert float((np.abs(got - ref) / scale).max()) <= 1e-5
        assert float(ss_new.item()) == pytest.approx(oracle.sumsq(ref), rel=2e-6)
        results.append((n, adam, t, gb, p_new, ss_new))
    ctx = B.sama_create(0, max(r[0] for r in results), 0, None)
    try:
        for n, adam, t, gb, p_new, ss_new in results:
            p_ref = torch.empty(n, dtype=torch.float32, device=dev)
            ss_ref = torch.zeros(1, dtype=torch.float64, device=dev)
            B.sama_adapt(ctx, n, t["m"], t["s"], gb, t["g_meta"], adam, p_ref, ss_ref)
            torch.cuda.synchronize()
            a, b = p_new.cpu().numpy().astype(np.float64), p_ref.cpu().numpy().astype(np.float64)
            scale = np.maximum(np.abs(b), 1e-3 * np.abs(b).max())
            assert float((np.abs(a - b) / scale).max()) <= 1e-5
            assert float(ss_new.item()) == pytest.approx(float(ss_ref.item()), rel=1e-6)
            assert float(ss_new.item()) > 0
    finally:
        torch.cuda.synchronize()
        B.sama_destroy(ctx)


def test_noalloc_rejects_sizes_beyond_its_maximum():
    from paper_2310_05674_b200 import binding as B
    x = torch.zeros(16, dtype=torch.float32, device="cuda:0")
    y = torch.zeros(16, dtype=torch.float32, device="cuda:0")
    ss = torch.zeros(1, dtype=torch.float64, device="cuda:0")
    with pytest.raises(B.SamaError) as e:
        B.sama_adapt_noalloc(B.SAMA_NOALLOC_MAX_N + 1, x, x, None, x, B.Adam(), y, ss)
    assert e.value.status == B.SAMA_ERR_SIZE
    with pytest.raises(B.SamaError) as e:
        B.sama_adapt_noalloc(16, x, x, None, x, B.Adam(), y, None)
    assert e.value.status == B.SAMA_ERR_NULL
