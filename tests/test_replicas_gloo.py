"""The N > 1 path of the benchmark on CPU: two gloo ranks as child processes.

Ranks are independent replicas (no data-path collective); what they share is
the timing protocol.  This checks the rank-dependent seeding, the barrier, the
max-over-ranks reduction and the aggregate rate."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import json, sys, time
    sys.path.insert(0, %r)
    import numpy as np
    from paper_2310_05674_b200 import replicas, workloads as W
    r = replicas.init(backend="gloo")
    w = W.flat_vector(1000, r.seed)
    r.barrier()
    t = 0.5 + 0.25 * r.rank                     # pretend rank 1 is slower
    out = {"rank": r.rank, "world": r.world, "seed": r.seed,
           "theta0": float(w["theta"][0]),
           "tmax": r.max_over_ranks(t),
           "rate": r.aggregate_rate(10.0, t)}
    r.barrier()
    r.close()
    print("RESULT " + json.dumps(out), flush=True)
""") % ROOT


def test_two_gloo_ranks_share_only_the_timing_protocol(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    res = {}
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        line = [l for l in out.splitlines() if l.startswith("RESULT ")][0]
        d = json.loads(line[7:])
        res[d["rank"]] = d
    assert res[0]["world"] == res[1]["world"] == 2
    assert (res[0]["seed"], res[1]["seed"]) == (0, 1)
    assert res[0]["theta0"] != res[1]["theta0"]           # independent problems
    assert res[0]["tmax"] == res[1]["tmax"] == 0.75        # slowest rank's time on every rank
    assert abs(res[0]["rate"] - 2 * 10.0 / 0.75) < 1e-12   # all ranks' units over that time


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2310_05674_b200 import replicas
    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        r = replicas.init()
        assert (r.rank, r.world, r.backend) == (0, 1, None)
        assert r.max_over_ranks(1.5) == 1.5 and r.aggregate_rate(3.0, 1.5) == 2.0
        r.barrier()
        r.close()
    finally:
        os.environ.update(env)


CHILD_SYNC = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    import oracle
    from paper_2310_05674_b200 import replicas
    r = replicas.init(backend="gloo")
    rng = np.random.default_rng(0)                       # the same batch on both ranks; each takes its rows
    B, H = 24, 5
    lp = np.abs(rng.normal(size=B)) + 0.1
    lm = lp * (1 + 1e-3 * rng.normal(size=B))
    lam = (0.5 * rng.normal(size=3 * H + 1)).astype(np.float32)
    rows = slice(r.rank * B // r.world, (r.rank + 1) * B // r.world)
    local = oracle.fd_reweight(lp[rows], lm[rows], lam, 0.05, B_norm=B)   # the whole batch's normaliser
    t = torch.from_numpy(local.copy())
    r.all_reduce_sum(t)
    full = oracle.fd_reweight(lp, lm, lam, 0.05, B_norm=B)
    m = torch.from_numpy(local.copy())
    r.all_reduce_mean(m)
    out = {"rank": r.rank, "err": float(np.abs(t.numpy() - full).max() / np.abs(full).max()),
           "mean_err": float(np.abs(m.numpy() * r.world - full).max() / np.abs(full).max()),
           "local_differs": bool(np.abs(local - full).max() > 0)}
    r.barrier()
    r.close()
    print("RESULT " + json.dumps(out), flush=True)
""") % ROOT


def test_one_gradient_synchronisation_gives_the_batch_meta_gradient(tmp_path):
    """Sec. 3.3 / Fig. 2 on CPU with two gloo ranks: each rank's central difference over its own rows (normalised
    by the whole batch), summed once over ranks, is the central difference over the whole batch."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "child_sync.py"
    script.write_text(CHILD_SYNC)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        d = json.loads([l for l in out.splitlines() if l.startswith("RESULT ")][0][7:])
        assert d["err"] < 1e-10 and d["mean_err"] < 1e-10 and d["local_differs"]


CHILD_SHARD = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    import oracle
    from paper_2310_05674_b200 import replicas, workloads as W
    r = replicas.init(backend="gloo")
    n, alpha = 100003, 0.37
    w = W.flat_vector(n, 5)                               # the same vector on both ranks; each takes its share
    adam = oracle.Adam(step=7)
    lo, hi = r.shard_range(n)
    p = oracle.adapt(w["m"][lo:hi], w["s"][lo:hi], w["g_base"][lo:hi], w["g_meta"][lo:hi], adam)
    ss = torch.tensor([oracle.sumsq(p)], dtype=torch.float64)
    r.all_reduce_sum(ss)                                  # the one exchange: 8 bytes
    tp, tm, eps, bad = oracle.perturb_given_sumsq(w["theta"][lo:hi], p, float(ss.item()), alpha)
    p_all = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], adam)
    tp_all, tm_all, eps_all, _ = oracle.perturb(w["theta"], p_all, alpha)
    out = {"rank": r.rank, "lo": lo, "hi": hi, "bad": bool(bad),
           "eps_rel": abs(eps - eps_all) / eps_all,
           "same": bool(np.array_equal(p, p_all[lo:hi])),
           "tp_err": float(np.abs(tp - tp_all[lo:hi]).max()), "tm_err": float(np.abs(tm - tm_all[lo:hi]).max())}
    r.barrier()
    r.close()
    print("RESULT " + json.dumps(out), flush=True)
""") % ROOT


def test_sharded_vector_needs_one_eight_byte_exchange(tmp_path):
    """Sec. 3.2's norm is over the whole vector: two gloo ranks adapt their contiguous shares, add their sums of
    squares once, and perturb their shares with the global step size; together that is the unsharded result."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "child_shard.py"
    script.write_text(CHILD_SHARD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    res = {}
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        d = json.loads([l for l in out.splitlines() if l.startswith("RESULT ")][0][7:])
        res[d["rank"]] = d
    assert res[0]["lo"] == 0 and res[0]["hi"] == res[1]["lo"] and res[1]["hi"] == 100003 and res[0]["hi"] % 4 == 0
    for d in res.values():
        assert d["same"] and not d["bad"] and d["eps_rel"] < 1e-12 and d["tp_err"] < 1e-12 and d["tm_err"] < 1e-12
