#!/usr/bin/env python
"""Benchmark of the SAMA meta-gradient step (arXiv 2310.05674, Fig. 2 / Eq. 5).

One "step" is one pass of the whole path -- adaptation + norm, perturbation,
dual-branch forward, cross-entropy + central difference -- over one synthetic
batch.  Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU
checker on the host cores instead (rank 0 only).

Timing: CUDA events on the launching stream around each step, an L2 flush
(a write larger than L2) between steps outside the events, W >= 3 warm-ups,
barrier + synchronize on both sides, max over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2310_05674_b200 import workloads as W  # noqa: E402

METRIC = "SAMA meta-grad steps/sec"
FALLBACK_HBM_GBS = 6650.0
FMA_LANES_PER_SM = 128


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", 0)),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 0)), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML while the timed regions run (read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_dev_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.active = threading.Event()
        self.stop_flag = threading.Event()
        self.h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = getattr(torch.cuda.get_device_properties(torch_dev_index), "uuid", None)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = int(vis.split(",")[torch_dev_index]) if vis and vis.split(",")[0].isdigit() else torch_dev_index
                self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def run(self):
        if self.h is None:
            return
        nv = self.nv
        while not self.stop_flag.is_set():
            if self.active.is_set():
                try:
                    self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                    try:
                        mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                    except Exception:
                        mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                    for bit, name in self.REASONS.items():
                        if mask & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(0.01)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def source_hash(*names):
    h = hashlib.sha256()
    for n in names:
        h.update(open(os.path.join(ROOT, "paper_2310_05674_b200", "csrc", n), "rb").read())
    return h.hexdigest()[:16]


KERNEL_SOURCES = {"adapt_sumsq": ("adapt_perturb.cu",), "perturb": ("adapt_perturb.cu",), "sumsq": ("adapt_perturb.cu",),
                  "perturb_split": ("adapt_perturb.cu",), "head_ce_fd": ("head_ce_fd.cu",),
                  "gemm_ffma": ("gemm_ffma.cu",), "ce_fd": ("ce_fd.cu",), "gemm_tf32x3": ("gemm_tf32x3.cu",),
                  "split_tf32": ("gemm_tf32x3.cu",)}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu capture, or None if absent or
    if the kernel's source changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    try:
        for rec in json.load(open(path)):
            if rec["kernel"] == kernel and rec["workload"] == workload:
                if rec.get("source_sha") == source_hash(*KERNEL_SOURCES[kernel]):
                    return float(rec["bytes_per_launch"])
    except Exception:
        return None
    return None


class OracleTimer:
    """Times the CPU checker, as it stands, on a bounded sample of the workload:
    the elementwise stages on the first `cnt` of n parameters and the forward +
    finite difference on the first `rows` of B samples, each scaled to the whole
    workload.  theta+- for the forward are prepared once, outside the timing."""

    def __init__(self, name, w, cfg):
        import oracle
        self.o, self.name, self.w, self.cfg = oracle, name, w, cfg
        self.n = w["theta"].size
        self.adam = oracle.Adam(float(np.float32(1e-3)), float(np.float32(0.9)), float(np.float32(0.999)),
                                float(np.float32(1e-8)), 100)
        self.alpha = cfg.alpha if cfg else 1.0
        self.elem_rate = None   # seconds per parameter
        self.row_rate = None    # seconds per sample
        if cfg:
            p = oracle.adapt(w["m"], w["s"], w["g_base"], w["g_meta"], self.adam)
            self.tp, self.tm, self.eps, _ = oracle.perturb(w["theta"], p, self.alpha)

    def elementwise(self, cnt):
        w, o = self.w, self.o
        t0 = time.perf_counter()
        p = o.adapt(w["m"][:cnt], w["s"][:cnt], w["g_base"][:cnt], w["g_meta"][:cnt], self.adam)
        o.perturb(w["theta"][:cnt], p, self.alpha)
        return time.perf_counter() - t0

    def forward(self, rows):
        w, o, cfg = self.w, self.o, self.cfg
        t0 = time.perf_counter()
        lp = o.losses(cfg.dims, self.tp, w["X"][:rows], w["y"][:rows])
        lm = o.losses(cfg.dims, self.tm, w["X"][:rows], w["y"][:rows])
        o.fd(lp, lm, w["lam"][:rows], self.eps, cfg.batch)
        return time.perf_counter() - t0

    def step_seconds(self, budget_s):
        """One sampled step within about budget_s of CPU time -> (seconds for a whole step, description)."""
        n = self.n
        if self.elem_rate is None:
            c0 = min(n, 1 << 16)
            self.elem_rate = self.elementwise(c0) / c0
            if self.cfg:
                self.row_rate = self.forward(1)
        share = budget_s / (2.0 if self.cfg else 1.0)
        cnt = int(max(1, min(n, share / self.elem_rate)))
        t = self.elementwise(cnt) * (n / cnt)
        desc = "adapt+norm+perturb on parameters 0..%d of %d (time x %d/%d)" % (cnt - 1, n, n, cnt)
        if self.cfg:
            B = self.cfg.batch
            rows = int(max(1, min(B, share / self.row_rate)))
            t += self.forward(rows) * (B / rows)
            desc += "; dual forward + FD on samples 0..%d of %d (time x %d/%d)" % (rows - 1, B, B, rows)
        return t, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    flat = name in W.FLAT_SIZES
    cfg = None if flat else W.CONFIGS[name]
    w = W.flat_vector(W.FLAT_SIZES[name], 0) if flat else W.mlp_workload(cfg, 0)
    timer = OracleTimer(name, w, cfg)
    budget = 150.0 / max(1, args.steps + args.warmup)
    times, desc = [], ""
    for i in range(args.warmup + args.steps):
        t, desc = timer.step_seconds(budget)
        if i >= args.warmup:
            times.append(t)
    sec = sum(times) / len(times)
    value = 1.0 / sec
    out = {"impl": "reference", "metric": METRIC if not flat else "adapt+perturb sweeps/sec", "value": value,
           "unit": "steps/s", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": name},
           "cpu_baseline": {"value": value, "unit": "steps/s", "cores": 1, "kind": "oracle",
                            "sample": "each step: " + desc},
           "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp3072", choices=sorted(W.CONFIGS) + sorted(W.FLAT_SIZES))
    ap.add_argument("--gemm-mode", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--flat-n", type=int, default=0, help="override the length of a flat-vector workload")
    ap.add_argument("--meta-grad", action="store_true",
                    help="also time sama_meta_grad (the direct gradient that produces g_meta) on the same batch")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2310_05674_b200 import binding as S
    from paper_2310_05674_b200 import replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    group = replicas.init(backend="nccl", device=dev)   # one process per GPU; independent replicas
    world, rank = group.world, group.rank

    def barrier():
        group.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return group.max_over_ranks(x, dev)

    peaks = load_peaks()
    name = args.workload
    flat = name in W.FLAT_SIZES
    seed = group.seed  # each rank owns an independent batch / vector: no data-path collective
    if flat:
        n = args.flat_n or W.FLAT_SIZES[name]
        w = W.flat_vector(n, seed)
        cfg = None
        ctx = S.sama_create(local, n, 0, None)
        mlp = None
    else:
        cfg = W.CONFIGS[name]
        w = W.mlp_workload(cfg, seed)
        n = cfg.n_params
        mlp = S.MLP(cfg.dims)
        ctx = S.sama_create(local, n, cfg.batch, mlp)
    if args.gemm_mode:
        S.sama_set_gemm_mode(ctx, args.gemm_mode)
    adam = S.Adam()
    alpha = cfg.alpha if cfg else 1.0

    keys = ["theta", "m", "s", "g_base", "g_meta"] + ([] if flat else ["X", "y", "lam"])
    host = {k: torch.from_numpy(np.ascontiguousarray(w[k])).pin_memory() for k in keys}
    d = {k: host[k].to(dev) for k in keys}
    p, tp, tm = (torch.empty(n, dtype=torch.float32, device=dev) for _ in range(3))
    B = cfg.batch if cfg else 0
    mg = torch.empty(max(B, 1), dtype=torch.float32, device=dev)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def one_step():
        if flat:
            S.sama_adapt(ctx, n, d["m"], d["s"], d["g_base"], d["g_meta"], adam, p, None, stream)
            S.sama_perturb(ctx, n, d["theta"], p, S.sama_ctx_sumsq(ctx), alpha, tp, tm, None, stream)
        else:
            S.sama_step(ctx, mlp, n, d["theta"], d["m"], d["s"], d["g_base"], d["g_meta"], adam, alpha, d["X"],
                        d["y"], d["lam"], B, p, tp, tm, mg, None, None, stream)

    def timed(K, profile=False):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for a, b in ev:
            flush_buf.fill_(1)
            a.record(stream)
            one_step()
            b.record(stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    sampler = ClockSampler(local)
    sampler.start()

    for _ in range(args.warmup):
        flush_buf.fill_(1)
        one_step()
    barrier()
    l0 = S.sama_launch_count(ctx)
    sampler.active.set()
    t_wall0 = time.perf_counter()
    ms = timed(args.steps)
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = S.sama_launch_count(ctx) - l0
    total_ms = max_over_ranks(sum(ms))
    ms_per_step = total_ms / args.steps
    value = world * args.steps / (total_ms * 1e-3)
    status = S.sama_device_status(ctx)

    # ---- per-kernel times (events recorded by the library around each launch, same stream) ----
    S.sama_profile_enable(ctx, True)
    Kp = min(args.steps, 50)
    timed(Kp)
    recs = S.sama_profile_collect(ctx)
    S.sama_profile_enable(ctx, False)
    sampler.active.clear()
    per_kernel = {}
    for kind, layer, t in recs:
        key = S.KERNEL_KINDS.get(kind, str(kind))
        e = per_kernel.setdefault(key, {"ms_per_step": 0.0, "launches_per_step": 0.0, "layers": {}})
        e["ms_per_step"] += t / Kp
        e["launches_per_step"] += 1.0 / Kp
        if layer >= 0:
            e["layers"][layer] = e["layers"].get(layer, 0.0) + t / Kp
    dominant = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_step"])
    clocks_mid = sampler.summary()
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count

    def hbm_roof(kernel, bytes_per_launch):
        t = per_kernel[kernel]["ms_per_step"] / max(per_kernel[kernel]["launches_per_step"], 1e-9) * 1e-3
        ach = bytes_per_launch / t / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                "frac_of_nominal_8TBs": ach / 8000.0, "traffic": recorded_traffic(kernel, name),
                "algorithmic_bytes_per_launch": bytes_per_launch}

    rooflines = {}
    if "adapt_sumsq" in per_kernel:
        rooflines["adapt_sumsq"] = hbm_roof("adapt_sumsq", 20.0 * n)
    if "perturb" in per_kernel:
        rooflines["perturb"] = hbm_roof("perturb", 16.0 * n)
    if "perturb_split" in per_kernel:  # perturb + TF32 hi/lo of both branches: 8 read + 8 + 16 written per element
        # ... plus the batch's operand split done by the same sweep: 4 read + 8 written per element of X
        rooflines["perturb_split"] = hbm_roof("perturb_split", 32.0 * n + (12.0 * B * cfg.dims[0] if cfg else 0.0))
    for gk in ("gemm_ffma", "gemm_tf32x3"):
        if gk in per_kernel and cfg:
            flops = float(cfg.forward_flops)
            t = per_kernel[gk]["ms_per_step"] * 1e-3
            ach = flops / t / 1e12
            if gk == "gemm_ffma":
                mhz = clocks_mid["sm_mhz"] or clocks_mid["sm_max_mhz"] or 1965.0
                peak = sm_count * FMA_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
                rooflines[gk] = {"bound": "alu", "kernel": gk, "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                                 "frac": ach / peak,
                                 "peak_source": "%d SMs x 128 FMA lanes x 2 x %.0f MHz (median SM clock sampled "
                                                "during the run)" % (sm_count, mhz),
                                 "traffic": recorded_traffic(gk, name), "algorithmic_flops_per_step": flops}
            else:
                peak = peaks["bf16_tflops_sustained"] * 0.5 / 3.0
                rooflines[gk] = {"bound": "tensor", "kernel": gk, "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                                 "frac": ach / peak,
                                 "peak_source": peaks["source"] + " sustained bf16 x 0.5 (nominal tf32:bf16) / 3 "
                                                "products per fp32-faithful product",
                                 "traffic": recorded_traffic(gk, name), "algorithmic_flops_per_step": flops}
    roofline = rooflines.get(dominant) or next(iter(rooflines.values()))

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not flat and not args.no_e2e:
        mg_h = torch.empty(B, dtype=torch.float32).pin_memory()
        eps_h = torch.empty(1, dtype=torch.float32).pin_memory()
        Ke = max(3, min(args.steps, 30))

        def host_step():
            S.sama_step_host(ctx, mlp, n, host["theta"], host["m"], host["s"], host["g_base"], host["g_meta"], adam,
                             alpha, host["X"], host["y"], host["lam"], B, mg_h, eps_h, None, stream)
        for _ in range(3):
            host_step()
        barrier()
        sampler.active.set()
        t0 = time.perf_counter()
        for _ in range(Ke):
            host_step()
        barrier()
        te = max_over_ranks(time.perf_counter() - t0)
        sampler.active.clear()
        h2d = sum(host[k].numel() * host[k].element_size() for k in keys)
        e2e = {"value": world * Ke / te, "unit": "steps/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(4 * B + 4), "steps": Ke,
               "note": "sama_step_host: all inputs copied from pinned host memory every step"}
    meta = None
    if args.meta_grad and not flat:
        gm_out = torch.empty(n, dtype=torch.float32, device=dev)
        for _ in range(3):
            S.sama_meta_grad(ctx, mlp, d["theta"], d["X"], d["y"], B, gm_out, None, stream)
        Km = max(3, min(args.steps, 50))
        evm = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Km)]
        sampler.active.set()
        for a_, b_ in evm:
            flush_buf.fill_(1)
            a_.record(stream)
            S.sama_meta_grad(ctx, mlp, d["theta"], d["X"], d["y"], B, gm_out, None, stream)
            b_.record(stream)
        torch.cuda.synchronize()
        sampler.active.clear()
        msm = sum(a_.elapsed_time(b_) for a_, b_ in evm) / Km
        flops_m = 1.5 * cfg.forward_flops   # forward + dz W + dz^T h of ONE branch = 3/2 of the dual-branch forward
        if args.gemm_mode == 1:
            mhz = (sampler.summary()["sm_mhz"] or 1965.0)
            peak_m = sm_count * FMA_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
            bound_m, src_m = "alu", "%d SMs x 128 FMA lanes x 2 x %.0f MHz" % (sm_count, mhz)
        else:
            peak_m = peaks["bf16_tflops_sustained"] * 0.5 / 3.0
            bound_m, src_m = "tensor", peaks["source"] + " sustained bf16 x 0.5 / 3 products per fp32-faithful product"
        ach_m = flops_m / (msm * 1e-3) / 1e12
        meta = {"ms_per_call": msm, "calls_per_s": 1e3 / msm, "bound": bound_m, "achieved": ach_m, "peak": peak_m,
                "unit": "TFLOP/s", "frac": ach_m / peak_m, "peak_source": src_m,
                "note": "algorithmic flops = 3 single-branch matrix products per layer (forward, dz W, dz^T h); "
                        "time includes the operand split / transpose kernels"}
    sampler.stop_flag.set()
    clocks = sampler.summary()

    out = {"metric": METRIC if not flat else "adapt+perturb sweeps/sec", "value": value, "unit": "steps/s",
           "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": name, "dims": list(cfg.dims) if cfg else None, "batch": B, "n_params": n,
                      "alpha": alpha, "l2": "flushed between steps (256 MiB write, outside the events)",
                      "replicas": "one independent step per rank, no data-path collective"},
           "clocks": clocks, "gpu_launches": int(launches), "device_status": int(status),
           "wall_s_timed_region": t_wall, "roofline": roofline, "rooflines": rooflines, "kernels": per_kernel}
    if meta:
        out["meta_grad"] = meta
    if e2e:
        out["e2e"] = e2e
    if flat:
        out["adapt_perturb_gbs"] = 36.0 * n / (ms_per_step * 1e-3) / 1e9

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, desc = OracleTimer(name, w, cfg).step_seconds(20.0)
        out["cpu_baseline"] = {"value": 1.0 / sec, "unit": "steps/s", "cores": 1, "kind": "oracle", "sample": desc,
                               "host_cores_available": os.cpu_count()}
    S.sama_destroy(ctx)
    if rank == 0:
        print(json.dumps(out), flush=True)
    group.close()


if __name__ == "__main__":
    main()
