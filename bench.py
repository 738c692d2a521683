#!/usr/bin/env python
"""Benchmark of the SAMA meta-gradient step (arXiv 2310.05674, Fig. 2 / Eq. 5).

One "step" is one pass of the whole path -- adaptation + norm, perturbation,
dual-branch forward, cross-entropy + central difference -- over one synthetic
batch.  Prints ONE JSON line (rank 0).  The line's headline (value, roofline,
e2e, cpu_baseline) is the largest single-GPU workload, the 4096-wide MLP; with
one GPU the same line also carries, under "workloads", the other MLP workloads
(steps/s, forward fraction of roofline) and the adaptation + perturbation sweep
on the 110 M / 355 M flat vectors (HBM GB/s).  ``--impl reference`` times the
CPU checker on the host cores instead (rank 0 only).

Timing: CUDA events on the launching stream around each step, an L2 flush
between steps outside the events (a write larger than L2, then a read larger
than L2, so that the flush's own dirty lines are written back before the
timed step instead of under its first kernel), W >= 3 warm-ups,
barrier + synchronize on both sides, max over ranks.  ``--steps K`` is
multiplied inside: every one of the K steps is repeated ``inner_reps`` times
(each repetition timed by its own event pair) so that the timed region lasts
about a second and the clock sampler sees it; rates are per single step.
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


KERNEL_SOURCES = {"fused_sweep": ("adapt_perturb.cu",), "adapt_sumsq": ("adapt_perturb.cu",), "perturb": ("adapt_perturb.cu",), "sumsq": ("adapt_perturb.cu",),
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


PRIMARY = "wide4096"
EXTRAS = ["mlp3072", "head1024", "tiny", "flat355m", "flat110m"]


def config_for(name: str, flat_n: int = 0) -> dict:
    """The workload description both arms print (identical dicts)."""
    if name in W.FLAT_SIZES:
        return {"workload": name, "dims": None, "batch": 0, "n_params": int(flat_n or W.FLAT_SIZES[name]),
                "alpha": 1.0, "l2": "flushed between steps (256 MiB written, then 256 MiB read; outside the events)",
                "replicas": "one independent step per rank, no data-path collective"}
    cfg = W.CONFIGS[name]
    return {"workload": name, "dims": list(cfg.dims), "batch": cfg.batch, "n_params": cfg.n_params,
            "alpha": cfg.alpha, "l2": "flushed between steps (256 MiB written, then 256 MiB read; outside the events)",
            "replicas": "one independent step per rank, no data-path collective"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    flat = name in W.FLAT_SIZES
    cfg = None if flat else W.CONFIGS[name]
    w = W.flat_vector(args.flat_n or W.FLAT_SIZES[name], 0) if flat else W.mlp_workload(cfg, 0)
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
           "config": config_for(name, args.flat_n),
           "cpu_baseline": {"value": value, "unit": "steps/s", "cores": 1, "kind": "oracle",
                            "sample": "each step: " + desc},
           "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


class Bench:
    """Shared state of one rank's measurements: device, replica group, peaks, the L2-flush buffer."""

    def __init__(self, args):
        import torch
        from paper_2310_05674_b200 import binding as S
        from paper_2310_05674_b200 import replicas
        self.torch, self.S, self.args = torch, S, args
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        self.dev = "cuda:%d" % self.local
        self.group = replicas.init(backend="nccl", device=self.dev)   # one process per GPU; independent replicas
        self.peaks = load_peaks()
        self.flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=self.dev)
        self.flush_read = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=self.dev)
        self.stream = torch.cuda.current_stream()
        self.sm_count = torch.cuda.get_device_properties(self.local).multi_processor_count

    def flush(self):
        """Cold L2 for the next step: 256 MiB written (evicts everything), then 256 MiB read (the written lines go
        back to HBM now, not under the step's first kernel; what is left in L2 is clean)."""
        self.flush_buf.fill_(1)
        self.flush_read.max()

    def barrier(self):
        self.group.barrier()
        self.torch.cuda.synchronize()

    def tensor_peaks(self):
        """fp32-faithful tensor-core peak: dense TF32 = measured bf16 x 0.5 (nominal ratio), three products per
        fp32 product.  Burst for a kernel timed at full clock, sustained under the board's power cap."""
        p = self.peaks
        return p["bf16_tflops"] * 0.5 / 3.0, p["bf16_tflops_sustained"] * 0.5 / 3.0

    def measure(self, name, w, region_s, with_e2e=False, with_meta=False, flat_n=0):
        """Times one workload: W warm-ups, then K x inner_reps steps, each between its own pair of events."""
        torch, S, args = self.torch, self.S, self.args
        dev, stream, group = self.dev, self.stream, self.group
        flat = name in W.FLAT_SIZES
        cfg = None if flat else W.CONFIGS[name]
        n = w["theta"].size
        mlp = None if flat else S.MLP(cfg.dims)
        B = cfg.batch if cfg else 0
        ctx = S.sama_create(self.local, n, B, mlp)
        if args.gemm_mode:
            S.sama_set_gemm_mode(ctx, args.gemm_mode)
        adam = S.Adam()
        alpha = cfg.alpha if cfg else 1.0
        keys = ["theta", "m", "s", "g_base", "g_meta"] + ([] if flat else ["X", "y", "lam"])
        pin = with_e2e and not flat
        host = {k: torch.from_numpy(np.ascontiguousarray(w[k])) for k in keys}
        if pin:
            host = {k: v.pin_memory() for k, v in host.items()}
        d = {k: host[k].to(dev) for k in keys}
        p, tp, tm = (torch.empty(n, dtype=torch.float32, device=dev) for _ in range(3))
        mg = torch.empty(max(B, 1), dtype=torch.float32, device=dev)
        outputs = {"plus": tp if args.theta_outputs == "both" else None,
                   "minus": tm if args.theta_outputs != "none" else None}
        self.store_theta_pm = args.theta_outputs == "both"

        def one_step():
            if flat:
                S.sama_adapt(ctx, n, d["m"], d["s"], d["g_base"], d["g_meta"], adam, p, None, stream)
                S.sama_perturb(ctx, n, d["theta"], p, S.sama_ctx_sumsq(ctx), alpha, tp, tm, None, stream)
            else:
                S.sama_step(ctx, mlp, n, d["theta"], d["m"], d["s"], d["g_base"], d["g_meta"], adam, alpha, d["X"],
                            d["y"], d["lam"], B, p, outputs["plus"], outputs["minus"], mg, None, None, stream)

        def timed(K):
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
            for a, b in ev:
                self.flush()
                a.record(stream)
                one_step()
                b.record(stream)
            torch.cuda.synchronize()
            return [a.elapsed_time(b) for a, b in ev]

        sampler = ClockSampler(self.local)
        sampler.start()
        for _ in range(args.warmup):
            self.flush()
            one_step()
        torch.cuda.synchronize()
        # inner repetitions: enough for the timed region to last about region_s (every rank takes the same count)
        est_ms = max(group.max_over_ranks(sum(timed(3)) / 3.0, dev), 1e-3)
        reps = int(min(max(1, round(region_s * 1e3 / (est_ms * args.steps))), 4096))
        total_steps = args.steps * reps
        self.barrier()
        l0 = S.sama_launch_count(ctx)
        sampler.active.set()
        t_wall0 = time.perf_counter()
        ms = timed(total_steps)
        self.barrier()
        t_wall = time.perf_counter() - t_wall0
        sampler.active.clear()
        launches = S.sama_launch_count(ctx) - l0
        total_ms = group.max_over_ranks(sum(ms), dev)
        ms_per_step = total_ms / total_steps
        value = group.world * total_steps / (total_ms * 1e-3)
        status = S.sama_device_status(ctx)
        clocks = sampler.summary()

        # ---- per-kernel times (events recorded by the library around each launch, same stream) ----
        S.sama_profile_enable(ctx, True)
        Kp = min(total_steps, 50)
        sampler.active.set()
        timed(Kp)
        sampler.active.clear()
        recs = S.sama_profile_collect(ctx)
        per_kernel = {}
        for kind, layer, t in recs:
            key = S.KERNEL_KINDS.get(kind, str(kind))
            e = per_kernel.setdefault(key, {"ms_per_step": 0.0, "launches_per_step": 0.0, "layers": {}})
            e["ms_per_step"] += t / Kp
            e["launches_per_step"] += 1.0 / Kp
            if layer >= 0:
                e["layers"][layer] = e["layers"].get(layer, 0.0) + t / Kp
        # second pass, grouped: the forward layers of a step between ONE pair of events (an event between two
        # launches serialises them and removes the dependent-launch overlap they have in an untimed step)
        S.sama_profile_enable(ctx, 2)
        sampler.active.set()
        timed(Kp)
        sampler.active.clear()
        grouped = {}
        for kind, layer, t, run_len in S.sama_profile_collect(ctx, with_launches=True):
            key = S.KERNEL_KINDS.get(kind, str(kind))
            e = grouped.setdefault(key, {"ms_per_step": 0.0, "launches_per_step": 0.0})
            e["ms_per_step"] += t / Kp
            e["launches_per_step"] += run_len / Kp
        S.sama_profile_enable(ctx, 0)
        for key, e in grouped.items():
            if key in per_kernel and key.startswith("gemm"):
                per_kernel[key]["ms_per_step_per_launch_events"] = per_kernel[key]["ms_per_step"]
                per_kernel[key]["ms_per_step"] = e["ms_per_step"]
                per_kernel[key]["timing"] = "one event pair around the step's consecutive launches of this kernel"
        dominant = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_step"])
        peaks = self.peaks
        power_capped = "sw_power_cap" in clocks["reasons"] or (
            clocks["sm_mhz"] and clocks["sm_max_mhz"] and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"])

        def launch_s(kernel):
            return per_kernel[kernel]["ms_per_step"] / max(per_kernel[kernel]["launches_per_step"], 1e-9) * 1e-3

        def hbm_roof(kernel, bytes_per_launch, seconds=None, moved=None):
            t = seconds if seconds is not None else launch_s(kernel)
            ach = bytes_per_launch / t / 1e9
            r = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                 "frac_of_nominal_8TBs": ach / 8000.0, "traffic": recorded_traffic(kernel, name),
                 "algorithmic_bytes_per_launch": bytes_per_launch, "launch_us": t * 1e6}
            if moved is not None:   # bytes the kernel moves including the forward's operand preparation (L2 and HBM)
                r["bytes_moved_incl_operand_prep"] = moved
                r["moved_gbs"] = moved / t / 1e9
            return r

        rooflines = {}
        if "adapt_sumsq" in per_kernel:
            rooflines["adapt_sumsq"] = hbm_roof("adapt_sumsq", 20.0 * n)
        if "perturb" in per_kernel:
            rooflines["perturb"] = hbm_roof("perturb", 16.0 * n)
        # Bytes the sweeps move beyond the algorithmic ones: what they also write for the tensor-core forward (hi / lo
        # of W+-: 32 B/element; none in gemm mode 3, where the product kernel forms them) and the split of X;
        # theta+- count only where they are stored.
        stored = {"both": 8.0, "minus": 4.0, "none": 0.0}[args.theta_outputs]
        prep = 0.0 if args.gemm_mode == 3 else 32.0
        x_prep = 12.0 * B * cfg.dims[0] if cfg else 0.0
        if "perturb_split" in per_kernel:
            # the perturbation of Sec. 3.2 is 16 B/element (theta, p in; theta+, theta- out)
            read = 8.0 if (prep or stored) else 0.0   # with nothing to store per weight, the weights are not read
            rooflines["perturb_split"] = hbm_roof("perturb_split", 16.0 * n, moved=(read + stored + prep) * n + x_prep)
        if "fused_sweep" in per_kernel:   # adaptation + norm + perturbation (+ operand split) in one launch
            # reads m, s, g_base, g_meta, theta (p stays in shared memory), writes p
            rooflines["fused_sweep"] = hbm_roof("fused_sweep", 36.0 * n, moved=(28.0 + stored + prep) * n + x_prep)
        sweep = [k for k in ("adapt_sumsq", "perturb", "perturb_split", "sumsq", "fused_sweep") if k in per_kernel]
        if sweep:   # adaptation + norm + perturbation together: 36 B/element over the sum of their launch times
            t = sum(per_kernel[k]["ms_per_step"] for k in sweep) * 1e-3
            rooflines["adapt_perturb"] = hbm_roof("+".join(sweep), 36.0 * n, seconds=t)
        for gk in ("gemm_ffma", "gemm_tf32x3"):
            if gk in per_kernel and cfg:
                flops = float(cfg.forward_flops)
                t = per_kernel[gk]["ms_per_step"] * 1e-3
                ach = flops / t / 1e12
                if gk == "gemm_ffma":
                    mhz = clocks["sm_mhz"] or clocks["sm_max_mhz"] or 1965.0
                    peak = self.sm_count * FMA_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
                    rooflines[gk] = {"bound": "alu", "kernel": gk, "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                                     "frac": ach / peak,
                                     "peak_source": "%d SMs x 128 FMA lanes x 2 x %.0f MHz (median SM clock sampled "
                                                    "during the run)" % (self.sm_count, mhz),
                                     "traffic": recorded_traffic(gk, name), "algorithmic_flops_per_step": flops}
                else:
                    burst, sustained = self.tensor_peaks()
                    peak = sustained if power_capped else burst
                    rooflines[gk] = {"bound": "tensor", "kernel": gk, "achieved": ach, "peak": peak,
                                     "unit": "TFLOP/s", "frac": ach / peak,
                                     "regime": "sustained (power cap or reduced clock seen)" if power_capped
                                               else "burst (full clock, no cap)",
                                     "frac_of_burst_peak": ach / burst, "frac_of_sustained_peak": ach / sustained,
                                     "peak_source": peaks["source"] + " bf16 (burst %.1f / sustained %.1f TFLOP/s) x 0.5 "
                                                    "(nominal tf32:bf16) / 3 products per fp32-faithful product"
                                                    % (peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]),
                                     "traffic": recorded_traffic(gk, name), "algorithmic_flops_per_step": flops,
                                     "launches_per_step": per_kernel[gk]["launches_per_step"]}
        roofline = rooflines.get(dominant) or next(iter(rooflines.values()))

        out = {"value": value, "unit": "steps/s", "ms_per_step": ms_per_step, "steps": args.steps,
               "inner_reps": reps, "timed_steps": total_steps, "config": config_for(name, flat_n),
               "clocks": clocks, "gpu_launches": int(launches), "device_status": int(status),
               "forward_path": {0: "none", 1: "fp32 FMA", 2: "tensor cores, 3xTF32",
                                3: "tensor cores, 3xTF32, weights perturbed in the operand stage"}[S.sama_last_forward_path(ctx)],
               "wall_s_timed_region": t_wall, "roofline": roofline, "rooflines": rooflines, "kernels": per_kernel}
        if flat:
            out["adapt_perturb_gbs"] = 36.0 * n / (ms_per_step * 1e-3) / 1e9

        # ---- the same step for a caller that keeps only what the method hands on: the meta gradient and the nudged
        # base parameters theta- (Sec. 3.2); theta+ is not requested, so the sweep never writes it ----
        if not flat and not args.no_variants:
            outputs["plus"] = None
            Kv = min(total_steps, 200)
            for _ in range(3):
                self.flush()
                one_step()
            msv = sum(timed(Kv)) / Kv
            S.sama_profile_enable(ctx, 1)
            timed(min(Kv, 20))
            pv = {}
            for kind, layer, t in S.sama_profile_collect(ctx):
                key = S.KERNEL_KINDS.get(kind, str(kind))
                pv[key] = pv.get(key, 0.0) + t / min(Kv, 20)
            S.sama_profile_enable(ctx, 0)
            outputs["plus"] = tp if args.theta_outputs == "both" else None
            out["without_theta_plus_output"] = {"value": group.world * 1e3 / group.max_over_ranks(msv, dev), "unit": "steps/s",
                                                "ms_per_step": msv, "steps": Kv, "kernels": pv}

        # ---- the step with a shared reweighting network as the meta learner (Sec. 4.1): same sweeps and forward,
        # plus the reduction of the per-sample differences to the network's gradient ----
        if with_e2e and not flat and not args.no_variants:
            hidden = 100
            lam_r = (0.5 * torch.randn(3 * hidden + 1, generator=torch.Generator().manual_seed(0))).to(dev)
            mg_r = torch.empty(3 * hidden + 1, dtype=torch.float32, device=dev)

            def rw_step():
                S.sama_step_reweight(ctx, mlp, n, d["theta"], d["m"], d["s"], d["g_base"], d["g_meta"], adam, alpha,
                                     d["X"], d["y"], B, hidden, lam_r, p, tp, tm, mg_r, None, None, stream)
            for _ in range(3):
                rw_step()
            Kr = min(total_steps, 100)
            evr = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Kr)]
            for a_, b_ in evr:
                self.flush()
                a_.record(stream)
                rw_step()
                b_.record(stream)
            torch.cuda.synchronize()
            msr = sum(a_.elapsed_time(b_) for a_, b_ in evr) / Kr
            out["shared_reweighting_network"] = {"hidden": hidden, "dim_lambda": 3 * hidden + 1, "ms_per_step": msr,
                                                 "value": group.world * 1e3 / group.max_over_ranks(msr, dev),
                                                 "unit": "steps/s", "steps": Kr}

        # ---- end to end through the host-buffer entry point ----
        if with_e2e and not flat and not args.no_e2e:
            mg_h = torch.empty(B, dtype=torch.float32).pin_memory()
            eps_h = torch.empty(1, dtype=torch.float32).pin_memory()
            Ke = max(3, min(args.steps, 30))

            def host_step():
                S.sama_step_host(ctx, mlp, n, host["theta"], host["m"], host["s"], host["g_base"], host["g_meta"],
                                 adam, alpha, host["X"], host["y"], host["lam"], B, mg_h, eps_h, None, stream)
            for _ in range(3):
                host_step()
            self.barrier()
            t0 = time.perf_counter()
            for _ in range(Ke):
                host_step()
            self.barrier()
            te = group.max_over_ranks(time.perf_counter() - t0, dev)
            h2d = sum(host[k].numel() * host[k].element_size() for k in keys)
            out["e2e"] = {"value": group.world * Ke / te, "unit": "steps/s", "h2d_bytes_per_step": int(h2d),
                          "d2h_bytes_per_step": int(4 * B + 4), "steps": Ke,
                          "note": "sama_step_host: all inputs copied from pinned host memory every step"}
        if with_meta and not flat:
            gm_out = torch.empty(n, dtype=torch.float32, device=dev)
            for _ in range(3):
                S.sama_meta_grad(ctx, mlp, d["theta"], d["X"], d["y"], B, gm_out, None, stream)
            Km = max(3, min(args.steps, 50))
            evm = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Km)]
            for a_, b_ in evm:
                self.flush()
                a_.record(stream)
                S.sama_meta_grad(ctx, mlp, d["theta"], d["X"], d["y"], B, gm_out, None, stream)
                b_.record(stream)
            torch.cuda.synchronize()
            msm = sum(a_.elapsed_time(b_) for a_, b_ in evm) / Km
            flops_m = 1.5 * cfg.forward_flops   # forward + dz W + dz^T h of ONE branch = 3/2 of the dual-branch forward
            if args.gemm_mode == 1:
                mhz = clocks["sm_mhz"] or 1965.0
                peak_m = self.sm_count * FMA_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
                bound_m, src_m = "alu", "%d SMs x 128 FMA lanes x 2 x %.0f MHz" % (self.sm_count, mhz)
            else:
                peak_m = self.tensor_peaks()[1]
                bound_m, src_m = "tensor", peaks["source"] + " sustained bf16 x 0.5 / 3 products per fp32-faithful product"
            ach_m = flops_m / (msm * 1e-3) / 1e12
            out["meta_grad"] = {"ms_per_call": msm, "calls_per_s": 1e3 / msm, "bound": bound_m, "achieved": ach_m,
                                "peak": peak_m, "unit": "TFLOP/s", "frac": ach_m / peak_m, "peak_source": src_m,
                                "note": "algorithmic flops = 3 single-branch matrix products per layer (forward, "
                                        "dz W, dz^T h); time includes the operand split / transpose kernels"}
        sampler.stop_flag.set()
        S.sama_destroy(ctx)
        del d, p, tp, tm, host
        torch.cuda.empty_cache()
        return out

    store_theta_pm = True   # the benchmark asks sama_step for theta+ and theta- (the paper's nudge uses theta-)


def biased_regression_stage(b, seed):
    """Appendix E's study with the meta gradient computed by the library: 100 meta updates at beta = 0.1 on the
    small workload (base level solved in closed form here, with numpy; plain gradient descent on lambda with step
    1 / lambda_max of the update's linear map), reporting cos(g_true, g_SAMA) and ||lambda_t - lambda*||; and the
    time of one SAMA meta-gradient step (direct gradient, adaptation, perturbation, central difference) on
    both sizes.  The figure in the paper prints no numbers, so there is nothing to compare the values with."""
    torch, S, dev, stream = b.torch, b.S, b.dev, b.stream
    out = {}
    for name, cfg in W.BIASREG.items():
        w = W.biased_regression(cfg, seed)
        d, nv = cfg.d, cfg.n_val
        ctx = S.sama_create(b.local, d, 0, None)
        t = {k: torch.from_numpy(np.ascontiguousarray(w[k])).to(dev) for k in ("Xv", "yv")}
        fl = lambda: torch.empty(d, dtype=torch.float32, device=dev)
        g, p, wp, wm, mg = fl(), fl(), fl(), fl(), fl()
        w_dev, lam_dev = fl(), fl()
        sgd = S.Adam(identity=True)

        def step():
            S.sama_biasreg_step(ctx, d, nv, t["Xv"], t["yv"], w_dev, lam_dev, cfg.beta, None, None, None, sgd, 1.0,
                                g, p, wp, wm, mg, stream)
        rec = {"d": d, "n": cfg.n, "n_val": nv, "beta": cfg.beta}
        if d <= 512:
            X, y, Xv, yv = (w[k].astype(np.float64) for k in ("X", "y", "Xv", "yv"))
            H = X.T @ X + cfg.beta * np.eye(d)
            Hi = np.linalg.inv(H)
            A = cfg.beta * Xv @ Hi
            lam_star = np.linalg.solve(A.T @ A, A.T @ (yv - Xv @ (Hi @ (X.T @ y))))
            eta = 1.0 / np.linalg.eigvals(4 * cfg.beta ** 2 * (Xv.T @ Xv) @ Hi).real.max()
            lam = w["lam0"].astype(np.float64)
            cosv, dist = [], []
            for _ in range(cfg.meta_updates):
                w_star = Hi @ (X.T @ y + cfg.beta * lam)
                w_dev.copy_(torch.from_numpy(w_star.astype(np.float32)))
                lam_dev.copy_(torch.from_numpy(lam.astype(np.float32)))
                step()
                torch.cuda.synchronize()
                gs = mg.cpu().numpy().astype(np.float64)
                gt = 2 * cfg.beta * (Hi @ (Xv.T @ (Xv @ w_star - yv)))
                cosv.append(float(gs @ gt / (np.linalg.norm(gs) * np.linalg.norm(gt))))
                dist.append(float(np.linalg.norm(lam - lam_star)))
                lam = lam - eta * gs
            rec["study"] = {"meta_updates": cfg.meta_updates, "cos_first": cosv[0], "cos_min": min(cosv),
                            "cos_last": cosv[-1], "dist_first": dist[0], "dist_last": dist[-1],
                            "dist_monotone": all(y_ < x_ for x_, y_ in zip(dist, dist[1:]))}
        else:
            w_dev.copy_(torch.from_numpy(w["w_true"]))
            lam_dev.copy_(torch.from_numpy(w["lam0"]))
        for _ in range(5):
            step()
        K = 50
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for a_, b_ in ev:
            b.flush()
            a_.record(stream)
            step()
            b_.record(stream)
        torch.cuda.synchronize()
        ms = sum(a_.elapsed_time(b_) for a_, b_ in ev) / K
        rec["ms_per_meta_gradient"] = ms
        rec["direct_grad_gbs"] = 4.0 * d * nv / (ms * 1e-3) / 1e9   # X' read once: the step's algorithmic bytes
        rec["device_status"] = int(S.sama_device_status(ctx))
        S.sama_destroy(ctx)
        out[name] = rec
    return out


def brief(r):
    """What the line keeps of a secondary workload."""
    keep = {k: r[k] for k in ("value", "unit", "ms_per_step", "inner_reps", "timed_steps", "clocks", "forward_path",
                              "device_status", "adapt_perturb_gbs", "without_theta_plus_output") if k in r}
    keep["rooflines"] = r["rooflines"]
    keep["kernels"] = {k: round(v["ms_per_step"], 6) for k, v in r["kernels"].items()}
    keep["gemm_layers_ms"] = {k: v["layers"] for k, v in r["kernels"].items() if k.startswith("gemm")}
    return keep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=PRIMARY, choices=sorted(W.CONFIGS) + sorted(W.FLAT_SIZES))
    ap.add_argument("--gemm-mode", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--theta-outputs", default="both", choices=["both", "minus", "none"],
                    help="which of theta+ / theta- the timed step asks sama_step to store (default both; the "
                         "forward needs neither)")
    ap.add_argument("--no-variants", action="store_true",
                    help="skip the extra passes on the headline workload (theta+ not stored; shared reweighting network)")
    ap.add_argument("--no-extras", action="store_true",
                    help="time only --workload (the other workloads are added by default on one GPU)")
    ap.add_argument("--biasreg-only", action="store_true",
                    help="run only the biased-regression stage (Appendix E) and print its record")
    ap.add_argument("--region-s", type=float, default=1.2, help="target length of the primary timed region")
    ap.add_argument("--flat-n", type=int, default=0, help="override the length of a flat-vector workload")
    ap.add_argument("--meta-grad", action="store_true",
                    help="also time sama_meta_grad (the direct gradient that produces g_meta) on the same batch")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    b = Bench(args)
    world, rank = b.group.world, b.group.rank
    if args.biasreg_only:
        rec = biased_regression_stage(b, b.group.seed)
        if rank == 0:
            print(json.dumps({"biased_regression": rec}), flush=True)
        b.group.close()
        return
    name = args.workload
    flat = name in W.FLAT_SIZES
    seed = b.group.seed  # each rank owns an independent batch / vector: no data-path collective
    cfg = None if flat else W.CONFIGS[name]
    w = W.flat_vector(args.flat_n or W.FLAT_SIZES[name], seed) if flat else W.mlp_workload(cfg, seed)
    r = b.measure(name, w, args.region_s, with_e2e=True, with_meta=args.meta_grad, flat_n=args.flat_n)

    out = {"metric": METRIC if not flat else "adapt+perturb sweeps/sec", "value": r["value"], "unit": "steps/s",
           "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"],
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic"}
    for k in ("inner_reps", "timed_steps", "config", "clocks", "gpu_launches", "device_status", "forward_path",
              "wall_s_timed_region", "roofline", "rooflines", "kernels", "meta_grad", "e2e", "adapt_perturb_gbs",
              "without_theta_plus_output", "shared_reweighting_network"):
        if k in r:
            out[k] = r[k]

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, desc = OracleTimer(name, w, cfg).step_seconds(20.0)
        out["cpu_baseline"] = {"value": 1.0 / sec, "unit": "steps/s", "cores": 1, "kind": "oracle", "sample": desc,
                               "host_cores_available": os.cpu_count()}
    del w

    # ---- the metric's other configurations (one GPU only: the scaling runs time the headline workload) ----
    if world == 1 and not args.no_extras and name == PRIMARY:
        extras = {}
        flat_w = None
        for ex in EXTRAS:
            if ex in W.FLAT_SIZES:
                nx = W.FLAT_SIZES[ex]
                if flat_w is None or flat_w["theta"].size < nx:
                    flat_w = W.flat_vector(nx, seed)
                # the generator is counter-based: a prefix of the longer vector IS the shorter workload
                wx = {k: v[:nx] for k, v in flat_w.items()}
            else:
                wx = W.mlp_workload(W.CONFIGS[ex], seed)
            extras[ex] = brief(b.measure(ex, wx, 0.6))
            del wx
        out["workloads"] = extras
        out["biased_regression"] = biased_regression_stage(b, seed)
        # the metric's three parts in one place
        out["summary"] = {
            "steps_per_s": dict([(PRIMARY, r["value"])] + [(k, v["value"]) for k, v in extras.items()
                                                           if k not in W.FLAT_SIZES]),
            "adapt_perturb_hbm_gbs": {k: v["adapt_perturb_gbs"] for k, v in extras.items() if k in W.FLAT_SIZES},
            "adapt_perturb_frac_of_measured_hbm": {k: v["rooflines"]["adapt_perturb"]["frac"] for k, v in extras.items()
                                                  if k in W.FLAT_SIZES},
            "forward_frac_of_roofline": dict(
                [(PRIMARY, r["rooflines"].get("gemm_tf32x3", r["rooflines"].get("gemm_ffma", {})).get("frac"))] +
                [(k, v["rooflines"].get("gemm_tf32x3", v["rooflines"].get("gemm_ffma", {})).get("frac"))
                 for k, v in extras.items() if k in ("mlp3072", "head1024")])}
    if rank == 0:
        print(json.dumps(out), flush=True)
    b.group.close()


if __name__ == "__main__":
    main()
