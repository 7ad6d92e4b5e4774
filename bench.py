"""Throughput of the G-CADA step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl ours|reference]

A step is one full G-CADA iteration (minibatch draw, dual-point gradients of
all groups, innovation test, lazy aggregation, AMSGrad update, straggler
clock) on the named synthetic workload.  One JSON line is printed by rank 0.

--impl reference times the fp64 CPU oracle on the host cores instead (a
deliberately plain program: its ratio to the CUDA path says nothing about
kernel quality; the roofline fraction does).
"""
import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

METRIC = "G-CADA iterations/sec (all groups)"
UNIT = "it/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant
# kernel, from the ncu capture summarised under profiles/; valid only for the
# kernel source whose digest is recorded with it.
NCU_TRAFFIC = {
    # config: (kernel source file, sha256 of that file at capture time, bytes per launch)
    "cfg3": ("grad_linear.cu", "490f34b4841bad050f5c69bad92b285663cbf92604b2704cac93e813e8f318e1", 522317824),
}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TFLOPS, bf16_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while running."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag, self.max_mhz = index, [], set(), False, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake_slowdown": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.02)

    def sample_once(self):
        """One synchronous sample (so that even a very short timed region has clock data)."""
        if self.nv is None:
            return
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM))
        except Exception:
            pass

    def result(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def _dist_setup(n_gpus, backend="nccl"):
    """One process per GPU (replicas only: no collective on the data path).  Reads RANK / LOCAL_RANK /
    WORLD_SIZE / MASTER_* from the environment; `backend="gloo"` runs the same host logic on CPU."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if backend == "nccl":
        torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return rank, local, world


def _barrier_max(world, value_ms, device):
    """Max over ranks of a per-rank time (the job is as slow as its slowest replica)."""
    import torch
    if world == 1:
        return value_ms
    import torch.distributed as dist
    t = torch.tensor([value_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def _barrier(world):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def aggregate_value(world, steps, ms):
    """Whole-job iterations per second: every rank ran `steps` iterations in at most `ms`."""
    return world * steps / (ms * 1e-3)


def algorithmic_bytes_per_launch(w):
    """Bytes the dominant (gradient) kernel must move per launch: every sampled
    row once (it serves both points) plus its label."""
    rows = (w["M"] // w["M_G"]) * w["batch"]
    esz = 2 if w["compute"] == "bf16" else 4
    return rows * (w["dims"][0] * esz + 4)


def mlp_flops_per_iteration(w):
    """Dense flops of the dual-point forward/backward as specified: per row and
    point 2*n_in*n_out forward, the same for dW, and for dA except at layer 1."""
    dims = w["dims"]
    rows = (w["M"] // w["M_G"]) * w["batch"] * 2
    f = 0
    for l in range(1, len(dims)):
        f += 2 * dims[l - 1] * dims[l] * (3 if l > 1 else 2)
    return rows * f


MIN_REGION_MS = 50.0      # a timed region shorter than this is repeated (own event pair each) and the median kept
SHORT_REPEATS = 7


def time_steps(g, stream, steps, world, dev, sampler=None):
    """Time gcada_step(steps) on the device: barrier + synchronize on both sides, one CUDA-event pair on the
    launching stream, max over ranks.  When the region is short it is repeated SHORT_REPEATS times, each
    repeat being exactly `steps` iterations under its own event pair.  Returns the per-repeat times (ms)."""
    import torch
    times = []
    n_rep = 1
    while len(times) < n_rep:
        _barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.step(steps)
        e1.record(stream)
        if sampler is not None:
            sampler.sample_once()          # work is in flight
        e1.synchronize()
        _barrier(world)
        times.append(_barrier_max(world, e0.elapsed_time(e1), dev))
        if len(times) == 1 and times[0] < MIN_REGION_MS:
            n_rep = SHORT_REPEATS
    return times


def _median(v):
    s = sorted(v)
    return s[len(s) // 2]


def roofline_of(w, name, rule, peaks, ms_step, steps, launches_per_region, ms_grad, ms_grad_b2b, sel_frac, max_mhz):
    """The roofline object of one workload: dominant kernel, algorithmic work per launch, achieved rate."""
    if w["kind"] == "mlp" and w["compute"] == "fp32":
        # plain fp32 FFMA tiles (a 1e-5 tolerance rules out single-pass tensor-core arithmetic):
        # peak = SMs x 128 FMA lanes x 2 flop x max SM clock
        import torch
        flops = mlp_flops_per_iteration(w)
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        peak = sms * 128 * 2 * (max_mhz or 1965) * 1e6 / 1e12
        achieved = flops / (ms_grad * 1e-3) / 1e12 if ms_grad and ms_grad > 0 else None
        return {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None, "traffic": None,
                "kernel": "gradient (all launches of one iteration; latency-bound at this size)",
                "peak_source": "derived: SMs x 128 lanes x 2 x max SM clock", "flops_per_iteration": flops,
                "whole_step_tflops": flops / (ms_step * 1e-3) / 1e12}
    if launches_per_region == 1:
        # narrow model: the whole timed region was ONE launch of the cluster kernel (all iterations inside it)
        bytes_launch = algorithmic_bytes_per_launch(w) * steps
        achieved = bytes_launch / (ms_step * steps * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s",
                "frac": achieved / peaks["hbm"], "traffic": None,
                "kernel": "linear_cluster_kernel (one launch = all %d iterations; latency-bound workload: "
                          "%.0f KB per iteration)" % (steps, algorithmic_bytes_per_launch(w) / 1e3),
                "peak_source": peaks["source"], "duration_ms": ms_step * steps,
                "algorithmic_bytes_per_launch": bytes_launch}
    if w["kind"] != "mlp":
        bytes_launch = algorithmic_bytes_per_launch(w)
        achieved = bytes_launch / (ms_grad_b2b * 1e-3) / 1e9 if ms_grad_b2b and ms_grad_b2b > 0 else None
        traffic = None
        rec = NCU_TRAFFIC.get(name)
        if rec:
            src = os.path.join(ROOT, "paper_2201_04301_b200", "csrc", rec[0])
            if hashlib.sha256(open(src, "rb").read()).hexdigest() == rec[1]:
                traffic = rec[2]
        return {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s",
                "frac": achieved / peaks["hbm"] if achieved else None, "traffic": traffic,
                "kernel": "gradient", "peak_source": peaks["source"],
                "duration_ms": ms_grad_b2b, "duration_how": "200 back-to-back launches, one CUDA-event pair",
                "achieved_from_bracketed_launches": bytes_launch / (ms_grad * 1e-3) / 1e9 if ms_grad and ms_grad > 0 else None,
                "algorithmic_bytes_per_launch": bytes_launch,
                "frac_of_nominal_8TBs": achieved / 8000.0 if achieved else None,
                # the same bytes over the whole timed step (gradient + selection + update kernels)
                "whole_step_gbs": bytes_launch / (ms_step * 1e-3) / 1e9,
                "whole_step_frac": bytes_launch / (ms_step * 1e-3) / 1e9 / peaks["hbm"]}
    # bf16 MLP: the dominant "kernel" is the chain of tensor-core products of one iteration, timed as the
    # graph-replayed step the `value` comes from.  `achieved` counts the flops the kernels ISSUE (the weight
    # gradients of the two points are never formed: the innovation norm comes from Gram products, which is
    # fewer flops than the dual-point forward/backward "as specified"); the as-specified figure is given beside it.
    spec = mlp_flops_per_iteration(w)
    if rule == "ps":     # only the selected groups compute, at theta^k only; no innovation norms
        spec = spec / 2 * sel_frac
        issued = dict(total=spec * 2.0 / 3.0 + mlp_flops_issued(w, sel_frac)["aggregate"])
    else:
        issued = mlp_flops_issued(w, sel_frac)
    achieved = issued["total"] / (ms_step * 1e-3) / 1e12
    grad_issued = issued["total"] - issued.get("aggregate", 0.0)
    grad = grad_issued / (ms_grad * 1e-3) / 1e12 if ms_grad and ms_grad > 0 else None
    return {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
            "frac": achieved / peaks["bf16_sustained"], "traffic": None,
            "kernel": "whole iteration (all tensor-core launches; graph replay)",
            "peak_source": peaks["source"] + " (sustained; the step runs for seconds under the power cap)",
            "frac_of_burst_peak": achieved / peaks["bf16"], "burst_peak": peaks["bf16"],
            "flops_issued_per_iteration": issued,
            "flops_as_specified_per_iteration": spec,
            "as_specified_tflops": spec / (ms_step * 1e-3) / 1e12,
            "as_specified_frac": spec / (ms_step * 1e-3) / 1e12 / peaks["bf16_sustained"],
            "gradient_phase_tflops": grad,
            "gradient_phase_frac": grad / peaks["bf16_sustained"] if grad else None,
            "gradient_phase_how": "issued flops of the gradient phase / event-bracketed gradient kernels (plain launches)"}


def measure(g, w, name, rule, stream, dev, world, local, steps, warmup, peaks, timing_iters=256):
    """Warm up, time gcada_step(steps), then the per-kernel legs; returns the measured part of a bench line."""
    import torch
    from paper_2201_04301_b200 import binding
    g.step(warmup)
    if warmup < 16:
        g.step(16)               # at least one replay of the 16-iteration graph before anything is timed
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    l0 = g.get_launch_count()
    sampler.start()
    times = time_steps(g, stream, steps, world, dev, sampler)
    sampler.stop_flag = True
    sampler.join()
    launches = (g.get_launch_count() - l0) // len(times)
    ms = _median(times)
    n_hist = min(steps, 4096)
    sel_frac = float(g.get_selection_mask(g.get_iteration() - n_hist, n_hist).mean())
    # per-kernel times (plain launches bracketed by events)
    g.set_option(binding.OPT_TIMING, 1)
    g.step(min(steps, timing_iters))
    (ms_grad, ms_sel, ms_upd), n_timed = g.get_kernel_times()
    g.set_option(binding.OPT_TIMING, 0)
    # the dominant kernel alone, back to back, one event pair (no per-launch bracket gaps); each repetition
    # streams the same rows, more than four times the L2 on the wide workload, so nothing is served from cache
    ms_grad_b2b = g.time_gradient(200 if w["kind"] != "mlp" else 5)
    floor_us = g.time_empty_chain(max(16, min(steps, 2048)))
    res = {
        "value": aggregate_value(world, steps, ms), "unit": UNIT, "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps, "ms_per_step_best": min(times) / steps, "timed_repeats": len(times),
        "gpu_launches": int(launches), "selected_fraction": sel_frac, "clocks": sampler.result(),
        "kernel_ms": {"gradient": ms_grad, "select": ms_sel, "update": ms_upd, "timed_iterations": n_timed},
        "latency_floor_us": floor_us, "us_per_step": ms / steps * 1e3,
        "latency_floor_how": "the iteration's launch structure replayed with empty kernels (same graph nodes, "
                             "edges and launch shapes; for the one-cluster kernel: its cluster barrier per iteration)",
    }
    res["roofline"] = roofline_of(w, name, rule, peaks, ms / steps, steps, launches, ms_grad, ms_grad_b2b, sel_frac,
                                  sampler.max_mhz)
    return res


def mlp_flops_issued(w, sel_frac):
    """Tensor-core flops the bf16 path actually issues per iteration: forward and backward-data products of
    both points as specified; the innovation norm from two Gram products per group and layer (rows = both
    points' minibatch rows, the first layer's input is shared) instead of the two weight-gradient products;
    the aggregate of Eq. (3) as one product per layer over the uploading groups' rows (twice: replaced and new
    uploads) or, when half of the groups upload and every 16th iteration, over all groups' rows."""
    dims = w["dims"]
    G = w["M"] // w["M_G"]
    Bp = -(-w["batch"] // 128) * 128
    rows2 = G * w["batch"] * 2
    fwd = sum(2 * dims[l - 1] * dims[l] for l in range(1, len(dims))) * rows2
    bwd = sum(2 * dims[l - 1] * dims[l] for l in range(2, len(dims))) * rows2
    gram = G * sum(2 * ((1 if l == 1 else 2) * Bp) ** 2 * (dims[l] + dims[l - 1]) for l in range(1, len(dims)))
    k_rows = G * Bp if sel_frac >= 0.5 else (15.0 / 16.0) * 2 * sel_frac * G * Bp + (1.0 / 16.0) * G * Bp
    agg = sum(2 * dims[l - 1] * dims[l] for l in range(1, len(dims))) * k_rows
    return {"forward": fwd, "backward_data": bwd, "gram_norm": gram, "aggregate": agg, "total": fwd + bwd + gram + agg}


def run_ours(args):
    import torch
    from paper_2201_04301_b200 import binding
    from paper_2201_04301_b200 import build as _build
    from paper_2201_04301_b200.workloads import make_workload

    rank, local, world = _dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    if rank == 0:
        _build.build()
    _barrier(world)
    binding.load()
    peaks = _peaks()
    t0 = time.time()
    overrides = {}
    if args.workers:
        overrides["M"] = args.workers
    w = make_workload(args.config, device=dev, data_seed=rank, rows=args.rows, **overrides)
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize()
    opts = {binding.OPT_GRAPH: 0.0 if args.no_graph else 1.0}
    smooth = None
    if args.rule == "ps":      # Eq. (9) as printed, with one smoothness constant for every group
        opts[binding.OPT_RULE] = 1.0
        smooth = [args.smoothness] * (w["M"] // w["M_G"])
    g = binding.from_workload(w, stream=stream, options=opts, smoothness=smooth)
    gen_s = time.time() - t0
    G = g.G

    # --- device-resident timing ------------------------------------------------
    m = measure(g, w, args.config, args.rule, stream, dev, world, local, args.steps, args.warmup, peaks)

    # --- end to end: minibatches fed from pinned host memory, theta read back ----
    e2e = None
    if not args.no_e2e:
        rows = G * w["batch"]
        d = w["dims"][0]
        n_g = w["X"].shape[0] // G
        idx = torch.cat([torch.randint(0, n_g, (w["batch"],), device=dev) + gi * n_g for gi in range(G)])
        Xb = w["X"].index_select(0, idx)[:, :d].contiguous().cpu().pin_memory()
        yb = w["y"].index_select(0, idx).contiguous().cpu().pin_memory()
        h = binding.GCada(w["kind"], w["dims"], w["M"], w["M_G"], w["D"], w["c"], w["alpha"], w["beta1"],
                          w["beta2"], w["eps"], compute=w["compute"], stream=stream)
        h.set_batch(w["batch"])
        h.set_theta(w["theta0"])
        n_e2e = max(3, min(args.steps, args.e2e_steps))
        theta_host = torch.empty(g.p, dtype=torch.float32).pin_memory()   # the step's result lands here
        for _ in range(3):
            h.step_host_batch(Xb, yb)
            h.get_theta(out=theta_host)
        _barrier(world)
        t_a = time.perf_counter()
        for _ in range(n_e2e):
            h.step_host_batch(Xb, yb)
            h.get_theta(out=theta_host)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t_a
        _barrier(world)
        dt = _barrier_max(world, dt * 1e3, dev) * 1e-3
        e2e = {"value": world * n_e2e / dt, "unit": UNIT, "steps": n_e2e,
               "h2d_bytes_per_step": int(Xb.numel() * Xb.element_size() + yb.numel() * yb.element_size()),
               "d2h_bytes_per_step": int(g.p * 4 + 64)}
        h.close()

    if rank != 0:
        return
    out = {
        "metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w["compute"] == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": "%s: %s dims=%s N=%d M=%d M_G=%d batch=%d D=%d c=%g rule=%s" % (
            args.config, w["kind"], list(w["dims"]), w["X"].shape[0], w["M"], w["M_G"], w["batch"], w["D"], w["c"],
            args.rule),
            "parallelism": "replicas only (%d)" % world,
            "l2": "inputs larger than L2: each step gathers its rows from the resident training set"
                  if w["X"].numel() * w["X"].element_size() > 126e6 else "training set smaller than L2 (latency-bound workload)",
            "setup_s": round(gen_s, 1)},
    }
    for key in ("ms_per_step_best", "timed_repeats", "clocks", "gpu_launches", "selected_fraction", "kernel_ms",
                "latency_floor_us", "latency_floor_how", "roofline"):
        out[key] = m[key]
    if e2e:
        out["e2e"] = e2e
    if world == 1 and not (args.no_others or args.no_e2e or args.no_cpu):   # any --no-* switch: a short / profiling run
        # the remaining workloads of the statement, each for its own number of iterations (device-resident,
        # same protocol); parity cases elsewhere, here so that every workload's rate and roofline are on record
        g.close()
        del g, w
        torch.cuda.empty_cache()
        out["other_workloads"] = other_workloads(args.config, dev, stream, local, peaks)
    if world == 1 and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline_both(args.config, budget_s=args.cpu_budget)
    print(json.dumps(out), flush=True)


def other_workloads(skip, dev, stream, local, peaks):
    """Every other named workload, timed like the main one, each with its own roofline, clocks and latency floor."""
    import torch
    from paper_2201_04301_b200 import binding
    from paper_2201_04301_b200.workloads import CONFIGS, make_workload
    res = {}
    for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5"):
        if name == skip:
            continue
        w = make_workload(name, device=dev)
        g = binding.from_workload(w, stream=stream, options={binding.OPT_GRAPH: 1.0})
        K = int(CONFIGS[name]["K"])
        m = measure(g, w, name, "innov", stream, dev, 1, local, K, max(3, min(20, K // 10)), peaks,
                    timing_iters=64 if name == "cfg5" else 256)
        m["dtype"] = "bf16" if w["compute"] == "bf16" else "f32"
        res[name] = m
        g.close()
        del g, w
        torch.cuda.empty_cache()
    return res


# ------------------------------------------------------------------------------
# CPU oracle timing
# ------------------------------------------------------------------------------
def _oracle_workload(config, shard_rows):
    """The named workload with every shard cut to `shard_rows` rows (same model,
    groups, batch): what one oracle iteration costs does not depend on the shard size."""
    from paper_2201_04301_b200.workloads import CONFIGS, make_workload
    from parity import make_oracle
    G = CONFIGS[config]["M"] // CONFIGS[config]["M_G"]
    n_full = CONFIGS[config]["N"]
    rows = min(n_full, G * shard_rows)
    w = make_workload(config, device="cpu", rows=rows)
    return w, make_oracle(w), G


def _cores_used():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def _time_groups(o, n_groups):
    """Time the dual-point gradients of `n_groups` groups plus the server update:
    n_groups / G of one oracle iteration."""
    import numpy as np
    t0 = time.perf_counter()
    theta_k = o.thetas[o.k]
    for g in range(n_groups):
        _, Xb, yb = o.minibatch(g)
        old = o.theta_at(o.k - int(o.tau[g]))
        a = o.model.grad(theta_k, Xb, yb, o.reduction)
        b = o.model.grad(old, Xb, yb, o.reduction)
        d = a - b
        float(d @ d)
    return time.perf_counter() - t0


def cpu_baseline(config, budget_s=15.0):
    from paper_2201_04301_b200.workloads import CONFIGS
    c = CONFIGS[config]
    G = c["M"] // c["M_G"]
    heavy = c["kind"] == "mlp" and c["compute"] == "bf16"
    w, o, G = _oracle_workload(config, shard_rows=max(c["batch"], 256) if heavy else max(c["batch"] * 2, 1024))
    t_one = _time_groups(o, 1)                       # calibration
    if t_one * G <= budget_s / 3:
        n = max(1, int(budget_s / (t_one * G)))
        n = min(n, 200)
        t0 = time.perf_counter()
        for _ in range(n):
            o.step()
        dt = time.perf_counter() - t0
        value, sample = n / dt, "%d full oracle iterations, shards cut to %d rows" % (n, w["X"].shape[0] // G)
    else:
        ng = max(1, min(G, int(budget_s / t_one)))
        dt = _time_groups(o, ng)
        value = 1.0 / (dt * G / ng)
        sample = "dual-point gradients of %d of %d groups, extrapolated to a full iteration" % (ng, G)
    return {"value": value, "unit": UNIT, "cores": _cores_used(), "kind": "oracle", "sample": sample}


def cpu_baseline_both(config, budget_s=15.0):
    """The oracle on the BLAS thread pool as it comes, and again held to one thread."""
    res = cpu_baseline(config, budget_s)
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            one = cpu_baseline(config, budget_s / 2)
        res["one_thread"] = {"value": one["value"], "unit": UNIT, "cores": 1, "sample": one["sample"]}
    except Exception as exc:       # no threadpoolctl: the pool figure stands alone
        res["one_thread"] = {"unavailable": repr(exc)}
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2201_04301_b200.workloads import CONFIGS
    c = CONFIGS[args.config]
    G = c["M"] // c["M_G"]
    w, o, G = _oracle_workload(args.config, shard_rows=max(c["batch"], 256))
    total_budget = 150.0
    per_step = total_budget / (args.steps + args.warmup)
    t_one = _time_groups(o, 1)
    ng = max(1, min(G, int(per_step / t_one)))
    full = ng == G
    for _ in range(args.warmup):
        o.step() if full else _time_groups(o, ng)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.step() if full else _time_groups(o, ng)
    dt = time.perf_counter() - t0
    step_s = dt / args.steps
    value = 1.0 / (step_s * G / ng)
    sample = ("full oracle iterations" if full else
              "each step = dual-point gradients of %d of %d groups, scaled to a full iteration" % (ng, G))
    sample += ", shards cut to %d rows" % (w["X"].shape[0] // G)
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3 * G / ng,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (CPU oracle, fp64 numpy)" % args.config},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": _cores_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=None, help="cut the training set to this many rows")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-others", action="store_true",
                    help="do not time the other named workloads after the main one (1 GPU; a few seconds)")
    ap.add_argument("--no-graph", action="store_true", help="plain launches instead of graph replay")
    ap.add_argument("--workers", type=int, default=None, help="override M (fewer groups, for profiling captures)")
    ap.add_argument("--rule", default="innov", choices=["innov", "ps"],
                    help="innov: measured gradient innovation (default); ps: left side of Eq. (9) as printed")
    ap.add_argument("--smoothness", type=float, default=0.25, help="L_g of every group for --rule ps")
    ap.add_argument("--e2e-steps", type=int, default=60)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 20
        args.warmup = args.warmup if args.warmup is not None else 3
        run_reference(args)
    else:
        args.steps = args.steps if args.steps is not None else 10000
        args.warmup = max(3, args.warmup if args.warmup is not None else 50)
        run_ours(args)


if __name__ == "__main__":
    main()
