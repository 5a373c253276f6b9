#!/usr/bin/env python
"""Benchmark of the deflated polar filter on synthetic GPT-2-XL-shaped Muon batches.

One step = one pass of the whole hot path (batched randomized SVD, deflate + normalise, five quintic
Newton-Schulz steps, restore) over one batch: 48 matrices 1600x6400 and 48 matrices 1600x1600 in
bf16 with the heavy-tailed spectrum sigma_i = max(200/i, 1e-4), k=32, oversampling 16, 2 subspace
iterations. Prints ONE JSON line (the keys are described in README.md).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--small] [--no-extras]

`value` counts the flops the method needs (symmetric products once when the symmetric tiles are on); the
dense-equivalent figure is a separate key. Besides the timed K steps the run reports a sustained leg (the step
repeated for at least 3 s, with its clock record), and under `extras` the other workloads: the GPT-2-small and
medium/large shape batches, the XL batch with the per-step minimax schedule and with the additive restore, and
the 20-call SDP projection sequence at n = 4096 with its stage split.

N > 1: every rank runs the same batch on its own GPU (independent matrices, no data-path collective) and the line
reports the whole-job aggregate; without an outer torchrun the script starts its N ranks itself.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "deflated polar-filter TFLOP/s & matrices/s per batch; % bf16 tensor peak"
MUON = (3.4445, -4.7750, 2.0315)
CLASSICAL = (1.875, -1.25, 0.375)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
_MINIMAX = {}

# name: shape groups (b, m, n), k, p, J, L, schedule, gamma, input recipe
WORKLOADS = {
    "gpt2_xl": {"groups": [(48, 1600, 6400), (48, 1600, 1600)], "k": 32, "p": 16, "J": 2, "L": 5, "schedule": "muon",
                "gamma": 1.01, "workload": 4, "recipe": ("power", 1.0, 200.0, 1e-4),
                "label": "GPT-2-XL Muon shapes, bf16: 48 x 1600x6400 + 48 x 1600x1600, sigma_i=max(200/i,1e-4), "
                         "k=32, p=16, J=2, 5 Muon quintic steps"},
    "gpt2_small": {"groups": [(12, 768, 768), (12, 768, 3072)], "k": 8, "p": 8, "J": 1, "L": 5, "schedule": "muon",
                   "gamma": 1.01, "workload": 2, "recipe": ("spiked",),
                   "label": "GPT-2-small Muon shapes, bf16: 12 x 768x768 + 12 x 768x3072, N(0,1) bulk + 8 spikes, "
                            "k=8, p=8, J=1, 5 Muon quintic steps"},
    "gpt2_medium_large": {"groups": [(24, 1024, 1024), (24, 1024, 3072), (24, 1024, 4096)], "k": 16, "p": 8, "J": 1,
                          "L": 5, "schedule": "minimax", "gamma": 1.1, "workload": 3, "recipe": ("power", 0.8, 50.0, 0.0),
                          "label": "GPT-2-medium/large Muon shapes, bf16: 24 x 1024x{1024,3072,4096}, sigma_i=50 i^-0.8, "
                                   "k=16, p=8, J=1, 5 per-step minimax quintic steps (Polar-Express-style)"},
    "small": {"groups": [(4, 256, 1024), (4, 256, 256)], "k": 8, "p": 8, "J": 1, "L": 5, "schedule": "muon",
              "gamma": 1.01, "workload": 4, "recipe": ("power", 1.0, 200.0, 1e-4),
              "label": "small check: 4 x 256x1024 + 4 x 256x256"},
}


def schedule_of(name, L):
    """[L][3] coefficients: Muon's quintic repeated, or per-step minimax quintics built by greedy Remez exchange from
    [1e-3, 1] (first step rescaled by 1.01): the Polar-Express-style mapping. Same products per step either way."""
    if name == "muon":
        return [list(MUON)] * L
    if L not in _MINIMAX:
        from paper_2609_21102_b200 import schedules
        _MINIMAX[L] = [list(c) for c in schedules.remez_sign_schedule(1e-3, L, margin=0.01)[0]]
    return _MINIMAX[L]


def filter_passes(m, n, sched, iterates=0):
    """How the library walks the filter steps of a bf16 batch of this shape: a list of 1s and 2s, one entry per pass
    over X (2 = two steps in one pass: A_{t+1} = B_t^2 A_t on the short side, X <- (B_{t+1} B_t) X). Greedily from the
    first step, a pair starts at step t when there is a next step, |a_t| <= 4.5 and |b_{t+1} + 2 c_{t+1}| <= 1, provided the long side is at least
    twice the short one (`iterates` = 1, bf16 throughout, pairs nothing)."""
    ms, ml = min(m, n), max(m, n)
    L = len(sched)
    if ml < 2 * ms or iterates == 1 or os.environ.get("DEFL_NO_PAIRED_STEPS"):
        return [1] * L
    out, t = [], 0
    while t < L:
        two = t + 1 < L and abs(sched[t][0]) <= 4.5 and abs(sched[t + 1][1] + 2.0 * sched[t + 1][2]) <= 1.0
        out.append(2 if two else 1)
        t += 2 if two else 1
    return out


def algorithmic_flops(m, n, k, p, J, L, symmetric, add_restore=False, passes=None):
    """Flops the method needs for one matrix: (filter, front end). Filter per single step: the Gram matrix and its
    square (each counted once per symmetric pair when the symmetric tiles are on, else in full) and the apply product;
    per paired step (see filter_passes): one Gram and one apply product and five short-side products; front end: the
    (2 + 2J) products of the randomized SVD with the l-column panel, the rank-k subtraction and, with the additive
    restore, the rank-k add. `passes` None = one pass per step (the per-step count)."""
    ms, ml = min(m, n), max(m, n)
    l = min(ms, k + p) if k > 0 else 0
    big_g, big_a = (ms * (ms + 1.0) * ml, 2.0 * ms * ms * ml) if symmetric else (2.0 * ms * ms * ml, 2.0 * ms * ms * ml)
    small = ms * ms * (ms + 1.0) if symmetric else 2.0 * ms ** 3
    filt = sum(big_g + big_a + (small if q == 1 else 5.0 * small) for q in (passes if passes is not None else [1] * L))
    front = (2.0 * ml * ms * l * (2 + 2 * J) + 2.0 * m * n * k * (2 if add_restore else 1)) if k > 0 else 0.0
    return filt, front


def dense_filter_flops(m, n, L):
    ms, ml = min(m, n), max(m, n)
    return L * (4.0 * ms * ms * ml + 2.0 * ms ** 3)


# Average DRAM bytes per filter-product launch: dram__bytes_read + dram__bytes_write of the 32 filter launches of one
# step (two paired steps and a single one on the wide group, five single steps on the square one) from the ncu capture
# summarised in the filter-kernel summary under profiles/ (8 matrices per group: 100.3 MB on average), scaled by 48/8.
FILTER_TRAFFIC_BYTES_PER_LAUNCH = 602e6


def max_over_ranks(value, dist=None, device="cpu"):
    """Largest `value` over all ranks (a time: the job is as slow as its slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank, world, ms_max):
    """Whole-job rate when every rank processes `units_per_rank` in `ms_max` milliseconds (weak scaling)."""
    return world * units_per_rank / (ms_max * 1e-3)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """SM clock, power and throttle reasons of one GPU while a timed region runs: NVML polled every 10 ms from a
    thread (read-only queries), nvidia-smi in loop mode as the fallback. Regions are cut out afterwards by time."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, index):
        self.index, self.rows, self._stop, self._t, self._p, self.max_mhz = index, [], False, None, None, None

    def _nvml(self):
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop:
            try:
                self.rows.append((time.time(), float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)),
                                  pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0, int(reasons(h))))
            except Exception:
                pass
            time.sleep(0.01)

    def _smi(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        self._p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q, "--format=csv,noheader,nounits",
                                    "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
        for line in self._p.stdout:
            parts = [x.strip() for x in line.strip().split(",")]
            if len(parts) >= 7 and parts[0].replace(".", "").isdigit():
                mask = sum(bit for (nm, bit), v in zip(self.REASONS, parts[3:7]) if v.lower().startswith("active"))
                self.max_mhz = float(parts[1])
                self.rows.append((time.time(), float(parts[0]), float(parts[2]) if parts[2].replace(".", "").isdigit() else 0.0, mask))

    def __enter__(self):
        try:
            import pynvml  # noqa: F401
            target = self._nvml
        except Exception:
            target = self._smi
        self._t = threading.Thread(target=target, daemon=True)
        self._t.start()
        time.sleep(0.2)
        return self

    def __exit__(self, *a):
        self._stop = True
        if self._p is not None:
            self._p.terminate()          # the one process this object started
            try:
                self._p.wait(timeout=5)
            except Exception:
                self._p.kill()
        self._t.join(timeout=5)

    def summary(self, t0, t1):
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows and self.rows:      # a region shorter than the period: the nearest sample
            mid = 0.5 * (t0 + t1)
            rows = [min(self.rows, key=lambda r: abs(r[0] - mid))]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unsampled"], "samples": 0}
        sm = sorted(r[1] for r in rows)
        pw = sorted(r[2] for r in rows)
        mask = 0
        for r in rows:
            mask |= r[3]
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": self.max_mhz,
                "power_w": pw[len(pw) // 2], "reasons": [nm for nm, bit in self.REASONS if mask & bit], "samples": len(rows)}


def make_inputs(wl, device):
    import torch
    from paper_2609_21102_b200 import inputs
    groups = []
    for si, (b, m, n) in enumerate(wl["groups"]):
        if wl["recipe"][0] == "spiked":
            G = inputs.workload_spiked(b, m, n, si, device=device)
        else:
            _, expo, top, floor = wl["recipe"]
            G = inputs.workload_power_law(b, m, n, wl["workload"], si, expo, top, floor, device=device)
        G = G.to(torch.bfloat16)
        l = min(min(m, n), wl["k"] + wl["p"])
        Om = inputs.sketch(b, min(m, n), l, wl["workload"], si, device=device)
        groups.append({"G": G, "Om": Om, "out": torch.empty_like(G)})
    return groups


def run_step(ctx, wl, groups, opts, lanes=None):
    """One step = every shape group through defl_polar_batched. With `lanes` (one (context, stream) pair per
    group) the independent groups are enqueued on their own streams, forked from and joined to the current stream."""
    import torch
    sched = schedule_of(wl["schedule"], wl["L"])
    kw = dict(gamma=wl["gamma"], exploit_symmetry=opts["sym"], bf16_iterates=opts["iterates"], restore_mode=opts["mode"])
    if not lanes:
        for g in groups:
            ctx.defl_polar_batched(g["G"], wl["k"], wl["p"], wl["J"], sched, out=g["out"], sketch=g["Om"], **kw)
        return
    main = torch.cuda.current_stream()
    fork = torch.cuda.Event()
    fork.record(main)
    for g, (c, s) in zip(groups, lanes):
        s.wait_event(fork)
        with torch.cuda.stream(s):
            c.defl_polar_batched(g["G"], wl["k"], wl["p"], wl["J"], sched, out=g["out"], sketch=g["Om"], **kw)
            done = torch.cuda.Event()
            done.record(s)
        main.wait_event(done)


def time_steps(fn, steps, sync):
    """ms per step of `steps` back-to-back calls of fn, by CUDA events on the current stream."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync()
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    sync()
    return e0.elapsed_time(e1) / steps


def workload_flops(wl, sym, add=False, iterates=0, per_step=False):
    """(filter, front end) flops of one batch as the library evaluates it (paired steps where it pairs them), or with
    `per_step` the count of one pass over X per step."""
    filt = front = 0.0
    for b, m, n in wl["groups"]:
        passes = None if per_step else filter_passes(m, n, schedule_of(wl["schedule"], wl["L"]), iterates)
        f, fr = algorithmic_flops(m, n, wl["k"], wl["p"], wl["J"], wl["L"], sym, add, passes)
        filt += b * f
        front += b * fr
    return filt, front


def filter_launches(wl, add=False, iterates=0):
    """Product launches of the filter stage per batch: three per single step, seven per paired step."""
    sched = schedule_of(wl["schedule"], wl["L"])
    return sum(sum(3 if q == 1 else 7 for q in filter_passes(m, n, sched, iterates)) for _, m, n in wl["groups"])


def oracle_sample(wl):
    """Times the fp64 oracle, as it stands, on ONE matrix of EACH shape group of the workload (a bounded sample);
    returns (seconds per group sample, flops per group sample, description)."""
    import oracle
    import torch
    from paper_2609_21102_b200 import inputs
    secs, fl = [], []
    sched = oracle.schedule(schedule_of(wl["schedule"], wl["L"]))
    for si, (b, m, n) in enumerate(wl["groups"]):
        _, expo, top, floor = wl["recipe"]
        G = inputs.workload_power_law(1, m, n, wl["workload"], si, expo, top, floor).to(torch.bfloat16).double().numpy()[0]
        l = min(min(m, n), wl["k"] + wl["p"])
        Om = inputs.sketch(1, min(m, n), l, wl["workload"], si).double().numpy()[0]
        t0 = time.perf_counter()
        oracle.deflated_polar(G, wl["k"], l, Om, wl["J"], sched, gamma=wl["gamma"])
        secs.append(time.perf_counter() - t0)
        # the oracle evaluates every product in full (no symmetric shortcut)
        fl.append(sum(algorithmic_flops(m, n, wl["k"], wl["p"], wl["J"], wl["L"], False)))
    what = " + ".join("1 of %d matrices %dx%d" % g for g in wl["groups"])
    return secs, fl, what + ", full path, fp64"


def reference_arm(args, wl, config):
    """The oracle as the reference arm: each step runs it on one matrix of each shape group."""
    cores = os.cpu_count() or 1
    for _ in range(max(0, args.warmup)):
        oracle_sample(wl)
    times, fl, sample = [], None, ""
    for _ in range(max(1, args.steps)):
        secs, fl, sample = oracle_sample(wl)
        times.append(sum(secs))
    dt = sum(times) / len(times)
    val = sum(fl) / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": len(times), "warmup": max(0, args.warmup), "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "matrices_per_s": len(wl["groups"]) / dt,
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def measure_tf32_peak():
    """Dense tf32 product rate of this GPU the way the bf16 peak was taken: torch.matmul 8192^3 with tf32 allowed,
    best of 10 (the denominator of the SDP filter's roofline fraction; a library product, outside every timed path)."""
    import torch
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        a = torch.randn((8192, 8192), device="cuda")
        b = torch.randn((8192, 8192), device="cuda")
        for _ in range(3):
            torch.matmul(a, b)
        best = 1e9
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch.matmul(a, b)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2.0 * 8192 ** 3 / (best * 1e-3) / 1e12
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev


def extra_polar(ctx, name, opts, device, steps=10, label=None, graph=False):
    """ms per batch, TFLOP/s (flops the method needs), matrices/s and launches of one more workload."""
    import torch
    wl = WORKLOADS[name]
    groups = make_inputs(wl, device)
    for _ in range(3):
        run_step(ctx, wl, groups, opts)
    l0 = ctx.defl_launch_count()
    ms = time_steps(lambda: run_step(ctx, wl, groups, opts), steps, torch.cuda.synchronize)
    launches = (ctx.defl_launch_count() - l0) // steps
    st = ctx.defl_get_stage_ms(min(64, steps * len(groups)))
    per = min(64, steps * len(groups)) / len(groups)
    filt, front = workload_flops(wl, opts["sym"], opts["mode"] == 1, opts["iterates"], per_step=True)     # algorithmic
    filt_exec, _ = workload_flops(wl, opts["sym"], opts["mode"] == 1, opts["iterates"])
    graph_ms = None
    if graph:
        # the launch-bound small batches replayed from a CUDA graph: every call of the library only enqueues work on its
        # stream (no allocation once the workspace exists, no synchronisation), so a whole batch captures as it is
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                run_step(ctx, wl, groups, opts)
                gph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gph, stream=side):
                    run_step(ctx, wl, groups, opts)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            for _ in range(3):
                gph.replay()
            graph_ms = time_steps(gph.replay, steps, torch.cuda.synchronize)
            del gph
        except Exception as e:
            graph_ms = "capture failed: %r" % (e,)
    out = {"workload": label or wl["label"], "ms_per_batch": ms, "ms_per_batch_cuda_graph": graph_ms,
           "tflops": (filt + front) / (ms * 1e-3) / 1e12, "executed_tflops": (filt_exec + front) / (ms * 1e-3) / 1e12,
           "matrices_per_s": sum(b for b, _, _ in wl["groups"]) / (ms * 1e-3), "launches_per_batch": int(launches),
           "stage_ms": {"rsvd": st[0] / per, "deflate_normalise": st[1] / per, "filter": st[2] / per, "restore": st[3] / per}}
    del groups
    torch.cuda.empty_cache()
    return out


def extra_sdp(ctx, peaks, device, n=4096, calls=20, warm=2, tf32_peak=True):
    """The SDP projection sequence at n = 4096 (tf32 filter): ms per projection over the deflated calls, the seven-stage
    split, the filter + reconstruction products against a measured tf32 peak, and the Lanczos passes against HBM."""
    import torch
    from paper_2609_21102_b200 import inputs
    K, k, T = 16, 8, 7
    sched = [list(CLASSICAL)] * T
    x, _ = inputs.sdp_first(n, heads=k, head_mag=1.0e3, device=device)
    V = inputs.randn((n, K), inputs.seed_for(5, 0, inputs.PURPOSE_BASIS), device).float()
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, device=device)
    P = torch.empty((n, n), dtype=torch.float32, device=device)
    times, warm_times = [], []
    for t in range(calls):
        X = x.float()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.defl_psd_project(X, k, V, sched, out=P, gamma=1.1, lanczos_start=v0, warmup=t < warm, exploit_symmetry=True)
        e1.record()
        torch.cuda.synchronize()
        (warm_times if t < warm else times).append(e0.elapsed_time(e1))
        x = inputs.sdp_next(x, t + 1)
    nd = len(times)
    st = [s / nd for s in ctx.defl_get_stage_ms(nd)]
    names = ["block_step_rayleigh_ritz", "deflate", "lanczos_scale", "initialise", "filter", "reconstruct", "basis_update"]
    tf32_peak = measure_tf32_peak() if tf32_peak else float("nan")
    flops = T * 3.0 * n * n * (n + 1.0) + 2.0 * n ** 3          # symmetric products once, R g(X0) in full
    prod_ms = st[4] + st[5]
    symv_bytes = 42.0 * 4.0 * n * n
    times.sort()
    return {"workload": "SDP PSD projection, fp32 storage / tf32 filter: 20 drifting symmetric %dx%d matrices, 8 eigenvalues "
                        "+-1e3 over U(-1,1), k=8, K=16, 7 classical quintic steps, 2 warm-up calls" % (n, n),
            "ms_per_projection": sum(times) / nd, "ms_per_projection_median": times[nd // 2],
            "ms_per_warmup_call": sum(warm_times) / max(1, len(warm_times)),
            "stage_ms": dict(zip(names, st)),
            "roofline_filter": {"bound": "tensor", "kernel": "gemm_tc_kernel (tf32: X^2, W^2 polynomial, X T_t, R g(X0))",
                                "achieved": flops / (prod_ms * 1e-3) / 1e12, "peak": tf32_peak, "unit": "TFLOP/s",
                                "frac": flops / (prod_ms * 1e-3) / 1e12 / tf32_peak,
                                "peak_kind": "torch.matmul 8192^3 with tf32 allowed, best of 10, this run"},
            "roofline_lanczos": {"bound": "hbm", "kernel": "symv_kernel (42 passes over R) + lanczos_step_kernel",
                                 "achieved": symv_bytes / (st[2] * 1e-3) / 1e9, "peak": float(peaks.get("hbm_gbs", 6650.0)),
                                 "unit": "GB/s", "frac": symv_bytes / (st[2] * 1e-3) / 1e9 / float(peaks.get("hbm_gbs", 6650.0)),
                                 "note": "R (67 MB) fits the 126 MB L2: passes after the first are served from it"}}


def extra_inv_root(ctx, device, tf32_peak, n=4096, p=4, calls=12, warm=2):
    """The deflated inverse p-th root at n = 4096 (tf32 products): a static synthetic preconditioner statistic (8
    eigenvalues of 300..2000 over a bulk spread log-uniformly over [0.06, 1]), 2 warm-up calls, then deflated calls:
    ms per call, stage split, the iteration's products against the tf32 rate measured in this run."""
    import torch
    from paper_2609_21102_b200 import inputs
    K, k, T = 16, 8, 8
    u = inputs.rand((n - k,), 705, device=device).double()
    lam = torch.cat([torch.linspace(2000.0, 300.0, k, dtype=torch.float64, device=device), 0.06 ** u])
    q = inputs.haar(n, n, 700, device=device)
    A = ((q * lam.unsqueeze(0)) @ q.T)
    A = (0.5 * (A + A.T)).float()
    del q
    V = inputs.randn((n, K), inputs.seed_for(5, 1, inputs.PURPOSE_BASIS), device).float()
    v0 = inputs.gaussian_vector(n, 5, inputs.PURPOSE_LANCZOS, device=device)
    out = torch.empty((n, n), dtype=torch.float32, device=device)
    times = []
    for t in range(calls):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.defl_inv_root(A, p, k, V, T, out=out, gamma=1.1, lanczos_start=v0, warmup=t < warm, exploit_symmetry=True)
        e1.record()
        torch.cuda.synchronize()
        if t >= warm:
            times.append(e0.elapsed_time(e1))
    nd = len(times)
    st = [x / nd for x in ctx.defl_get_stage_ms(nd)]
    names = ["block_step_rayleigh_ritz", "deflate", "lanczos_scale", "initialise", "iteration", "restore", "basis_update"]
    # distance from the definition: A^(-1/p) from a library eigendecomposition in fp64 (outside every timed path)
    w, v = torch.linalg.eigh(A.double())
    exact = (v * w.pow(-1.0 / p).unsqueeze(0)) @ v.T
    rel_err = float((out.double() - exact).norm() / exact.norm())
    del w, v, exact
    nprod = {1: 2, 2: 3, 4: 4}[p] * (T - 1)                 # Z T and the M update, none of the former in the first step, none of the latter in the last
    flops = nprod * 1.0 * n * n * (n + 1.0)
    times.sort()
    return {"workload": "deflated inverse %d-th root, fp32 storage / tf32 products: static symmetric positive definite %dx%d "
                        "matrix, 8 eigenvalues 300..2000 over a bulk in [0.06, 1], k=8, K=16, %d coupled Newton steps, "
                        "2 warm-up calls" % (p, n, n, T),
            "ms_per_call": sum(times) / nd, "ms_per_call_median": times[nd // 2], "stage_ms": dict(zip(names, st)),
            "rel_error_vs_fp64_eigendecomposition": rel_err,
            "roofline_iteration": {"bound": "tensor", "kernel": "gemm_tc_kernel (tf32, symmetric: Z T, T^2, T^4, T^p M)",
                                   "achieved": flops / (st[4] * 1e-3) / 1e12, "peak": tf32_peak, "unit": "TFLOP/s",
                                   "frac": flops / (st[4] * 1e-3) / 1e12 / tf32_peak,
                                   "peak_kind": "torch.matmul 8192^3 with tf32 allowed, best of 10, this run"}}


def spawn_ranks(args):
    """--gpus N without an outer launcher: start the N ranks here (weak-scaling replicas, one batch per rank)."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--small", action="store_true", help="tiny workload for a quick functional check")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the other workloads, the sustained leg and the end-to-end leg")
    ap.add_argument("--no-symmetry", action="store_true", help="compute the symmetric products in full")
    ap.add_argument("--bf16-iterates", action="store_true", help="filter iterates stored in bf16 in every step (default: scaled IEEE half in the first two)")
    ap.add_argument("--half-iterates", action="store_true", help="filter iterates stored in scaled IEEE half in every step")
    ap.add_argument("--schedule", choices=["muon", "minimax"], default="muon",
                    help="muon: Muon's quintic every step; minimax: per-step minimax quintics (Polar-Express-style)")
    ap.add_argument("--add-restore", action="store_true", help="Eq. 3's post-add (fused into the last filter product) instead of the padded entry")
    ap.add_argument("--streams", type=int, default=2, help="2: one stream + context per shape group (the groups are independent); 1: one stream")
    ap.add_argument("--batch", type=int, default=0, help="override the matrices per shape group (profiling captures)")
    ap.add_argument("--sdp-only", type=int, default=0, metavar="CALLS",
                    help="run only the SDP projection sequence (n = 4096) with this many calls and print its figures (profiling captures)")
    ap.add_argument("--inv-root-only", type=int, default=0, metavar="CALLS",
                    help="run only the deflated inverse-root calls (n = 4096) and print their figures")
    args = ap.parse_args()

    wl_name = "small" if args.small else "gpt2_xl"
    wl = dict(WORKLOADS[wl_name])
    if args.schedule == "minimax":
        wl["schedule"], wl["gamma"] = "minimax", 1.1
        wl["label"] = wl["label"].replace("5 Muon quintic steps", "5 per-step minimax quintic steps (Polar-Express-style)")
    if args.batch > 0:
        wl["groups"] = [(args.batch, m, n) for _, m, n in wl["groups"]]
        wl["label"] += " [batch overridden to %d per group]" % args.batch
    opts = {"sym": not args.no_symmetry, "iterates": 1 if args.bf16_iterates else (2 if args.half_iterates else 0),
            "mode": 1 if args.add_restore else 0}
    storage = ("bf16" if opts["iterates"] == 1 else "IEEE half scaled by 32" if (opts["iterates"] == 2 or opts["mode"] == 1)
               else "IEEE half scaled by 32 in the first two steps and in the steps that share a pass over X, bf16 after")
    sched_note = ("Muon quintic (3.4445, -4.7750, 2.0315) every step" if wl["schedule"] == "muon" else
                  "per-step minimax quintics (greedy Remez from [1e-3, 1], first step / 1.01): the Polar-Express-style "
                  "mapping, coefficients computed by schedules.remez_sign_schedule")
    config = {"workload": wl["label"], "name": wl_name, "k": wl["k"], "oversample": wl["p"], "power_iters": wl["J"],
              "filter_steps": wl["L"], "restore": ("additive (Eq. 3), in the last filter product" if opts["mode"] else "padded, gamma=%g" % wl["gamma"]),
              "schedule": sched_note, "exploit_symmetry": opts["sym"],
              "storage": "input and output bf16; filter iterates " + storage,
              "l2": "inputs (1.2 GB per step) larger than L2; no flush"}

    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            reference_arm(args, wl, config)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    from paper_2609_21102_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    ctx = binding.Context(local_rank)
    ctx.defl_set_profiling(True)
    if args.inv_root_only > 0:
        print(json.dumps(extra_inv_root(ctx, device, float("nan"), calls=args.inv_root_only, warm=min(2, args.inv_root_only - 1))))
        return
    if args.sdp_only > 0:
        print(json.dumps(extra_sdp(ctx, load_peaks()[0], device, calls=args.sdp_only, warm=min(2, args.sdp_only - 1), tf32_peak=False)))
        return
    groups = make_inputs(wl, device)
    ngroups = len(groups)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    lanes = None
    if args.streams > 1:
        lanes = [(binding.Context(local_rank), torch.cuda.Stream()) for _ in groups]
    n_streams = len(lanes) if lanes else 1

    def launch_total():
        return ctx.defl_launch_count() + (sum(c.defl_launch_count() for c, _ in lanes) if lanes else 0)

    step = lambda: run_step(ctx, wl, groups, opts, lanes)
    # Two counts. Algorithmic: one Gram, one polynomial and one apply product per filter step (symmetric products once),
    # the work the method is defined by; it gives `value`, `roofline.achieved` and the end-to-end figure. Executed: the
    # products the library actually runs (where two steps share one pass over X: one Gram, one apply, five short-side
    # products); it gives `executed_tflops` and `roofline.executed_*`, which is what the tensor pipe did.
    filt_f, front_f = workload_flops(wl, opts["sym"], opts["mode"] == 1, opts["iterates"], per_step=True)
    tot_f = filt_f + front_f
    exec_filt_f, _ = workload_flops(wl, opts["sym"], opts["mode"] == 1, opts["iterates"])
    exec_f = exec_filt_f + front_f
    dense_f = sum(b * dense_filter_flops(m, n, wl["L"]) for b, m, n in wl["groups"]) + front_f
    nmat = sum(b for b, _, _ in wl["groups"])

    with ClockSampler(local_rank) as clk:
        for _ in range(max(args.warmup, 3)):
            step()
        barrier()
        launches0 = launch_total()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        barrier()
        t_start = time.time()
        ev[0].record()
        for i in range(args.steps):
            step()
        ev[1].record()
        barrier()
        t_end = time.time()
        launches = launch_total() - launches0
        total_ms = max_over_ranks(ev[0].elapsed_time(ev[1]), dist, "cuda")
        ms_per_step = total_ms / args.steps
        clocks = clk.summary(t_start, t_end)

        # Stage split and the dominant kernel's time: a second timed region of the same K steps on ONE stream, where the
        # events the library records between the stages of every call bracket exactly that stage's kernels (with one
        # stream per shape group the stages of the two groups interleave and a per-stage time is not defined).
        if lanes:
            for _ in range(2):
                run_step(ctx, wl, groups, opts, None)
            barrier()
            es = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            es[0].record()
            for i in range(args.steps):
                run_step(ctx, wl, groups, opts, None)
            es[1].record()
            barrier()
            one_stream_ms = max_over_ranks(es[0].elapsed_time(es[1]), dist, "cuda") / args.steps
        else:
            one_stream_ms = ms_per_step
        ncalls = min(64, args.steps * ngroups) // ngroups * ngroups
        st = ctx.defl_get_stage_ms(ncalls)
        stage_ms = [s / (ncalls / ngroups) for s in st[:4]]
        stage_src = ("CUDA events recorded by the library on its stream inside a timed region of %d steps on one stream "
                     "(%.3f ms per step there)" % (ncalls // ngroups, one_stream_ms))

        sustained = None
        plain_ms = None
        if not args.no_extras:
            # sustained leg: the same step back to back for at least 3 s (the board settles at its power cap)
            barrier()
            s0 = time.time()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            n_sus = 0
            while True:
                for _ in range(10):
                    step()
                n_sus += 10
                torch.cuda.synchronize()
                if time.time() - s0 >= 3.0:
                    break
            e1.record()
            barrier()
            s1 = time.time()
            sus_ms = max_over_ranks(e0.elapsed_time(e1) / n_sus, dist, "cuda")
            sustained = {"ms_per_step": sus_ms, "steps": n_sus, "tflops": aggregate_throughput(tot_f, world, sus_ms) / 1e12,
                         "clocks": clk.summary(s0 + 0.5, s1)}
        # the plain (undeflated) filter of the same batch, for the deflation overhead
        plain = lambda: [ctx.defl_polar_batched(g["G"], 0, 0, 0, schedule_of(wl["schedule"], wl["L"]), out=g["out"],
                                                exploit_symmetry=opts["sym"], bf16_iterates=opts["iterates"]) for g in groups]
        plain()
        plain_ms = time_steps(plain, 5, torch.cuda.synchronize)

    # end to end through the host-buffer entry point (pinned host tensors, copies inside the timed region)
    e2e = None
    if not args.no_extras:
        sched = schedule_of(wl["schedule"], wl["L"])
        hG = [g["G"].cpu().pin_memory() for g in groups]
        hO = [torch.empty_like(h).pin_memory() for h in hG]
        e2e_ctx = [binding.Context(local_rank) for _ in groups]
        e2e_streams = [torch.cuda.Stream() for _ in groups]

        def e2e_group(c, s, h, o, g):
            torch.cuda.set_device(local_rank)
            with torch.cuda.stream(s):
                c.defl_polar_batched_host(h, o, wl["k"], wl["p"], wl["J"], sched, sketch=g["Om"], gamma=wl["gamma"],
                                          exploit_symmetry=opts["sym"], restore_mode=opts["mode"])

        def e2e_step():
            # the call blocks until its output sits in host memory; the shape groups run from host threads of their
            # own (one context each), so that one group's copies overlap the other's computation
            ts = [threading.Thread(target=e2e_group, args=(c, s, h, o, g)) for c, s, h, o, g in zip(e2e_ctx, e2e_streams, hG, hO, groups)]
            for t in ts:
                t.start()
            for t in ts:
                t.join()
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        n_e2e = max(1, min(args.steps, 3))
        for _ in range(n_e2e):
            e2e_step()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / n_e2e, dist, "cuda")
        nbytes = sum(h.numel() * h.element_size() for h in hG)
        e2e = {"value": aggregate_throughput(tot_f, world, e2e_ms) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes}
        del hG, hO, e2e_ctx

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peaks_kind = load_peaks()
    burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    sust = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    value = aggregate_throughput(tot_f, world, ms_per_step) / 1e12
    filt_ms = stage_ms[2]
    n_filter_launches = filter_launches(wl, opts["mode"] == 1, opts["iterates"])
    ach = filt_f / (filt_ms * 1e-3) / 1e12 if filt_ms > 0 else None
    ach_exec = exec_filt_f / (filt_ms * 1e-3) / 1e12 if filt_ms > 0 else None
    sm_mhz = clocks.get("sm_mhz") or 0.0
    # a short timed region runs near the maximum clock (compare with the burst peak), a long one at the power cap
    # (compare with the sustained peak): both fractions are given, and time x clock so that runs at different clocks compare
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel (filter chain: X X^T, A^2 polynomial, B X)",
                "achieved": ach, "peak": burst, "unit": "TFLOP/s", "frac": (ach / burst) if ach else None,
                "peak_kind": "bf16_tflops (burst), of %s" % peaks_kind,
                "frac_of_sustained_peak": (ach / sust) if ach else None,
                "flops": "algorithmic: one Gram, one polynomial and one apply product per filter step, symmetric products once "
                         "(%.4g per step of the batch); executed_*: the products the library runs, two steps per pass over X "
                         "where it pairs them (%.4g per launch)" % (filt_f / wl["L"], exec_filt_f / n_filter_launches),
                "executed_achieved": ach_exec, "executed_frac": (ach_exec / burst) if ach_exec else None,
                "executed_frac_of_sustained_peak": (ach_exec / sust) if ach_exec else None,
                "launches_per_step": n_filter_launches, "avg_launch_ms": filt_ms / n_filter_launches,
                "stage_source": stage_src,
                "ms_x_mhz": filt_ms * sm_mhz,
                "dense_equivalent_tflops": sum(b * dense_filter_flops(m, n, wl["L"]) for b, m, n in wl["groups"]) / (filt_ms * 1e-3) / 1e12,
                "traffic": FILTER_TRAFFIC_BYTES_PER_LAUNCH if (wl_name == "gpt2_xl" and args.batch == 0) else None,
                "traffic_unit": "bytes per launch (ncu, 8-matrix capture scaled to the batch)"}
    front_ms = stage_ms[0] + stage_ms[1] + stage_ms[3]
    line = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
            "flops_convention": "value = algorithmic flops / time: per filter step one Gram, one polynomial and one apply product, "
                                "symmetric products counted once, plus the front end; executed_tflops counts the products the "
                                "library runs (fewer where two filter steps share one pass over X); dense_equivalent_tflops "
                                "counts every per-step product in full",
            "executed_tflops": aggregate_throughput(exec_f, world, ms_per_step) / 1e12,
            "dense_equivalent_tflops": aggregate_throughput(dense_f, world, ms_per_step) / 1e12,
            "matrices_per_s": world * nmat / (ms_per_step * 1e-3),
            "pct_bf16_peak": {"burst": 100.0 * value / world / burst, "sustained": 100.0 * value / world / sust},
            "stage_ms": {"rsvd": stage_ms[0], "deflate_normalise": stage_ms[1], "filter": stage_ms[2], "restore": stage_ms[3],
                         "one_stream_ms_per_step": one_stream_ms},
            "deflation_overhead_frac": (ms_per_step - plain_ms) / ms_per_step if plain_ms else None,
            "front_end_frac_of_step": front_ms / sum(stage_ms) if sum(stage_ms) > 0 else None,
            "plain_filter_ms": plain_ms,
            "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "streams": n_streams, "clocks": clocks,
            "sustained": sustained}

    if not args.no_extras and wl_name == "gpt2_xl" and args.batch == 0:
        extras = {}
        try:
            extras["gpt2_small"] = extra_polar(ctx, "gpt2_small", opts, device, steps=20, graph=True)
            extras["gpt2_medium_large"] = extra_polar(ctx, "gpt2_medium_large", opts, device, steps=10, graph=True)
            del groups
            torch.cuda.empty_cache()
            xl_minimax = dict(WORKLOADS["gpt2_xl"], schedule="minimax", gamma=1.1)
            WORKLOADS["_xl_minimax"] = xl_minimax
            extras["gpt2_xl_minimax_schedule"] = extra_polar(ctx, "_xl_minimax", opts, device, steps=10,
                                                             label="GPT-2-XL batch, per-step minimax schedule, gamma=1.1")
            extras["gpt2_xl_add_restore"] = extra_polar(ctx, "gpt2_xl", dict(opts, mode=1), device, steps=10,
                                                        label="GPT-2-XL batch, additive restore (Eq. 3) in the last filter product")
            extras["sdp_4096"] = extra_sdp(ctx, peaks, device)
            extras["inv_root_4096"] = extra_inv_root(ctx, device, extras["sdp_4096"]["roofline_filter"]["peak"])
        except Exception as e:      # an extra that fails must not take the headline with it
            extras["error"] = repr(e)
        line["extras"] = extras

    if not args.no_cpu_baseline:
        secs, fl, sample = oracle_sample(wl)
        # whole batch at the oracle's measured seconds per matrix of each shape (every matrix of a shape costs the same)
        batch_s = sum(b * s for (b, _, _), s in zip(wl["groups"], secs))
        batch_f = sum(b * f for (b, _, _), f in zip(wl["groups"], fl))
        line["cpu_baseline"] = {"value": batch_f / batch_s / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count() or 1,
                                "kind": "oracle", "sample": sample,
                                "seconds_per_matrix": {"%dx%d" % (m, n): s for (_, m, n), s in zip(wl["groups"], secs)},
                                "extrapolated": "batch figure = measured seconds per matrix of each shape x matrices of that shape",
                                "batch_seconds_extrapolated": batch_s, "matrices_per_s": nmat / batch_s}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
