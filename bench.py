#!/usr/bin/env python
"""Benchmark of the deflated polar filter on synthetic GPT-2-XL-shaped Muon batches.

One step = one pass of the whole hot path (batched randomized SVD, deflate + normalise, five quintic
Newton-Schulz steps, restore) over one batch: 48 matrices 1600x6400 and 48 matrices 1600x1600 in
bf16 with the heavy-tailed spectrum sigma_i = max(200/i, 1e-4), k=32, oversampling 16, 2 subspace
iterations. Prints ONE JSON line (see README / DESIGN for the keys).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--small]

N > 1 is launched under torchrun; every rank runs the same batch on its own GPU (independent
matrices, no data-path collective) and the line reports the whole-job aggregate.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "deflated polar-filter TFLOP/s & matrices/s per batch; % bf16 tensor peak"
MUON = (3.4445, -4.7750, 2.0315)
SYM = True   # compute X X^T and A A on the tiles that reach the diagonal and mirror them (--no-symmetry turns it off)
BF16_ITERATES = 0       # storage of the filter's iterates: 0 scaled IEEE half in the first two steps then bf16 (default),
                        # 1 bf16 throughout (--bf16-iterates), 2 scaled half throughout (--half-iterates)
GAMMA = 1.01            # padding of the restored head (1.1 with the minimax schedule, the value the paper uses with it)
SCHEDULE = "muon"       # --schedule minimax: per-step minimax quintics (the Polar-Express-style mapping)
SCHEDULE_NOTE = "Muon quintic (3.4445, -4.7750, 2.0315) every step"
_MINIMAX = {}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {
    # name: (list of (b, m, n), k, p, J, L)
    "gpt2_xl": {"groups": [(48, 1600, 6400), (48, 1600, 1600)], "k": 32, "p": 16, "J": 2, "L": 5,
                "label": "GPT-2-XL Muon shapes, bf16: 48 x 1600x6400 + 48 x 1600x1600, sigma_i=max(200/i,1e-4), "
                         "k=32, p=16, J=2, 5 Muon quintic steps"},
    "small": {"groups": [(4, 256, 1024), (4, 256, 256)], "k": 8, "p": 8, "J": 1, "L": 5,
              "label": "small check: 4 x 256x1024 + 4 x 256x256"},
}


def sched_of(wl):
    """The [L][3] coefficient schedule of the run: Muon's quintic repeated, or per-step minimax quintics built by
    greedy Remez exchange from [1e-3, 1] (first step rescaled by 1.01); same products per step either way."""
    L = wl["L"]
    if SCHEDULE == "muon":
        return [list(MUON)] * L
    if L not in _MINIMAX:
        from paper_2609_21102_b200 import schedules
        _MINIMAX[L] = [list(c) for c in schedules.remez_sign_schedule(1e-3, L, margin=0.01)[0]]
    return _MINIMAX[L]


def flops_per_matrix(m, n, k, p, J, L):
    """Algorithmic flops of one matrix: dense filter count, rSVD products, subtract and restore."""
    ms, ml = min(m, n), max(m, n)
    l = min(ms, k + p) if k > 0 else 0
    filt = L * (4.0 * ms * ms * ml + 2.0 * ms ** 3)
    rsvd = 2.0 * ml * ms * l * (2 + 2 * J) if k > 0 else 0.0
    defl = 2.0 * 2.0 * m * n * k          # residual norm pass + X0 pass
    return filt, rsvd + defl


# Average DRAM bytes per filter-product launch: dram__bytes_read + dram__bytes_write of the six kinds of filter
# launch (X X^T, A^2 polynomial, B X for each shape group) from the ncu captures summarised in
# the filter-kernel summary under profiles/ (8 matrices per group: 132.4 MB on average), scaled by 48/8.
FILTER_TRAFFIC_BYTES_PER_LAUNCH = 795e6


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


def executed_filter_flops(m, n, L, symmetric, tile=256):
    """Flops the tensor engine executes for the L filter steps of one matrix. It works on 256 x 256 output
    tiles made of two 128-row halves; edge tiles compute only the rows (in halves) and columns (in sixteens)
    that exist; with `symmetric` the two symmetric products skip every half-tile left of the diagonal."""
    ms, ml = min(m, n), max(m, n)

    def product(M, N, K, sym):
        total = 0.0
        for r0 in range(0, M, tile):
            for c0 in range(0, N, tile):
                cols = min(tile, ((N - c0 + 15) // 16) * 16)
                for h0 in (r0, r0 + 128):
                    if h0 >= M:
                        continue
                    if sym and c0 + tile <= h0:
                        continue
                    total += 2.0 * 128 * cols * K
        return total

    return L * (product(ms, ms, ml, symmetric) + product(ms, ms, ms, symmetric) +
                (product(m, n, m, False) if m <= n else product(m, n, n, False)))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs: one nvidia-smi process in loop
    mode (50 ms period), started ahead of the region; only samples that arrive between mark_start() and
    mark_end() are kept."""

    def __init__(self, index):
        self.index, self.rows, self._all, self._t, self._p = index, [], [], None, None
        self.t0 = self.t1 = None

    def _run(self):
        for line in self._p.stdout:
            parts = [x.strip() for x in line.strip().split(",")]
            if len(parts) >= 6:
                self._all.append((time.time(), parts))

    def __enter__(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self._p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q,
                                        "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                       stderr=subprocess.DEVNULL, text=True, bufsize=1)
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()
            time.sleep(0.3)      # let the first samples arrive before the region starts
        except Exception:
            self._p = None
        return self

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def __exit__(self, *a):
        if self._p is not None:
            self._p.terminate()          # the one process this object started
            try:
                self._p.wait(timeout=5)
            except Exception:
                self._p.kill()
            self._t.join(timeout=5)
        t0 = self.t0 if self.t0 is not None else 0.0
        t1 = self.t1 if self.t1 is not None else float("inf")
        self.rows = [r for (t, r) in self._all if t0 <= t <= t1]
        if not self.rows and self._all:      # a region shorter than the period: the nearest sample
            mid = 0.5 * (t0 + min(t1, time.time()))
            self.rows = [min(self._all, key=lambda tr: abs(tr[0] - mid))[1]]

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        sm = sorted(float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit())
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [nm for i, nm in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in self.rows)]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows)}


def make_inputs(wl, device):
    import torch
    from paper_2609_21102_b200 import inputs
    groups = []
    for si, (b, m, n) in enumerate(wl["groups"]):
        G = inputs.workload_power_law(b, m, n, 4, si, 1.0, 200.0, 1e-4, device=device).to(torch.bfloat16)
        l = min(min(m, n), wl["k"] + wl["p"])
        Om = inputs.sketch(b, min(m, n), l, 4, si, device=device)
        groups.append({"G": G, "Om": Om, "out": torch.empty_like(G)})
    return groups


def run_step(ctx, wl, groups, lanes=None):
    """One step = every shape group through defl_polar_batched. With `lanes` (one (context, stream) pair per
    group) the independent groups are enqueued on their own streams, forked from and joined to the current
    stream, so that the small latency-bound kernels of one group overlap the other group's work."""
    import torch
    if not lanes:
        for g in groups:
            ctx.defl_polar_batched(g["G"], wl["k"], wl["p"], wl["J"], sched_of(wl), out=g["out"],
                                   sketch=g["Om"], gamma=GAMMA, exploit_symmetry=SYM, bf16_iterates=BF16_ITERATES)
        return
    main = torch.cuda.current_stream()
    fork = torch.cuda.Event()
    fork.record(main)
    for g, (c, s) in zip(groups, lanes):
        s.wait_event(fork)
        with torch.cuda.stream(s):
            c.defl_polar_batched(g["G"], wl["k"], wl["p"], wl["J"], sched_of(wl), out=g["out"],
                                 sketch=g["Om"], gamma=GAMMA, exploit_symmetry=SYM, bf16_iterates=BF16_ITERATES)
            done = torch.cuda.Event()
            done.record(s)
        main.wait_event(done)


def oracle_sample(wl, seconds_hint=20.0):
    """Times the fp64 oracle on one matrix of the smallest group (a bounded sample of the workload)."""
    import numpy as np
    import oracle
    from paper_2609_21102_b200 import inputs
    import torch
    b, m, n = min(wl["groups"], key=lambda g: g[1] * g[2])
    si = wl["groups"].index((b, m, n))
    G = inputs.workload_power_law(1, m, n, 4, si, 1.0, 200.0, 1e-4).to(torch.bfloat16).double().numpy()[0]
    l = min(min(m, n), wl["k"] + wl["p"])
    Om = inputs.sketch(1, min(m, n), l, 4, si).double().numpy()[0]
    t0 = time.perf_counter()
    oracle.deflated_polar(G, wl["k"], l, Om, wl["J"], oracle.schedule(sched_of(wl)), gamma=GAMMA)
    dt = time.perf_counter() - t0
    filt, rest = flops_per_matrix(m, n, wl["k"], wl["p"], wl["J"], wl["L"])
    return dt, (filt + rest), "1 matrix %dx%d of the batch, full path, fp64" % (m, n)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--small", action="store_true", help="tiny workload for a quick functional check")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-symmetry", action="store_true", help="compute the symmetric products in full")
    ap.add_argument("--bf16-iterates", action="store_true", help="filter iterates stored in bf16 in every step (default: scaled IEEE half in the first two)")
    ap.add_argument("--half-iterates", action="store_true", help="filter iterates stored in scaled IEEE half in every step")
    ap.add_argument("--schedule", choices=["muon", "minimax"], default="muon",
                    help="muon: Muon's quintic every step; minimax: per-step minimax quintics (Polar-Express-style)")
    ap.add_argument("--streams", type=int, default=2, help="2: one stream + context per shape group; 1: one stream")
    ap.add_argument("--batch", type=int, default=0, help="override the matrices per shape group (profiling captures)")
    args = ap.parse_args()
    global SYM, BF16_ITERATES, SCHEDULE, SCHEDULE_NOTE, GAMMA
    SCHEDULE = args.schedule
    if SCHEDULE == "minimax":
        GAMMA = 1.1
        SCHEDULE_NOTE = ("per-step minimax quintics (greedy Remez from [1e-3, 1], first step / 1.01): the "
                         "Polar-Express-style mapping, coefficients computed by schedules.remez_sign_schedule")
    SYM = not args.no_symmetry
    BF16_ITERATES = 1 if args.bf16_iterates else (2 if args.half_iterates else 0)
    wl_name = "small" if args.small else "gpt2_xl"
    wl = dict(WORKLOADS[wl_name])
    if args.batch > 0:
        wl["groups"] = [(args.batch, m, n) for _, m, n in wl["groups"]]
        wl["label"] += " [batch overridden to %d per group]" % args.batch
    if SCHEDULE == "minimax":
        wl["label"] = wl["label"].replace("5 Muon quintic steps", "5 per-step minimax quintic steps (Polar-Express-style)")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": wl["label"], "name": wl_name, "k": wl["k"], "oversample": wl["p"], "power_iters": wl["J"],
              "filter_steps": wl["L"], "restore": "padded, gamma=%g" % GAMMA, "schedule": SCHEDULE_NOTE, "exploit_symmetry": SYM,
              "storage": "input and output bf16; filter iterates " + ("bf16" if BF16_ITERATES == 1 else ("IEEE half scaled by 32" if BF16_ITERATES == 2 else "IEEE half scaled by 32 in the first two steps, bf16 after")),
              "l2": "inputs (1.2 GB per step) larger than L2; no flush"}
    tot_f = sum(b * sum(flops_per_matrix(m, n, wl["k"], wl["p"], wl["J"], wl["L"])) for b, m, n in wl["groups"])
    nmat = sum(b for b, _, _ in wl["groups"])

    if args.impl == "reference":
        if rank != 0:
            return
        cores = os.cpu_count() or 1
        # W untimed and K timed steps, each the oracle's full path on one 1600x1600 matrix of the batch (about 1.5 s)
        for _ in range(max(0, args.warmup)):
            oracle_sample(wl)
        times = []
        for _ in range(max(1, args.steps)):
            dt, fl, sample = oracle_sample(wl)
            times.append(dt)
        dt = sum(times) / len(times)
        val = fl / dt / 1e12
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
                "steps": len(times), "warmup": max(0, args.warmup), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "matrices_per_s": 1.0 / dt,
                "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    from paper_2609_21102_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    ctx = binding.Context(local_rank)
    groups = make_inputs(wl, torch.device("cuda", local_rank))
    ctx.defl_set_profiling(True)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    lanes = None
    if args.streams > 1:
        lanes = [(binding.Context(local_rank), torch.cuda.Stream()) for _ in groups]
    config["streams"] = len(lanes) if lanes else 1

    def launch_total():
        return ctx.defl_launch_count() + (sum(c.defl_launch_count() for c, _ in lanes) if lanes else 0)

    for _ in range(max(args.warmup, 3)):
        run_step(ctx, wl, groups, lanes)
    barrier()
    launches0 = launch_total()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with ClockSampler(local_rank) as clk:
        barrier()
        clk.mark_start()
        ev[0].record()
        for i in range(args.steps):
            run_step(ctx, wl, groups, lanes)
            ev[i + 1].record()
        barrier()
        clk.mark_end()
    launches = launch_total() - launches0
    total_ms = max_over_ranks(ev[0].elapsed_time(ev[-1]), dist, "cuda")
    ms_per_step = total_ms / args.steps

    # stage split of one more (untimed) step, with the same events the library records on its stream
    stage_tot = [0.0, 0.0, 0.0, 0.0]
    filt_flops = 0.0        # dense count of the filter products
    filt_executed = 0.0     # flops the tensor cores actually execute (tiles below the diagonal are skipped)
    STAGE_REPS = 7          # median over the repetitions: a single step's split moves by several percent with the
                            # power state, and reading the events synchronises the stream after every call
    per_rep = []
    for rep in range(STAGE_REPS):
        tot = [0.0, 0.0, 0.0, 0.0]
        for g, (b, m, n) in zip(groups, wl["groups"]):
            ctx.defl_polar_batched(g["G"], wl["k"], wl["p"], wl["J"], sched_of(wl), out=g["out"], sketch=g["Om"],
                                   gamma=GAMMA, exploit_symmetry=SYM, bf16_iterates=BF16_ITERATES)
            ms = ctx.defl_get_stage_ms()
            for i in range(min(4, len(ms))):
                tot[i] += ms[i]
            if rep == 0:
                filt_flops += b * flops_per_matrix(m, n, wl["k"], wl["p"], wl["J"], wl["L"])[0]
                filt_executed += b * executed_filter_flops(m, n, wl["L"], SYM)
        per_rep.append(tot)
    for i in range(4):
        vals = sorted(r[i] for r in per_rep)
        stage_tot[i] = vals[len(vals) // 2]
    plain_ms = 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for g in groups:
        ctx.defl_polar_batched(g["G"], 0, 0, 0, sched_of(wl), out=g["out"], exploit_symmetry=SYM, bf16_iterates=BF16_ITERATES)
    e1.record()
    torch.cuda.synchronize()
    plain_ms = e0.elapsed_time(e1)

    # end to end through the host-buffer entry point (pinned host tensors, copies inside the timed region)
    e2e = None
    if rank == 0 or world > 1:
        hG = [g["G"].cpu().pin_memory() for g in groups]
        hO = [torch.empty_like(h).pin_memory() for h in hG]
        def e2e_group(c, h, o, g, stream=None):
            if stream is None:
                c.defl_polar_batched_host(h, o, wl["k"], wl["p"], wl["J"], sched_of(wl), sketch=g["Om"], gamma=GAMMA,
                                          exploit_symmetry=SYM)
            else:
                torch.cuda.set_device(local_rank)
                with torch.cuda.stream(stream):
                    c.defl_polar_batched_host(h, o, wl["k"], wl["p"], wl["J"], sched_of(wl), sketch=g["Om"],
                                              gamma=GAMMA, exploit_symmetry=SYM)

        def e2e_step():
            # the call blocks until its output sits in host memory; with one context per shape group the groups
            # run from host threads of their own, so that one group's copies overlap the other's computation
            if not lanes:
                for h, o, g in zip(hG, hO, groups):
                    e2e_group(ctx, h, o, g)
                return
            ts = [threading.Thread(target=e2e_group, args=(c, h, o, g, s)) for (c, s), h, o, g in zip(lanes, hG, hO, groups)]
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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks, peaks_kind = load_peaks()
    value = aggregate_throughput(tot_f, world, ms_per_step) / 1e12
    filt_ms = stage_tot[2]
    n_filter_launches = 3 * wl["L"] * len(groups)
    # achieved = flops the kernel really executes / its time (no credit for skipped symmetric tiles)
    ach = filt_executed / (filt_ms * 1e-3) / 1e12 if filt_ms > 0 else None
    ach_dense = filt_flops / (filt_ms * 1e-3) / 1e12 if filt_ms > 0 else None
    peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel (filter chain: X X^T, A^2 polynomial, B X)",
                "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": (ach / peak) if ach else None,
                "peak_kind": "bf16_tflops_sustained, of %s" % peaks_kind,
                "frac_of_burst": (ach / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))) if ach else None,
                "launches_per_step": n_filter_launches, "avg_launch_ms": filt_ms / n_filter_launches,
                "flops_per_launch_avg": filt_executed / n_filter_launches,
                "dense_equivalent_tflops": ach_dense,
                "traffic": FILTER_TRAFFIC_BYTES_PER_LAUNCH if (wl_name == "gpt2_xl" and args.batch == 0) else None,
                "traffic_unit": "bytes per launch (ncu, 8-matrix capture scaled to the batch)"}
    line = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
            "matrices_per_s": world * nmat / (ms_per_step * 1e-3),
            "pct_bf16_peak_sustained": 100.0 * value / world / peak,
            "stage_ms": {"rsvd": stage_tot[0], "deflate_normalise": stage_tot[1], "filter": stage_tot[2],
                         "restore": stage_tot[3]},
            "deflation_overhead_frac": (ms_per_step - plain_ms) / ms_per_step if ms_per_step > 0 else None,
            "plain_filter_ms": plain_ms,
            "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clk.summary()}
    if not args.no_cpu_baseline:
        dt, fl, sample = oracle_sample(wl)
        line["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count() or 1,
                                "kind": "oracle", "sample": sample, "seconds": dt, "matrices_per_s": 1.0 / dt}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
