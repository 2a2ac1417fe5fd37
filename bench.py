#!/usr/bin/env python
"""Benchmark of the AdaCGD hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--workload c5|c4|c3|c2|c1] [--impl reference]

One JSON line on stdout (rank 0).  The default workload is the compression-only
stress c5 (n = 8 rows, d = 25e6): one step = worker-side diff + select + error +
pick + update + mean over the 8 rows, followed by the master-side compression of
the d-vector.  The timed region of K steps is repeated R times (each repeat bracketed
by a barrier and a synchronize); `value` is the median repeat, the others are listed.
The default line also carries `worst_case` (the same workload with the trigger at
zeta = 0, which forces every row to its weakest compressor, 10 % of the entries) and
`full_iteration`: workloads c1-c4 timed as whole iterations a0-a5 of Algorithm 1
through adacgd_step.  With --gpus N > 1 (launched by torchrun) every rank runs an
independent replica of the workload on its own GPU: the path has no exchange step on
one node, so there is no data-path collective.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synthetic_inputs as S  # noqa: E402

METRIC = "compressed_elems_per_s"
UNIT = "elems/s"


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            time.sleep(0.3)   # let the first sample land before the timed region starts
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) == 6:
                self.samples.append(parts)

    def __exit__(self, *exc):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        for s in self.samples:
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), s[2:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup(backend: str = "nccl"):
    """One process per GPU (replicas only: the ranks exchange nothing but the timing).  With backend
    "gloo" no GPU is touched: the CPU tests run the same rendezvous, barrier and reduction."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if backend == "nccl":
        import torch
        torch.cuda.set_device(local)
    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return rank, world, local


def barrier_sync(world, device: str = "cuda"):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if device == "cuda":
        torch.cuda.synchronize()


def max_over_ranks(value: float, world, device: str = "cuda") -> float:
    """The slowest rank sets the time of the job."""
    import torch
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_step: float, steps: int, ms_max: float, world: int) -> float:
    """Whole-job units per second: every rank processed the same units in the time of the slowest."""
    return world * units_per_rank_step * steps / (ms_max * 1e-3)


# ----------------------------------------------------------------------------- oracle legs
def oracle_sample_c5(W, budget_s: float, seed=0):
    """Runs the CPU oracle, as it stands, on a bounded sample of workload c5: one worker
    row restricted to its first d_s columns, the Top-K sizes scaled with d_s."""
    from oracle import adacgd_oracle as O
    rate_guess = 4.0e5  # elements per second of the plain oracle, order of magnitude
    d_s = int(min(W["d"], max(1.0e5, budget_s * rate_guess)))
    Xs, G0 = S.stress_vectors(1, d_s, blocks=W["blocks"], period=W["period"], seed=seed, device="cpu")
    cands = [(k, max(1, int(p * d_s // W["d"]))) for k, p in W["worker"]]
    x, y, h = Xs[1][0].numpy(), Xs[0][0].numpy(), G0[0].numpy()
    t0 = time.perf_counter()
    res = O.adacgd(h, y, x, cands, 1.0)
    dt = time.perf_counter() - t0
    return d_s / dt, dt, f"1 of {W['n']} worker rows, first {d_s} of {W['d']} columns, K scaled, level {res['level']}"


def oracle_sample_dense(W, budget_s: float, seed=0):
    """One oracle iteration (all stages) of a dense workload with the sample count per
    worker cut to m_s and the workers cut to n_s so that it fits the time budget."""
    from oracle import adacgd_oracle as O
    n_s = min(W["n"], 2)
    m_s = int(max(8, min(W["m"], budget_s * 2.0e7 / (W["d"] * n_s))))
    if W["loss"] == 2:
        A, t, _ = S.least_squares_problem(n_s, W["d"], m_s, seed=seed)
    else:
        A, t = S.logistic_problem(n_s, W["d"], m_s, seed=seed)
    prob = dict(A=[A[i] for i in range(n_s)], target=[t[i] for i in range(n_s)], loss=W["loss"], lam=W["lam"])
    st = O.init_state(prob, np.zeros(W["d"], np.float32), W["worker"])
    t0 = time.perf_counter()
    O.step(st, prob, 0.1, W["worker"], 1.0, W["master"], 1.0)
    dt = time.perf_counter() - t0
    elems = n_s * W["d"] + (W["d"] if W["master"] else 0)
    return elems / dt, dt, f"{n_s} of {W['n']} workers, {m_s} of {W['m']} samples each, one iteration"


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores, one bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    W = S.WORKLOADS[args.workload]
    per_step = 150.0 / max(1, args.steps + args.warmup)
    fn = oracle_sample_c5 if args.workload == "c5" else oracle_sample_dense
    times, rates, sample = [], [], ""
    for it in range(args.warmup + args.steps):
        rate, dt, sample = fn(W, per_step)
        if it >= args.warmup:
            times.append(dt)
            rates.append(rate)
    value = float(np.mean(rates))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU legs
# algorithmic bytes per element and row that each streaming kernel of the compression must move
KERNEL_BYTES = {"k_pass1": 12, "k_update": 8, "k_hist<1>": 8, "k_hist<2>": 8, "k_hist<3>": 8, "k_energy": 12,
                "k_quant_err": 8}
NOMINAL_HBM_GBS = 7700.0   # HGX B200 data-sheet figure, for context beside the measured copy bandwidth


def counted_traffic(kernel: str):
    """DRAM bytes per element and row that ncu counted for `kernel` (dram__bytes_read.sum +
    dram__bytes_write.sum over one launch), from profiles/dram_bytes_per_element.txt.  Each line of that
    table names the source files the kernel lives in and their hash at the time of the capture: once one of
    them has changed the figure is stale and None is returned."""
    path = os.path.join(ROOT, "profiles", "dram_bytes_per_element.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        parts = line.split()
        if len(parts) < 4 or parts[0] != kernel:
            continue
        h = hashlib.sha256()
        for f in parts[2].split(","):
            src = os.path.join(ROOT, "paper_2211_00188_b200", "csrc", f)
            if not os.path.exists(src):
                return None
            h.update(open(src, "rb").read())
        return float(parts[1]) if h.hexdigest()[:16] == parts[3] else None
    return None


def kernel_table(prof, steps):
    tot = sum(v[0] for v in prof.values()) or 1.0
    return {k: {"ms_total": round(v[0], 4), "launches": v[1], "us_per_step": round(1e3 * v[0] / steps, 2),
                "share": round(v[0] / tot, 4)}
            for k, v in sorted(prof.items(), key=lambda kv: -kv[1][0])}


def timed_repeats(run_steps, steps, repeats, world, local):
    """`repeats` timed regions of exactly `steps` steps, each bracketed by a barrier and a synchronize and
    timed with CUDA events on the launching stream; the slowest rank sets each repeat's time."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    with ClockSampler(local) as clk:
        for _ in range(repeats):
            barrier_sync(world)
            e0.record()
            run_steps(steps)
            e1.record()
            barrier_sync(world)
            times.append(max_over_ranks(e0.elapsed_time(e1), world))
    return times, clk.summary()


def repeat_stats(times, steps):
    per = sorted(t / steps for t in times)
    return {"n": len(per), "ms_per_step": [round(t, 5) for t in per], "median": float(np.median(per)),
            "min": per[0], "max": per[-1]}


def bench_c5(args, rank, world, local):
    import torch
    import paper_2211_00188_b200 as pkg

    W = dict(S.WORKLOADS["c5"])
    if args.scale != 1.0:
        W["d"] = int(W["d"] * args.scale) // 4 * 4
        W["worker"] = [(k, max(1, int(p * args.scale))) for k, p in W["worker"]]
        W["master"] = [(k, max(1, int(p * args.scale))) for k, p in W["master"]]
    n, d = W["n"], W["d"]
    dev = torch.device("cuda", local)
    Xs, G0 = S.stress_vectors(n, d, W["blocks"], W["period"], seed=rank, device=dev)
    eng = pkg.AdaCGD(n, d, W["worker"], args.zeta, W["master"], args.zeta, host_staging=args.e2e_steps > 0, device=dev)
    level = torch.zeros(n, dtype=torch.int32, device=dev)
    bits = torch.zeros(n, dtype=torch.int64, device=dev)
    mlevel = torch.zeros(1, dtype=torch.int32, device=dev)
    P = W["period"]
    peak, peak_src = measured_peaks()
    elems_per_step = n * d + d
    step_floor_bytes = 20 * (n + 1) * d + 4 * d           # 12 B + 8 B per element and row, + the mean

    def run_case(zeta, steps, warmup, repeats):
        """The step loop at trigger `zeta` from a fresh copy of the start state."""
        G = G0.clone()
        gt = [G.mean(0), torch.empty(d, device=dev)]
        gm = gt[0].clone().view(1, d)
        state = {"t": 1}

        def run_steps(k):
            for _ in range(k):
                t = state["t"]
                X, Y = Xs[t % P], Xs[(t - 1) % P]
                cur, nxt = gt[t % 2], gt[(t + 1) % 2]
                eng.compress(X, G, Y, W["worker"], zeta, mean_out=nxt, level=level, bits=bits)
                eng.compress(nxt.view(1, d), gm, cur.view(1, d), W["master"], zeta, level=mlevel)
                state["t"] = t + 1

        run_steps(warmup)
        launches0 = eng.launch_count()
        times, clocks = timed_repeats(run_steps, steps, repeats, world, local)
        launches = (eng.launch_count() - launches0) // repeats
        # the same K steps once more with the library's per-kernel CUDA-event timers switched on
        eng.profile_enable(64 * steps + 64)
        hist = {}
        for _ in range(steps):
            run_steps(1)
            for l in level.cpu().tolist():
                hist[l] = hist.get(l, 0) + 1
        prof = eng.profile_read()
        eng.profile_enable(0)
        st = repeat_stats(times, steps)
        step_gbs = step_floor_bytes / (st["median"] * 1e-3) / 1e9
        return dict(stats=st, clocks=clocks, launches=launches, prof=prof, level_histogram={str(k): v for k, v in sorted(hist.items())},
                    levels_last_step=level.cpu().tolist() + mlevel.cpu().tolist(),
                    step_roofline={"algorithmic_bytes_per_step": step_floor_bytes, "achieved_gbs": step_gbs,
                                   "frac": step_gbs / peak, "frac_of_nominal_7700": step_gbs / NOMINAL_HBM_GBS},
                    state=(G, gt, gm, state))

    main = run_case(args.zeta, args.steps, args.warmup, args.repeats)
    ms = main["stats"]["median"] * args.steps
    value = job_throughput(elems_per_step, args.steps, ms, world)
    prof = main["prof"]

    # roofline of the dominant kernel: algorithmic bytes of its launches / its device time
    kern = {k: v for k, v in prof.items() if k in KERNEL_BYTES}
    top = max(kern, key=lambda k: kern[k][0])
    rows_total = (n + 1) * args.steps          # worker launch (n rows) + master launch (1 row) per step
    top_bytes = KERNEL_BYTES[top] * rows_total * d + (4 * d * args.steps if top == "k_update" else 0)
    achieved = top_bytes / (kern[top][0] * 1e-3) / 1e9
    per_elem = counted_traffic(top)
    traffic = None if per_elem is None else per_elem * rows_total * d / kern[top][1]   # bytes per launch, like achieved
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "launches": kern[top][1], "avg_launch_ms": kern[top][0] / kern[top][1],
                "whole_step_frac": main["step_roofline"]["frac"]}

    worst = None
    if not args.no_extra and args.zeta != 0.0:
        w = run_case(0.0, args.steps, args.warmup, 3)
        worst = {"what": "same workload with zeta = 0: no row may skip, every row applies its weakest compressor (10 % of the entries)",
                 "zeta": 0.0, "ms_per_step": w["stats"]["median"], "repeats": w["stats"],
                 "compressed_elems_per_s": job_throughput(elems_per_step, 1, w["stats"]["median"], world),
                 "level_histogram": w["level_histogram"], "levels_last_step": w["levels_last_step"],
                 "step_roofline": w["step_roofline"], "kernels": kernel_table(w["prof"], args.steps)}
        del w

    # end to end through the host entry point: pinned host buffers, copies inside the timed region
    e2e = None
    if args.e2e_steps > 0:
        G, gt, gm, state = main["state"]
        t = state["t"]
        hX = [x.cpu().pin_memory() for x in Xs]
        hG = G.cpu().pin_memory()
        hgt = [gt[0].cpu().pin_memory(), gt[1].cpu().pin_memory()]
        hgm = gm.cpu().pin_memory()
        hlevel = torch.zeros(n, dtype=torch.int32).pin_memory()
        hbits = torch.zeros(n, dtype=torch.int64).pin_memory()

        def host_step(tt):
            cur, nxt = hgt[tt % 2], hgt[(tt + 1) % 2]
            eng.compress_host(hX[tt % P], hG, hX[(tt - 1) % P], mean_out=nxt, level=hlevel, bits=hbits)
            eng.compress_host(nxt.view(1, d), hgm, cur.view(1, d), W["master"], args.zeta)

        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        host_step(t)
        barrier_sync(world)
        e0.record()
        for k in range(args.e2e_steps):
            host_step(t + 1 + k)
        e1.record()
        barrier_sync(world)
        ems = max_over_ranks(e0.elapsed_time(e1), world)
        h2d = 3 * n * d * 4 + 3 * d * 4
        d2h = n * d * 4 + d * 4 + n * 12 + d * 4
        e2e = {"value": world * elems_per_step * args.e2e_steps / (ems * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "ms_per_step": ems / args.e2e_steps}
    return dict(value=value, ms=ms, launches=main["launches"], roofline=roofline, step_roofline=main["step_roofline"],
                kernels=kernel_table(prof, args.steps), clocks=main["clocks"], e2e=e2e, repeats=main["stats"], worst_case=worst,
                iters_per_s=world * args.steps / (ms * 1e-3), rechecks=eng.get_state("rechecks"),
                side_paths={"fallback_rows": eng.get_state("fallbacks"), "list_level_rows": eng.get_state("list_levels")},
                config={"workload": "c5", "n": n, "d": d, "topk": [p for _, p in W["worker"]],
                        "master_topk": [p for _, p in W["master"]], "zeta": args.zeta,
                        "levels_last_step": main["levels_last_step"], "level_histogram": main["level_histogram"],
                        "l2": "inputs (3 x %.0f MB per pass) exceed the 126 MB L2; no flush needed" % (n * d * 4 / 1e6),
                        "replicas": world})


def bench_dense(args, name, rank, world, local, steps=None, warmup=None, repeats=None, incremental=False, k_scale=1.0):
    import torch
    import paper_2211_00188_b200 as pkg

    W = dict(S.WORKLOADS[name])
    if k_scale != 1.0:   # the same workload with a ladder of smaller Top-K sizes
        W["worker"] = [(k, max(1, int(p * k_scale)) if k == 0 else p) for k, p in W["worker"]]
        W["master"] = [(k, max(1, int(p * k_scale)) if k == 0 else p) for k, p in W["master"]]
    n, d, m = (args.workers or W["n"]), W["d"], W["m"]
    dev = torch.device("cuda", local)
    steps = steps or args.steps
    warmup = warmup or args.warmup
    repeats = repeats or args.repeats
    csr = None
    if name == "c4":  # 16.4 GB of features: drawn on the device with the same law
        gen = torch.Generator(device=dev)
        gen.manual_seed(rank)
        A = torch.empty(n, m, d, device=dev)
        for i in range(n):
            A[i] = torch.randn(m, d, generator=gen, device=dev) / d ** 0.5
        xs = torch.randn(d, generator=gen, device=dev)
        tgt = torch.einsum("nmd,d->nm", A, xs) + 0.1 * torch.randn(n, m, generator=gen, device=dev)
        # Gaussian features: lambda_max of the stacked (n m) x d matrix is about (1 + sqrt(n m / d))^2
        gamma = 0.5 / ((1.0 + (n * m / d) ** 0.5) ** 2 / (n * m))
    elif W["layout"] == "csr":
        rowptr, col, val, th = S.sparse_logistic_problem(n, d, m, density=W["density"], seed=rank)
        csr = tuple(torch.from_numpy(a).to(dev) for a in S.csr_global(rowptr, col, val))
        A, tgt = None, torch.from_numpy(th).to(dev)
        gamma = 0.5 / (0.25 + W["lam"])   # unit-norm rows: lambda_max(A^T A)/m <= 1
    else:
        if W["loss"] == 2:
            Ah, th, _ = S.least_squares_problem(n, d, m, seed=rank)
        else:
            Ah, th = S.logistic_problem(n, d, m, seed=rank)
        gamma = 0.5 / S.smoothness_estimate(Ah, W["loss"], W["lam"], iters=8)
        A, tgt = torch.from_numpy(Ah).to(dev), torch.from_numpy(th).to(dev)
    x0 = torch.zeros(d, device=dev)
    eng = pkg.AdaCGD(n, d, W["worker"], 1.0, W["master"], 1.0, loss=W["loss"], lam=W["lam"], A=A, target=tgt,
                     csr=csr, x0=x0, gamma=gamma, device=dev, incremental_forward=incremental)
    eng.step(warmup)
    cols0 = eng.get_state("inc_columns") if incremental else 0
    refr0 = eng.get_state("refreshes") if incremental else 0
    launches0 = eng.launch_count()
    times, clocks = timed_repeats(lambda k: eng.step(k), steps, repeats, world, local)
    launches = (eng.launch_count() - launches0) // repeats
    st = repeat_stats(times, steps)
    ms = st["median"] * steps
    inc_info = None
    if incremental:
        its = steps * repeats
        cols = (eng.get_state("inc_columns") - cols0) / its
        refr = (eng.get_state("refreshes") - refr0) / its
        # features read per iteration: the backward pass in full, a full forward pass (twice: z and u) at a
        # refresh, and the gathered columns of the column-major copy otherwise
        inc_info = {"changed_entries_of_g_per_iteration": cols, "refreshes_per_iteration": refr,
                    "feature_bytes_per_iteration": 4 * n * m * (d + 2 * d * refr + cols),
                    "feature_bytes_per_iteration_full_forward": 8 * n * m * d}
    # the same number of steps once more with the library's per-kernel CUDA-event timers switched on
    eng.profile_enable(80 * steps + 64)
    eng.step(steps)
    prof = eng.profile_read()
    eng.profile_enable(0)
    recs, levels = eng.step(1, report=True)
    elems_per_step = n * d + (d if W["master"] else 0)
    value = job_throughput(elems_per_step, steps, ms, world)
    peak, peak_src = measured_peaks()
    # one pass over the features: dense 4 B per entry; CSR value + column index per stored entry
    a_bytes = 4 * n * m * d if csr is None else 8 * int(csr[1].numel())
    top = max((k for k in ("k_dense_fwd", "k_dense_bwd", "k_csr_fwd", "k_csc_bwd") if k in prof), key=lambda k: prof[k][0])
    achieved = a_bytes * prof[top][1] / (prof[top][0] * 1e-3) / 1e9
    per_entry = counted_traffic(top)   # counted DRAM bytes per feature entry (dense) or stored entry (CSR)
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": None if per_entry is None else per_entry * a_bytes / (4 if csr is None else 8),
                "peak_source": peak_src, "launches": prof[top][1],
                "avg_launch_ms": prof[top][0] / prof[top][1]}
    floor = 2 * a_bytes + 20 * n * d + (24 * d if W["master"] else 0)
    step_gbs = floor / (ms / steps * 1e-3) / 1e9
    step_roofline = {"algorithmic_bytes_per_step": floor, "achieved_gbs": step_gbs, "frac": step_gbs / peak,
                     "frac_of_nominal_7700": step_gbs / NOMINAL_HBM_GBS}
    hist = {}
    for l in levels[0]:
        hist[str(l)] = hist.get(str(l), 0) + 1
    return dict(value=value, ms=ms, steps=steps, launches=launches, roofline=roofline, step_roofline=step_roofline,
                kernels=kernel_table(prof, steps), clocks=clocks, e2e=None, repeats=st, worst_case=None,
                iters_per_s=world * steps / (ms * 1e-3), rechecks=eng.get_state("rechecks"),
                side_paths={"fallback_rows": eng.get_state("fallbacks"), "list_level_rows": eng.get_state("list_levels")},
                config={"workload": name, "n": n, "d": d, "m": m, "loss": W["loss"], "gamma": gamma,
                        "cands": [list(c) for c in W["worker"]], "bidirectional": bool(W["master"]),
                        "loss_after": recs[0]["loss"], "level_histogram_last_step": hist, "incremental_forward": inc_info,
                        "l2": ("features (%.2f GB) exceed the 126 MB L2" % (a_bytes / 1e9)) if a_bytes > 2e8
                        else "working set fits in L2 (launch-latency bound workload)", "replicas": world})


FULL_ITERATION_RUNS = {"c1": (400, 20), "c2": (200, 20), "c3": (100, 10), "c4": (30, 5)}   # workload: (steps, warm-up)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps steps; value is their median")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c5", "c4", "c3", "c2", "c1"])
    ap.add_argument("--zeta", type=float, default=1.0)
    ap.add_argument("--scale", type=float, default=1.0, help="shrink d of workload c5 (profiling captures)")
    ap.add_argument("--workers", type=int, default=0, help="fewer workers for workloads c1-c4 (profiling captures)")
    ap.add_argument("--incremental", action="store_true", help="workloads c1, c2, c4: keep the forward products between iterations")
    ap.add_argument("--k-scale", type=float, default=1.0, help="workloads c1-c4: scale the Top-K sizes of the candidate lists")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the worst-case and the full-iteration measurements")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)
    args.repeats = max(args.repeats, 1)

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    rank, world, local = dist_setup()

    if args.workload == "c5":
        res = bench_c5(args, rank, world, local)
    else:
        res = bench_dense(args, args.workload, rank, world, local, incremental=args.incremental, k_scale=args.k_scale)
    ms_per_step = res["ms"] / args.steps

    extra = None
    if args.workload == "c5" and not args.no_extra and args.scale == 1.0:
        extra = []
        for name, (steps, warm) in FULL_ITERATION_RUNS.items():
            torch.cuda.empty_cache()
            r2 = bench_dense(args, name, rank, world, local, steps=steps, warmup=warm, repeats=3)
            extra.append({"workload": name, "what": "full iterations a0-a5 through adacgd_step", "steps": steps,
                          "iters_per_s": r2["iters_per_s"], "ms_per_step": r2["ms"] / r2["steps"], "repeats": r2["repeats"],
                          "compressed_elems_per_s": r2["value"], "roofline": r2["roofline"],
                          "step_roofline": r2["step_roofline"], "kernels": r2["kernels"], "config": r2["config"],
                          "gpu_launches": r2["launches"], "exact_rechecks": r2["rechecks"], "side_paths": r2["side_paths"],
                          "clocks": r2["clocks"]})
            del r2
        # the forward products kept between iterations: workloads c2 and c4 as they are (most entries of g move every
        # iteration there, so the pass mostly recomputes) and c4 with a ladder of Top-K sizes a hundred times smaller,
        # with and without the incremental pass
        for name, ks, inc in (("c2", 1.0, True), ("c4", 1.0, True), ("c4", 0.01, False), ("c4", 0.01, True)):
            torch.cuda.empty_cache()
            steps, warm = FULL_ITERATION_RUNS[name]
            r2 = bench_dense(args, name, rank, world, local, steps=steps + 2, warmup=warm, repeats=3, incremental=inc, k_scale=ks)
            extra.append({"workload": name, "what": "full iterations, " + ("incremental forward pass (refresh period 16)" if inc else "full forward pass")
                          + (", Top-K sizes x %g" % ks if ks != 1.0 else ""),
                          "steps": r2["steps"], "iters_per_s": r2["iters_per_s"], "ms_per_step": r2["ms"] / r2["steps"],
                          "repeats": r2["repeats"], "compressed_elems_per_s": r2["value"], "kernels": r2["kernels"],
                          "config": r2["config"], "gpu_launches": r2["launches"], "clocks": r2["clocks"]})
            del r2

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        W = S.WORKLOADS[args.workload]
        rate, dt, sample = (oracle_sample_c5(W, 20.0) if args.workload == "c5" else oracle_sample_dense(W, 20.0))
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample, "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "gpu_launches": res["launches"],
            "config": res["config"], "side_paths": res["side_paths"], "exact_rechecks": res["rechecks"],
            "repeats": res["repeats"], "iters_per_s": res["iters_per_s"], "roofline": res["roofline"],
            "step_roofline": res["step_roofline"], "clocks": res["clocks"], "e2e": res["e2e"], "cpu_baseline": cpu,
            "kernels": res["kernels"],
        }
        if res["worst_case"]:
            line["worst_case"] = res["worst_case"]
        if extra:
            line["full_iteration"] = extra
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
