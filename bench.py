#!/usr/bin/env python
"""Benchmark: full-graph sliced-GCN training throughput (epochs/s) and SpMM bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload citation] [--impl ours|reference]

One "step" is one training epoch (Algorithm 3 of the paper: forward over every slice, loss,
backward, one Adam update) on a seeded synthetic graph.  With N > 1 (launched under torchrun) every
rank trains an independent replica: the single-GPU path has no sharding and no collectives, so
`value` is the number of epochs all replicas finish per second (weak scaling).
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2408_11500_b200 import synth  # noqa: E402

# Every SPMM_SAMPLE_STRIDE-th SpMM call inside the timed region is bracketed by CUDA events (an event pair costs the
# stream ~10 us; bracketing all five calls of an epoch would add ~4 % to the step time).  7 is coprime to the 4-6 SpMM
# calls of an epoch, so every call site is sampled equally often.
SPMM_SAMPLE_STRIDE = 7


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        self.t0 = self.t1 = None          # the timed region; only samples taken inside it are used

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [t.strip() for t in line.split(",")]))

    def wait_first_sample(self, limit_s: float = 10.0):
        """nvidia-smi needs a moment to start; a short timed region would otherwise end before its first line."""
        t = time.time()
        while self.proc is not None and not self.rows and time.time() - t < limit_s:
            time.sleep(0.02)

    def samples_inside(self) -> int:
        return sum(1 for (t, _) in self.rows if self.t0 is not None and self.t0 <= t <= (self.t1 or time.time()))

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for (t, r) in self.rows if self.t0 is not None and self.t0 <= t <= (self.t1 or t) + 0.15]
        for r in (inside if inside else [r for (_, r) in self.rows[-3:]]):
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            for nm, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def scaled_workload(name: str, frac: float) -> dict:
    w = dict(synth.WORKLOADS[name])
    if frac < 1.0:
        w["n"] = max(int(w["n"] * frac), 64)
        w["m"] = max(int(w["m"] * frac), 64)
        if "max_degree" in w:
            w["max_degree"] = max(w["max_degree"] * frac, 16)
    return w


def model_kwargs(w: dict) -> dict:
    return dict(in_d=w["in_d"], hidden=w["hidden"], num_layers=w["layers"], num_classes=w["classes"],
                num_slices=w["p"], use_ff=w["use_ff"], use_se=w["use_se"])


# ---------------------------------------------------------------------------------- oracle timing

def oracle_epochs(w: dict, epochs: int, warm: int, single_thread: bool = False):
    """Times the CPU oracle, as it stands, on workload w.  Returns (seconds per epoch list, threads).
    single_thread: one OpenMP thread in the neighbor sum and one BLAS thread in the dense products."""
    from oracle import slicegcn_oracle as orc
    if single_thread:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            times, _ = oracle_epochs_impl(orc, w, epochs, warm, 1)
        return times, 1
    return oracle_epochs_impl(orc, w, epochs, warm, len(os.sched_getaffinity(0)))   # every core this process may use


def oracle_epochs_impl(orc, w: dict, epochs: int, warm: int, threads: int):
    src, dst = synth.make_graph(w, 0)
    X = synth.make_features(w, 0).astype(np.float64)
    y = synth.uniform_labels(w["n"], w["classes"], 0)
    od = orc.ModelDesc(w["in_d"], w["hidden"], w["layers"], w["classes"], p=w["p"], use_ff=w["use_ff"], use_se=w["use_se"])
    rnd = orc.round_bf16 if w["dtype"] == "bf16" else orc.identity
    if w["dtype"] == "bf16":
        X = orc.round_bf16(X)
    P = {k: v.astype(np.float64) for k, v in synth.init_params(orc.param_shapes(od), 0).items()}
    g = orc.build_graph(w["n"], src, dst, True, True)
    st = {"m1": {}, "m2": {}}
    times = []
    for ep in range(warm + epochs):
        t0 = time.perf_counter()
        orc.train_epoch(od, g, X, P, y, st, 1e-3, ep, max(warm + epochs, 2), rnd=rnd, threads=threads)
        if ep >= warm:
            times.append(time.perf_counter() - t0)
    return times, (threads if threads > 0 else orc.max_threads())


class SweepOracleLeg:
    """CPU-baseline leg of the SpMM sweep (`--sweep`): exact oracle values on a seeded sample of rows that includes the
    100 longest, and the oracle's own time on that sample scaled by (stored entries of the graph) / (entries of the
    sampled rows) -- an extrapolation, labelled as such in the table."""

    def __init__(self, n, src, dst, rows_wanted):
        from oracle import slicegcn_oracle as orc
        self.orc = orc
        self.g = orc.build_graph(n, src, dst, True, True)
        longest = np.argsort(self.g.deg, kind="stable")[-100:]
        rnd = np.random.default_rng(0).choice(n, size=min(rows_wanted, n), replace=False)
        self.rows = np.unique(np.concatenate([longest, rnd])).astype(np.int64)
        self.entries = int(self.g.deg[self.rows].astype(np.int64).sum())

    def check(self, X_dev, Y_rows, dtype_name):
        X = X_dev.float().cpu().numpy().astype(np.float64)
        t0 = time.perf_counter()
        want = self.orc.spmm(self.g, X, rows=self.rows)
        dt = time.perf_counter() - t0
        if dtype_name == "f32":
            err = float(np.abs(Y_rows - want).max() / np.abs(want).max())
            ok = err <= 2e-6
        else:   # one bf16 rounding of the fp32-accumulated result
            err = float((np.abs(Y_rows - want) / (np.abs(want) + 1e-5 * np.abs(want).max())).max())
            ok = bool(np.all(np.abs(Y_rows - want) <= 2 ** -8 * np.abs(want) + 1e-5 * np.abs(want).max()))
        return {"err": err, "ok": ok, "rows": int(self.rows.size), "threads": self.orc.max_threads(),
                "cpu_ms": 1e3 * dt * self.g.nnz / max(self.entries, 1)}


def run_reference(args, rank: int):
    """--impl reference: the oracle on the host cores, on a bounded sample of the same workload."""
    if rank != 0:
        return
    if args.steps <= 0:
        args.steps = 3
    total_steps = args.steps + args.warmup
    full_epoch_s = {"tiny": 0.4, "citation": 20.0, "social": 600.0, "copurchase": 900.0}[args.workload]
    frac = 1.0
    while frac > 1 / 512 and full_epoch_s * frac * total_steps > 150.0:
        frac /= 2
    w = scaled_workload(args.workload, frac)
    times, threads = oracle_epochs(w, args.steps, args.warmup)
    ms = 1e3 * sum(times) / len(times)
    value = (1e3 / ms) * frac              # linear extrapolation to the full workload
    sample = (f"{args.steps} epochs of the same generator at {frac:g} of the nodes and edges "
              f"(n={w['n']}), epochs/s scaled by {frac:g}") if frac < 1 else f"{args.steps} full epochs"
    line = {"impl": "reference", "metric": "full-graph GCN training throughput", "value": value, "unit": "epochs/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / frac,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample_fraction": frac},
            "cpu_baseline": {"value": value, "unit": "epochs/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "epochs/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------- CUDA path

# DRAM traffic of the dominant SpMM launch (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture, per launch),
# with the committed summary each figure comes from; None where no capture exists.
NCU_SPMM_TRAFFIC = {
    "citation": (897e6, "profiles/spmm_rows_kernel_citation_w256.md (fp32 width-256 launch: every SpMM of a steady-state epoch)"),
    "copurchase": (38.1e9, "profiles/spmm_sweep_rmat.md (bf16 width-256 forward launch, 4 of the 6 per epoch; single-pass capture)"),
    "social": (12.0e9, "profiles/spmm_sweep_rmat.md (fp32 width-256 launch, all 4 per epoch alike)"),
}
DEFAULT_STEPS = {"tiny": 200, "citation": 200, "social": 20, "copurchase": 20}
DEFAULT_CPU_FRACTION = {"tiny": 1.0, "citation": 1.0, "social": 1 / 16, "copurchase": 1 / 16}


def max_over_ranks(x: float, world: int, dist=None, device=None, torch=None) -> float:
    """The slowest rank's elapsed time: the only cross-rank reduction of a replica run (after a barrier)."""
    if world == 1:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, steps: int, elapsed_ms: float) -> float:
    """Epochs all replicas finished per second of the slowest replica's time."""
    return world * steps / (elapsed_ms / 1e3)


def measure(workload: str, steps: int, warmup: int, world: int, local_rank: int, with_e2e: bool, dist=None, fraction: float = 1.0):
    """Device-resident timing (and, if asked, the end-to-end run from host buffers) of one workload.
    Returns the fields of the JSON line that depend on the workload.  fraction < 1 shrinks the graph (same generator,
    that share of the nodes and edges): a profiling aid for counter captures, which must stay on small cases."""
    import torch
    from paper_2408_11500_b200 import binding as B

    dev = torch.device("cuda", local_rank)
    w = scaled_workload(workload, fraction)
    src, dst = synth.make_graph(w, 0)
    Xh = synth.make_features(w, 0)
    yh = synth.uniform_labels(w["n"], w["classes"], 0)
    n = w["n"]
    dtype = B.BF16 if w["dtype"] == "bf16" else B.F32
    tdt = torch.bfloat16 if dtype == B.BF16 else torch.float32
    g = B.slicegcn_graph_create(n, src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    del src, dst
    info = B.slicegcn_graph_info(g)
    # The features are sliced once, outside the epoch loop (Algorithm 3): with X resident on the device the first
    # layer's aggregate is kept across epochs.  (The end-to-end run copies X anew every epoch and recomputes it.)
    m = B.slicegcn_model_create(dtype=dtype, cache_input_aggregate=True, **model_kwargs(w))
    params0 = torch.from_numpy(B.pack_params(m, synth.init_params(B.named_param_shapes(m), 0))).to(dev)
    params = params0.clone()
    grads, m1, m2 = torch.zeros_like(params), torch.zeros_like(params), torch.zeros_like(params)
    ws_bytes = B.slicegcn_train_workspace_bytes(m, g)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    X = torch.from_numpy(Xh).to(dev).to(tdt).contiguous()
    y = torch.from_numpy(yh).to(dev)
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    total_epochs = 500                        # the paper's schedule length (Table II); sets the cosine period

    def epoch(ep, Xd, yd):
        B.slicegcn_train_epoch(m, g, Xd, w["in_d"], yd, None, 0, params, grads, m1, m2,
                               B.make_opt_desc(1e-3, ep, total_epochs), None, loss, ws, ws_bytes, stream.cuda_stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    mor = lambda x: max_over_ranks(x, world, dist, dev, torch)

    # ---- device-resident run
    sampler = ClockSampler(local_rank)
    sampler.start()
    for ep in range(warmup - 1):
        epoch(ep, X, y)
    B.slicegcn_profile_begin()                 # the last warm-up epoch counts the SpMM calls and launches of one epoch
    epoch(warmup - 1, X, y)
    per_epoch = B.slicegcn_profile_end()
    sampler.wait_first_sample()
    barrier()
    sampler.mark_begin()
    B.slicegcn_profile_begin_sampled(SPMM_SAMPLE_STRIDE)   # CUDA events around every 7th SpMM call of the timed region
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record(stream)
    for ep in range(steps):
        epoch(warmup + ep, X, y)
        ev[ep + 1].record(stream)
    barrier()
    prof = B.slicegcn_profile_end()
    ms_total = mor(ev[0].elapsed_time(ev[-1]))
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    final_loss = float(loss.item())
    # A timed region shorter than a few sampling periods holds too few clock samples: keep the same load running
    # (untimed, on copies of the optimizer state) until the sampler has seen at least three.
    clock_extension = 0
    if sampler.proc is not None and sampler.samples_inside() < 3:
        keep = [t.clone() for t in (params, grads, m1, m2, loss)]
        t_ext = time.time()
        while sampler.samples_inside() < 3 and time.time() - t_ext < 3.0:
            for ep in range(8):
                epoch(warmup + steps + clock_extension + ep, X, y)
            torch.cuda.synchronize()
            clock_extension += 8
        for t, k in zip((params, grads, m1, m2, loss), keep):
            t.copy_(k)
        torch.cuda.synchronize()
    sampler.mark_end()
    clocks = sampler.stop()
    if clock_extension:
        clocks["note"] = (f"timed region of {ms_total:.0f} ms is shorter than three sampling periods: sampled over it and "
                          f"{clock_extension} further untimed epochs of the same load")

    peak, peak_src = measured_peak_gbs()
    spmm_avg_ms = prof["spmm_ms"] / max(prof["spmm_calls"], 1)
    achieved = (prof["spmm_bytes"] / 1e9) / (prof["spmm_ms"] / 1e3) if prof["spmm_ms"] > 0 else 0.0
    traffic, traffic_src = NCU_SPMM_TRAFFIC.get(workload, (None, None)) if fraction >= 1.0 else (None, None)
    ms_per_step = ms_total / steps
    out = {
        "value": whole_job_rate(world, steps, ms_total), "ms_per_step": ms_per_step,
        "ms_per_step_median": statistics.median(step_ms), "ms_per_step_min": min(step_ms),
        "dtype": "f32" if dtype == B.F32 else "bf16",
        "config": {"workload": workload, "nodes": n, "nnz": info["nnz"], "in_d": w["in_d"], "hidden": w["hidden"],
                   "layers": w["layers"], "classes": w["classes"], "num_slices": w["p"], "use_ff": w["use_ff"],
                   "use_se": w["use_se"], "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "working set per epoch is larger than L2 (no flush needed)", "final_loss": final_loss,
                   "input_aggregate_cached": bool(not w["use_ff"]), "fraction_of_workload": fraction},
        "clocks": clocks,
        "gpu_launches": int(prof["kernel_launches"]),
        "roofline": {"bound": "hbm", "kernel": "spmm_rows_kernel",
                     "achieved": achieved, "peak": peak, "peak_source": f"of {peak_src}", "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
                     "launches": int(prof["spmm_calls"]), "sampled_every": SPMM_SAMPLE_STRIDE, "avg_ms": spmm_avg_ms,
                     "algorithmic_bytes_per_launch": prof["spmm_bytes"] / max(prof["spmm_calls"], 1),
                     "spmm_calls_per_step": int(per_epoch["spmm_calls"]),
                     "share_of_step": spmm_avg_ms * per_epoch["spmm_calls"] / ms_per_step},
    }

    if with_e2e:
        # ---- end to end: ONE C-ABI call runs the epochs from host buffers.  Every epoch copies X and the
        # labels from page-locked host memory again and returns its loss to the host; the library overlaps the
        # copy for epoch e+1 with the kernels of epoch e (two staging buffers).
        Xp = (torch.from_numpy(Xh).to(tdt) if dtype == B.BF16 else torch.from_numpy(Xh)).pin_memory()
        yp = torch.from_numpy(yh).pin_memory()
        n_e2e = max(steps, warmup, 1)
        losses_host = torch.zeros(n_e2e, dtype=torch.float32).pin_memory()
        losses_dev = torch.zeros(n_e2e, dtype=torch.float32, device=dev)
        Xd = [torch.empty_like(X), torch.empty_like(X)]
        yd = [torch.empty_like(y), torch.empty_like(y)]
        params.copy_(params0); m1.zero_(); m2.zero_()

        def e2e_run(first_epoch, count):
            B.slicegcn_train_epochs_host(m, g, Xp, w["in_d"], yp, Xd[0], Xd[1], yd[0], yd[1], None, 0, params, grads, m1, m2,
                                         B.make_opt_desc(1e-3, first_epoch, total_epochs), count, losses_dev, losses_host,
                                         ws, ws_bytes, stream.cuda_stream)

        e2e_run(0, max(warmup, 1))
        barrier()
        t0 = time.perf_counter()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        e2e_run(warmup, steps)          # returns after the last loss has reached the host
        f1.record(stream)
        barrier()
        e2e_ms = mor(max(f0.elapsed_time(f1), 1e3 * (time.perf_counter() - t0)))
        if not all(np.isfinite(losses_host[:steps].numpy())):
            raise SystemExit("end-to-end run produced a non-finite loss")
        out["e2e"] = {"value": whole_job_rate(world, steps, e2e_ms), "unit": "epochs/s",
                      "h2d_bytes_per_step": Xp.numel() * Xp.element_size() + yp.numel() * 4, "d2h_bytes_per_step": 4}
    B.slicegcn_model_destroy(m)
    B.slicegcn_graph_destroy(g)
    del ws, X, y, params, grads, m1, m2
    torch.cuda.empty_cache()
    return out


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    import torch.distributed as dist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    steps = args.steps if args.steps > 0 else DEFAULT_STEPS[args.workload]
    main_part = measure(args.workload, steps, args.warmup, world, local_rank, True, dist, args.fraction)
    line = {"metric": "full-graph GCN training throughput", "value": main_part.pop("value"), "unit": "epochs/s",
            "n_gpus": world, "steps": steps, "warmup": args.warmup, "ms_per_step": main_part.pop("ms_per_step"),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "data": "synthetic"}
    line.update(main_part)
    # the other model workloads, device-resident timing only (one line covers all three)
    if world == 1 and not args.no_secondary and args.fraction >= 1.0:
        line["secondary"] = []
        for name in [k for k in ("citation", "social", "copurchase") if k != args.workload]:
            part = measure(name, DEFAULT_STEPS[name] if args.steps <= 0 else min(DEFAULT_STEPS[name], max(args.steps, 5)),
                           args.warmup, 1, local_rank, False)
            line["secondary"].append({"workload": name, "value": part["value"], "unit": "epochs/s",
                                      "ms_per_step": part["ms_per_step"], "ms_per_step_median": part["ms_per_step_median"],
                                      "ms_per_step_min": part["ms_per_step_min"], "dtype": part["dtype"],
                                      "nodes": part["config"]["nodes"], "nnz": part["config"]["nnz"],
                                      "clocks": part["clocks"], "roofline": part["roofline"]})
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        frac = args.cpu_fraction if args.cpu_fraction > 0 else DEFAULT_CPU_FRACTION[args.workload]
        cw = scaled_workload(args.workload, frac)
        times, threads = oracle_epochs(cw, 1, 0)
        v = frac / times[0]
        sample = ("1 full epoch of the same workload" if frac >= 1 else
                  f"1 epoch of the same generator at {frac:g} of the nodes and edges (n={cw['n']}), epochs/s scaled by {frac:g}")
        line["cpu_baseline"] = {"value": v, "unit": "epochs/s", "cores": threads, "kind": "oracle", "sample": sample}
        # the same oracle on ONE thread, on a quarter of that sample (it is ~10x slower)
        f1 = frac / 4
        c1 = scaled_workload(args.workload, f1)
        t1, _ = oracle_epochs(c1, 1, 0, single_thread=True)
        line["cpu_baseline"]["single_thread"] = {"value": f1 / t1[0], "unit": "epochs/s", "cores": 1,
                                                 "sample": f"1 epoch at {f1:g} of the nodes and edges (n={c1['n']}), scaled"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed epochs (0: a default per workload that runs a second or two)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="copurchase", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--cpu-fraction", type=float, default=0.0, help="size of the oracle's timed sample (0: a default per workload)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the device-resident timing of the other workloads")
    ap.add_argument("--fraction", type=float, default=1.0,
                    help="shrink the workload to this share of its nodes and edges (profiling aid: not the benchmark configuration)")
    ap.add_argument("--sweep", action="store_true",
                    help="the SpMM kernel sweep on R-MAT graphs with the oracle's leg; the remaining arguments are spmm_sweep.py's")
    args, rest = ap.parse_known_args()
    if args.sweep:
        import spmm_sweep
        spmm_sweep.main(rest, oracle_leg=SweepOracleLeg)
        return
    if rest:
        ap.error("unrecognised arguments: " + " ".join(rest))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
