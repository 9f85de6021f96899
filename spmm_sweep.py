"""SpMM kernel sweep on R-MAT graphs: rates per feature width against the HBM copy peak.

R-MAT (a, b, c) = (0.57, 0.19, 0.19), edge factor 16, self pairs dropped, repeats merged, symmetrized,
self-loops added, int32 CSR; node ids as generated ("natural": hubs at low ids) and under a seeded random
relabeling.  For every (graph, dtype, width) the aggregation Y = A_hat X runs `reps` times, each launch between
its own pair of CUDA events, back to back and with L2 flushed before every launch; the median, the minimum and the
flushed median are printed, and three rates from the median:

    algorithmic   (4 nnz + 4 (N+1) + 4 N + 2 N w e) / t     each array once -- the roofline numerator
    gathered      nnz w e / t                                what the SMs request from L2
    fraction      algorithmic / measured copy peak

Every case is also checked at full size without a reference run: with X = sqrt(deg) in every column the
normalized aggregation returns sqrt(deg) again (row i sums deg_i terms sqrt(deg_j) / (sqrt(deg_i) sqrt(deg_j))),
so max |Y / sqrt(deg) - 1| must stay at rounding level.  The pattern is symmetric, so the transposed pass of
the backward runs the same launch.

    python spmm_sweep.py --scales 20,22 --widths 16,32,64,128,256,512 --dtypes f32,bf16

This file holds the CUDA-side measurement only.  `python bench.py --sweep ...` runs the same cases and adds the CPU
oracle's leg: exact values on a seeded sample of rows (the 100 longest included) and the oracle's own time on that
sample, extrapolated to the whole graph.
"""
from __future__ import annotations

import argparse
import json
import os
import time

import numpy as np


def copy_peak_gbs() -> float:
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"])
    return 6650.0


def run_case(B, torch, g, info, deg_dev, width, dtype_name, reps, budget_bytes, flush_buf=None, sample_rows=None):
    """Times one (graph, dtype, width) case and checks the identity.  With sample_rows (int64 row ids) the result also
    carries "X" (the Gaussian operand on the device) and "Y_rows" (the sampled output rows, fp32 on the host)."""
    n, nnz = info["n"], info["nnz"]
    tdt, bdt, e = (torch.float32, B.F32, 4) if dtype_name == "f32" else (torch.bfloat16, B.BF16, 2)
    if 2 * n * width * e > budget_bytes:
        return None
    st = torch.cuda.current_stream()
    wsb = B.slicegcn_spmm_workspace_bytes(g, width)
    ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
    X = torch.empty(n, width, dtype=tdt, device="cuda")
    Y = torch.empty_like(X)

    def spmm():
        B.slicegcn_spmm(g, 0, bdt, bdt, X, width, Y, width, width, ws, wsb, st.cuda_stream)

    # identity check at full size
    root = deg_dev.to(torch.float32).sqrt()
    X.copy_(root.to(tdt)[:, None].expand(n, width))
    spmm()
    torch.cuda.synchronize()
    # compare with what the kernel was given (sqrt(deg) after rounding to the storage type)
    err = 0.0
    step = max(1, (1 << 28) // width)                       # row blocks: no full-size fp32 temporaries
    for r in range(0, n, step):
        q = Y[r:r + step].to(torch.float32) / X[r:r + step].to(torch.float32) - 1.0
        err = max(err, float(q.abs().max().item()))
    # timing on Gaussian features: every launch between its own pair of events; back to back ("warm": whatever
    # the previous launch left in L2 stays) and with L2 flushed before each launch (a write larger than L2)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(width)
    X.normal_(generator=gen)
    for _ in range(3):
        spmm()
    torch.cuda.synchronize()

    def timed(flush):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in ev:
            if flush is not None:
                flush.zero_()
            a.record(st)
            spmm()
            b.record(st)
        torch.cuda.synchronize()
        return sorted(a.elapsed_time(b) for a, b in ev)

    warm = timed(None)
    cold = timed(flush_buf) if flush_buf is not None else warm
    ms = warm[len(warm) // 2]
    alg = 4.0 * nnz + 4.0 * (n + 1) + 4.0 * n + 2.0 * n * width * e
    extra = {}
    if sample_rows is not None:
        extra = {"X": X, "Y_rows": Y[torch.from_numpy(sample_rows).cuda()].to(torch.float32).cpu().numpy()}
    return {**extra, "ms": ms, "ms_min": warm[0], "ms_flushed": cold[len(cold) // 2], "alg_gbs": alg / ms / 1e6,
            "gather_gbs": float(nnz) * width * e / ms / 1e6, "identity_err": err}


def main(argv=None, oracle_leg=None):
    """oracle_leg(n, src, dst, rows_wanted) -> checker with .rows and .check(X_dev, Y_rows, dtype_name) -> dict, or None:
    supplied by bench.py --sweep (this module never touches the oracle)."""
    import torch
    from paper_2408_11500_b200 import binding as B, synth
    ap = argparse.ArgumentParser()
    ap.add_argument("--scales", default="20")
    ap.add_argument("--widths", default="16,32,64,128,256,512")
    ap.add_argument("--dtypes", default="f32,bf16")
    ap.add_argument("--ids", default="natural,relabeled")
    ap.add_argument("--reps", type=int, default=10, help="timed launches per case (median reported)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--max-gb", type=float, default=100.0, help="skip cases whose X and Y together exceed this")
    ap.add_argument("--oracle-rows", type=int, default=10000, help="(bench.py --sweep) rows of the oracle's sample")
    ap.add_argument("--oracle-max-gb", type=float, default=6.0, help="(bench.py --sweep) largest operand the oracle leg copies to the host")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device (there is no CPU path)")
    peak = copy_peak_gbs()
    widths = [int(v) for v in args.widths.split(",")]
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # twice the L2
    print(f"copy peak {peak:,.0f} GB/s; 3 warm-up and {args.reps} timed launches per case (median; rates from the median)\n")
    print("| scale | ids | N | nnz | long-row segments | dtype | width | us (median) | us (min) | us (L2 flushed) | "
          "algorithmic GB/s | of copy peak | gathered GB/s | identity err |" +
          (" sampled rows vs oracle | oracle ms (extrapolated from the sample) |" if oracle_leg else ""))
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|" + ("---|---|" if oracle_leg else ""))
    for scale in (int(v) for v in args.scales.split(",")):
        t0 = time.time()
        n, src, dst = synth.rmat(scale, 16, seed=args.seed)
        gen_s = time.time() - t0
        for ids in args.ids.split(","):
            s, d = (src, dst) if ids == "natural" else synth.random_relabel(n, src, dst, args.seed)
            g = B.slicegcn_graph_create(n, np.ascontiguousarray(s), np.ascontiguousarray(d),
                                        B.SYMMETRIZE | B.ADD_SELF_LOOPS)
            try:
                info = B.slicegcn_graph_info(g)
                deg_dev = torch.from_numpy(B.slicegcn_graph_degrees(g)).cuda()
                checker = oracle_leg(n, s, d, args.oracle_rows) if oracle_leg else None
                for dtype_name in args.dtypes.split(","):
                    for width in widths:
                        e = 4 if dtype_name == "f32" else 2
                        with_oracle = checker is not None and n * width * e <= args.oracle_max_gb * 1e9
                        r = run_case(B, torch, g, info, deg_dev, width, dtype_name, args.reps, args.max_gb * 1e9, flush_buf,
                                     checker.rows if with_oracle else None)
                        if r is None:
                            continue
                        tail = ""
                        if checker is not None:
                            if with_oracle:
                                c = checker.check(r.pop("X"), r.pop("Y_rows"), dtype_name)
                                tail = f" {c['err']:.1e} ({'ok' if c['ok'] else 'ABOVE TOLERANCE'}, {c['rows']:,} rows) | {c['cpu_ms']:,.0f} ({c['threads']} threads) |"
                            else:
                                tail = " operand over the host budget | |"
                        tol = 1e-5 if dtype_name == "f32" else 1e-2
                        flag = "" if r["identity_err"] <= tol else " (ABOVE TOLERANCE)"
                        print(f"| {scale} | {ids} | {n:,} | {info['nnz']:,} | {info['n_segments']:,} | {dtype_name} | {width} | "
                              f"{r['ms'] * 1e3:,.0f} | {r['ms_min'] * 1e3:,.0f} | {r['ms_flushed'] * 1e3:,.0f} | "
                              f"{r['alg_gbs']:,.0f} | {r['alg_gbs'] / peak:.3f} | "
                              f"{r['gather_gbs']:,.0f} | {r['identity_err']:.1e}{flag} |{tail}", flush=True)
                if B.slicegcn_graph_device_status(g) != 0:
                    raise SystemExit("a bounded wait in a kernel ran out (device status word set)")
            finally:
                B.slicegcn_graph_destroy(g)
        print(f"<!-- scale {scale}: edge list generated in {gen_s:.0f} s on the host -->", flush=True)


if __name__ == "__main__":
    main()
