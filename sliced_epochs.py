"""Training epochs with the paper's own placement (Section IV-A, Eq. 8): one process per GPU, each computing an equal
range of the feature slices through `slicegcn_train_epoch_sliced`, the slice outputs meeting in one all-gather per
epoch (`slice_exchange.make_exchange` over NCCL).

    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 --master-port P \
        sliced_epochs.py --workload copurchase --epochs 10

With one process this is the ordinary epoch (no exchange).  Prints one JSON line on rank 0: epochs/s from the slowest
process's device time (CUDA events, max over processes).  Every process builds the same seeded graph, features,
labels and initial parameters, so the parameters stay replicas without being sent.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np


def main() -> None:
    import torch
    import torch.distributed as dist
    from paper_2408_11500_b200 import binding as B, slice_exchange as sx, synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="copurchase", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--fraction", type=float, default=1.0, help="scale the workload's nodes and edges")
    ap.add_argument("--epochs", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if world > 1:
        dist.init_process_group("nccl", rank=rank, world_size=world)
    w = dict(synth.WORKLOADS[args.workload])
    if args.fraction < 1.0:                              # the same generator on a smaller graph
        w["n"] = max(int(w["n"] * args.fraction), 64)
        w["m"] = max(int(w["m"] * args.fraction), 64)
        if "max_degree" in w:
            w["max_degree"] = max(w["max_degree"] * args.fraction, 16)
    s0, s1 = sx.slice_ranges(w["p"], world)[rank]
    src, dst = synth.make_graph(w, 0)
    g = B.slicegcn_graph_create(w["n"], src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    bf16 = w["dtype"] == "bf16"
    X = torch.from_numpy(synth.make_features(w, 0)).cuda().to(torch.bfloat16 if bf16 else torch.float32).contiguous()
    y = torch.from_numpy(synth.uniform_labels(w["n"], w["classes"], 0)).cuda()
    m = B.slicegcn_model_create(in_d=w["in_d"], hidden=w["hidden"], num_layers=w["layers"], num_classes=w["classes"],
                                num_slices=w["p"], use_ff=w.get("use_ff", False), use_se=w.get("use_se", False),
                                dtype=B.BF16 if bf16 else B.F32)
    rng = np.random.default_rng(0)                       # the same draw on every process
    params = torch.from_numpy((0.05 * rng.standard_normal(B.slicegcn_model_param_elems(m))).astype(np.float32)).cuda()
    grads, m1, m2 = torch.zeros_like(params), torch.zeros_like(params), torch.zeros_like(params)
    ws_bytes = B.slicegcn_train_workspace_bytes(m, g)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    loss = torch.zeros(1, device="cuda")
    exchange = sx.make_exchange(None, device="cuda") if world > 1 else None
    stream = torch.cuda.current_stream().cuda_stream

    def epoch(e: int) -> None:
        opt = B.OptDesc(1e-3, 0.9, 0.999, 1e-8, 0.0, e, args.warmup + args.epochs)
        B.slicegcn_train_epoch_sliced(m, g, X, X.shape[1], y, None, 0, params, grads, m1, m2, opt, s0, s1, exchange, None, loss,
                                      ws, ws_bytes, stream)

    for e in range(args.warmup):
        epoch(e)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for e in range(args.epochs):
        epoch(args.warmup + e)
    t1.record()
    torch.cuda.synchronize()
    ms = torch.tensor([t0.elapsed_time(t1)], device="cuda")
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"metric": "full-graph GCN training throughput, slices on separate processes", "unit": "epochs/s",
                          "value": args.epochs / (ms.item() * 1e-3), "ms_per_epoch": ms.item() / args.epochs, "processes": world,
                          "slices_per_process": s1 - s0, "workload": args.workload, "nodes": w["n"],
                          "final_loss": float(loss.item())}))
    B.slicegcn_model_destroy(m)
    B.slicegcn_graph_destroy(g)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
