"""Training throughput of the paper's model variants on one synthetic graph shape.

The layout follows the paper's Table IV (methods x number of slices): plain GCN (one slice, no self
branch), SliceGCN with p slices, and the -SE / -FF / -FFSE variants.  Accuracy columns need the
paper's datasets and are not reproduced; this prints epochs/s of the CUDA path only.

    python variant_grid.py --workload citation --epochs 20
"""
from __future__ import annotations

import argparse

import numpy as np


def time_variant(B, torch, g, w, X, y, p, use_ff, use_se, use_self, epochs, warmup=3, table3=False, dropout=0.0):
    from paper_2408_11500_b200 import synth
    dev = X.device
    # table3: the shapes behind the paper's parameter counts (Table III): slices of floor(d'/p) + 1 columns and a
    # second bias vector per layer
    m = B.slicegcn_model_create(in_d=w["in_d"], hidden=w["hidden"], num_layers=w["layers"], num_classes=w["classes"],
                                num_slices=p, use_ff=use_ff, use_se=use_se, use_self=use_self,
                                slice_rule=B.RULE_FLOOR_PLUS_1 if (table3 and p > 1) else B.RULE_CEIL,
                                use_b_self=bool(table3 and use_self),
                                dtype=B.BF16 if X.dtype == torch.bfloat16 else B.F32, cache_input_aggregate=True)
    try:
        params = torch.from_numpy(B.pack_params(m, synth.init_params(B.named_param_shapes(m), 0))).to(dev)
        grads, m1, m2 = torch.zeros_like(params), torch.zeros_like(params), torch.zeros_like(params)
        ws_bytes = B.slicegcn_train_workspace_bytes(m, g)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        loss = torch.zeros(1, dtype=torch.float32, device=dev)
        st = torch.cuda.current_stream()

        drop = None
        if dropout > 0 and w["layers"] > 1:   # one fixed seeded mask per layer but the last (the library draws no random numbers)
            h_s = B.slicegcn_model_slices(m, p)[2]
            gen = torch.Generator(device=dev)
            gen.manual_seed(1)
            masks = [(torch.rand((w["n"], p * h_s), generator=gen, device=dev) >= dropout).to(torch.uint8) for _ in range(w["layers"] - 1)]
            drop = B.make_dropout_desc(dropout, masks, p * h_s)

        def epoch(ep):
            if drop is None:
                B.slicegcn_train_epoch(m, g, X, w["in_d"], y, None, 0, params, grads, m1, m2, B.make_opt_desc(1e-3, ep, 500),
                                       None, loss, ws, ws_bytes, st.cuda_stream)
            else:
                B.slicegcn_train_epoch_dropout(m, g, X, w["in_d"], y, None, 0, params, grads, m1, m2, B.make_opt_desc(1e-3, ep, 500),
                                               drop, None, loss, ws, ws_bytes, st.cuda_stream)

        for ep in range(warmup):
            epoch(ep)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for ep in range(epochs):
            epoch(warmup + ep)
        e1.record(st)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / epochs
        count = B.slicegcn_model_param_count(m)
        return ms, count, float(loss.item())
    finally:
        B.slicegcn_model_destroy(m)


def main():
    import torch
    from paper_2408_11500_b200 import binding as B, synth
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="citation", choices=sorted(synth.WORKLOADS) + sorted(synth.TABLE1_SHAPES),
                    help="a named workload, or t1_<nodes>: a seeded graph with the sizes of the paper's Table I, the layer count and "
                         "dropout rate of its Table II and width 512")
    ap.add_argument("--epochs", type=int, default=20)
    ap.add_argument("--slices", default="2,4,8")
    ap.add_argument("--hidden", type=int, default=0, help="override the workload's hidden width (the paper's Table III uses 512)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (the paper goes up to 7)")
    ap.add_argument("--table3-shapes", action="store_true",
                    help="slices of floor(d'/p) + 1 columns and two bias vectors per layer, as the paper's parameter counts imply")
    args = ap.parse_args()
    w = dict(synth.WORKLOADS[args.workload]) if args.workload in synth.WORKLOADS else synth.table1_workload(args.workload)
    dropout = float(w.get("dropout", 0.0))
    if args.hidden:
        w["hidden"] = args.hidden
    if args.layers:
        w["layers"] = args.layers
    src, dst = synth.make_graph(w, 0)
    g = B.slicegcn_graph_create(w["n"], src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    info = B.slicegcn_graph_info(g)
    tdt = torch.bfloat16 if w["dtype"] == "bf16" else torch.float32
    X = torch.from_numpy(synth.make_features(w, 0)).cuda().to(tdt).contiguous()
    y = torch.from_numpy(synth.uniform_labels(w["n"], w["classes"], 0)).cuda()
    ps = [int(v) for v in args.slices.split(",")]
    print(f"workload `{args.workload}`: N={w['n']:,}, nnz={info['nnz']:,}, in_d={w['in_d']}, hidden={w['hidden']}, "
          f"layers={w['layers']}, classes={w['classes']}, {w['dtype']}, dropout {dropout:g}; {args.epochs} timed epochs per cell\n")
    print("| method | " + " | ".join(f"p={p}: ms/epoch (epochs/s) [params]" for p in ps) + " |")
    print("|---|" + "---|" * len(ps))
    t3 = args.table3_shapes
    # Table III counts two weight matrices and two bias vectors per GCN layer: with --table3-shapes the one-slice row
    # keeps the self branch so that the parameter count printed here is the table's
    ms, cnt, _ = time_variant(B, torch, g, w, X, y, 1, False, False, t3, args.epochs, table3=t3, dropout=dropout)
    label = "GCN (one slice, self branch as in Table III)" if t3 else "GCN (one slice, no self branch)"
    print(f"| {label} | {ms:.2f} ({1e3 / ms:.1f}) [{cnt:,}] |" + " |" * (len(ps) - 1))
    for name, ff, se in (("SliceGCN", False, False), ("SliceGCN-SE", False, True), ("SliceGCN-FF", True, False),
                         ("SliceGCN-FFSE", True, True)):
        cells = []
        for p in ps:
            ms, cnt, _ = time_variant(B, torch, g, w, X, y, p, ff, se, True, args.epochs, table3=t3, dropout=dropout)
            cells.append(f"{ms:.2f} ({1e3 / ms:.1f}) [{cnt:,}]")
        print(f"| {name} | " + " | ".join(cells) + " |")
    B.slicegcn_graph_destroy(g)


if __name__ == "__main__":
    main()
