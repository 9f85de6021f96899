"""Shared plumbing of the GPU parity tests: runs the same seeded problem through the CUDA
library (via the C ABI binding) and through the CPU oracle."""
from __future__ import annotations

import numpy as np

from oracle import slicegcn_oracle as orc
from paper_2408_11500_b200 import synth


def rel_inf(a, b):
    """max|a-b| / max|b|: the per-tensor error metric of the parity gates."""
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    den = np.abs(b).max()
    return float(np.abs(a - b).max() / (den if den > 0 else 1.0))


def oracle_desc(**kw):
    return orc.ModelDesc(kw["in_d"], kw["hidden"], kw["num_layers"], kw["num_classes"], p=kw.get("num_slices", 1),
                         scale=kw.get("slice_size_scale", 1.0), use_ff=kw.get("use_ff", False),
                         use_se=kw.get("use_se", False), use_self=kw.get("use_self", True),
                         use_b_self=kw.get("use_b_self", False),
                         slice_rule="floor_plus_1" if kw.get("slice_rule", 0) == 1 else "ceil",
                         aggregator=kw.get("aggregator", "sym"))


class GpuProblem:
    """Device-side state of one model on one graph (torch is used for memory only)."""

    def __init__(self, n, src, dst, X, y, named_params, self_loops=True, symmetrize=True, train_idx=None, aggregator="sym",
                 **model_kw):
        import torch
        from paper_2408_11500_b200 import binding as B
        self.B, self.torch = B, torch
        dev = torch.device("cuda:0")
        flags = (B.SYMMETRIZE if symmetrize else 0) | (B.ADD_SELF_LOOPS if self_loops else 0)
        flags |= {"sym": 0, "mean": B.NORM_MEAN, "sum": B.NORM_SUM}[aggregator]      # the aggregator is a property of the graph object
        self.g = B.slicegcn_graph_create(n, np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32), flags)
        self.m = B.slicegcn_model_create(**model_kw)
        self.kw = model_kw
        self.n = n
        dt = torch.bfloat16 if model_kw.get("dtype", 0) == B.BF16 else torch.float32
        self.X = torch.from_numpy(np.ascontiguousarray(X, np.float32)).to(dev).to(dt).contiguous()
        self.y = torch.from_numpy(np.ascontiguousarray(y, np.int32)).to(dev)
        self.train_idx = None if train_idx is None else torch.from_numpy(np.ascontiguousarray(train_idx, np.int32)).to(dev)
        self.params = torch.from_numpy(B.pack_params(self.m, named_params)).to(dev)
        self.grads = torch.zeros_like(self.params)
        self.m1 = torch.zeros_like(self.params)
        self.m2 = torch.zeros_like(self.params)
        self.ws_bytes = B.slicegcn_train_workspace_bytes(self.m, self.g)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.logits = torch.empty((n, model_kw["num_classes"]), dtype=torch.float32, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)

    def epoch(self, opt=None):
        B = self.B
        B.slicegcn_train_epoch(self.m, self.g, self.X, self.X.shape[1], self.y, self.train_idx,
                               0 if self.train_idx is None else self.train_idx.numel(), self.params, self.grads,
                               self.m1, self.m2, opt, self.logits, self.loss, self.ws, self.ws_bytes,
                               self.torch.cuda.current_stream().cuda_stream)
        self.torch.cuda.synchronize()
        return float(self.loss.item())

    def named_grads(self):
        return self.B.unpack_params(self.m, self.grads.cpu().numpy())

    def named_params(self):
        return self.B.unpack_params(self.m, self.params.cpu().numpy())

    def close(self):
        self.B.slicegcn_model_destroy(self.m)
        self.B.slicegcn_graph_destroy(self.g)


def small_problem(n=600, m_edges=2400, in_d=37, hidden=24, L=2, C=5, p=4, seed=0, max_degree=400, **kw):
    """A graph with a few hub rows (longer than the SpMM's long-row threshold), ragged sizes."""
    src, dst = synth.chung_lu_powerlaw(n, m_edges, 2.2, max_degree, seed=seed)
    X = synth.gaussian_features(n, in_d, seed=seed)
    y = synth.uniform_labels(n, C, seed=seed)
    model_kw = dict(in_d=in_d, hidden=hidden, num_layers=L, num_classes=C, num_slices=p, **kw)
    od = oracle_desc(**model_kw)
    params = synth.init_params(orc.param_shapes(od), seed=seed, bias_scale=0.2, se_scale=0.3)
    return src, dst, X, y, model_kw, od, params
