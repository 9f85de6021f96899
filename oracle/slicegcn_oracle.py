"""TEST INFRASTRUCTURE ONLY -- plain CPU oracle for the SliceGCN hot path.

A slow, obviously-correct float64 restatement of what the paper's method
computes, written from the paper's equations and algorithms.  It shares no
code with the CUDA library and never imports it.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may call it.

What is pinned (see tests/test_oracle_*.py) and what is not:
  * slice strategy (Algorithm 1)      -- hand-executed values, Eq. 3 closed form
  * graph normalisation (Eq. 1)       -- 4-node worked example, dense brute force,
                                          A_hat*sqrt(deg) = sqrt(deg)
  * neighbor aggregation, transposed  -- adjoint identity on a directed graph
  * sliced layer (Eq. 6), SE (Eq. 7), concat (Eq. 8)
                                       -- block-diagonal equivalence, p=1 => Eq. 1
  * model shapes                      -- the parameter counts of Table III
  * backward                          -- central finite differences of the loss
  * cross entropy (Eq. 10)            -- uniform logits => ln C
  * Adam / cosine schedule            -- first-step closed form, lr(T/2), lr(T)
  * epoch loop (Algorithm 3)          -- two epochs of a three-parameter problem worked by
                                          hand: which index feeds the rate, which the step
  * storage rounding (bf16 configs)   -- which tensors are representable afterwards, call counts
  * parity unpinned: the activation inside MLP_FF and MLP_CLS (ReLU is a choice;
    the paper prints none), Adam's beta/eps constants, the placement of dropout
    (Table II lists a rate, the text never says where it acts).

Array conventions: row-major numpy float64 unless stated; node features are
n x d'; slices are column ranges [start, end) (0-based, half-open, as in
Algorithm 1).
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def build_c(force: bool = False) -> str:
    """Compile the C neighbor-sum loop (spmm_ref.c) next to its source."""
    src = os.path.join(_HERE, "spmm_ref.c")
    out = os.path.join(_HERE, "liboracle_spmm.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", src, "-o", out, "-lm"])
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build_c())
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_spmm_gather.argtypes = [i64, p, p, p, p, i64, i64, p, i64, p, i64, ctypes.c_int, ctypes.c_int]
        lib.oracle_spmm_gather.restype = None
        lib.oracle_spmm_scatter_t.argtypes = [i64, p, p, p, p, i64, i64, p, i64, ctypes.c_int]
        lib.oracle_spmm_scatter_t.restype = None
        lib.oracle_max_threads.restype = ctypes.c_int
        _LIB = lib
    return _LIB


def max_threads() -> int:
    return int(_lib().oracle_max_threads())


# --------------------------------------------------------------------------
# Algorithm 1 (slice strategy) and Eq. 3
# --------------------------------------------------------------------------

def slice_strategy(in_d: int, p: int, scale: float = 1.0, rule: str = "ceil") -> Tuple[List[Tuple[int, int]], int]:
    """Algorithm 1: list of (slice_start, slice_end) and slice_size.

    rule="ceil" is the algorithm as printed (slice_size = ceil(in_d / p));
    rule="floor_plus_1" is the width the text gives for W_FF (floor(in_d/p)+1),
    the only one that reproduces Table III.
    """
    if in_d < 1 or p < 1:
        raise ValueError("in_d and p must be >= 1")
    if rule == "ceil":
        slice_size = -(-in_d // p)
    elif rule == "floor_plus_1":
        slice_size = in_d // p + 1
    else:
        raise ValueError(rule)
    width = int(slice_size * scale)          # Algorithm 1 truncates the scaled width toward zero
    if width < 1 or width > in_d:
        raise ValueError("scaled slice width outside [1, in_d]")
    # Slice i would start at i * slice_size; one that would run past the last column is moved
    # left until it ends there (Algorithm 1's correction step; Eq. 3's second case).
    starts = [min(i * slice_size, in_d - width) for i in range(p)]
    return [(s0, s0 + width) for s0 in starts], slice_size


def slice_bounds_eq3(d_in: int, p: int, i: int) -> Tuple[int, int]:
    """Eq. 3: 1-based inclusive (start, end) of slice i in [1, p] (reading d as d')."""
    c = -(-d_in // p)
    if i * c < d_in:
        return (i - 1) * c + 1, i * c
    return d_in - c + 1, d_in


def slice_feature(x: np.ndarray, in_sizes: Sequence[Tuple[int, int]]) -> List[np.ndarray]:
    """Algorithm 2 / Eq. 2: X^i = X[:, start:end] (device placement dropped)."""
    return [x[:, s:e] for (s, e) in in_sizes]


# --------------------------------------------------------------------------
# Graph: canonical CSR of A in {0,1}^{n x n}, |N(v)|, and A_hat
# --------------------------------------------------------------------------

@dataclass
class Graph:
    n: int
    rowptr: np.ndarray      # int32 [n+1]
    colidx: np.ndarray      # int32 [nnz], ascending inside each row, no duplicates
    deg: np.ndarray         # int32 [n] = |N(v_i)| = stored entries of row i
    symmetric: bool

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])


def build_graph(n: int, src: np.ndarray, dst: np.ndarray, symmetrize: bool = True,
                self_loops: bool = True) -> Graph:
    """Edge list -> canonical CSR.  Entry (i, j) is stored when j is a neighbor
    of i; an input pair (src, dst) = (u, v) makes v a neighbor of u (row u,
    column v).  A is 0/1: repeated pairs are merged; with self_loops every
    diagonal entry is stored exactly once."""
    src = np.asarray(src)
    dst = np.asarray(dst)
    if src.shape != dst.shape:
        raise ValueError("src/dst length mismatch")
    if src.size and (src.min() < 0 or dst.min() < 0 or src.max() >= n or dst.max() >= n):
        raise ValueError("node id out of range")
    # one key row * n + col per candidate entry: the input pairs, their reverses, the diagonal
    m = src.size
    key = np.empty(m * (2 if symmetrize else 1) + (n if self_loops else 0), dtype=np.int64)
    key[:m] = src
    key[:m] *= n
    key[:m] += dst
    if symmetrize:
        key[m:2 * m] = dst
        key[m:2 * m] *= n
        key[m:2 * m] += src
    if self_loops:
        key[key.size - n:] = np.arange(n, dtype=np.int64) * (n + 1)
    key.sort()                               # sorted by (row, col) ...
    if key.size:
        key = key[np.concatenate(([True], key[1:] != key[:-1]))]   # ... repeated pairs merged (A is 0/1)
    rows = key // n
    cols = (key - rows * n).astype(np.int32)
    deg = np.bincount(rows, minlength=n).astype(np.int64)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg, out=rowptr[1:])
    if rowptr[-1] >= 2 ** 31:
        raise OverflowError("nnz does not fit int32")
    g = Graph(n, rowptr.astype(np.int32), cols, deg.astype(np.int32), False)
    # symmetric pattern: the transposed keys, sorted, are the keys
    key_t = cols.astype(np.int64)
    key_t *= n
    key_t += rows
    key_t.sort()
    g.symmetric = bool(np.array_equal(key, key_t))
    return g


def dinv_f32(deg: np.ndarray) -> np.ndarray:
    """1/sqrt(|N(v)|) in IEEE float32 (correctly rounded sqrt, then division);
    0 for an empty neighbor set.  Used only for the bit-level check of the
    library's degree vector."""
    d = deg.astype(np.float32)
    out = np.zeros_like(d)
    nz = deg > 0
    out[nz] = np.float32(1.0) / np.sqrt(d[nz])
    return out


AGGREGATORS = {"sym": 0, "mean": 1, "sum": 2}


def spmm(g: Graph, x: np.ndarray, transpose: bool = False, rows: Optional[np.ndarray] = None,
         threads: int = 0, norm: str = "sym") -> np.ndarray:
    """A_hat @ x (or A_hat^T @ x).  norm="sym" (the paper's): the normalised neighbor sum of Eq. 1 / Eq. 6,
    1/c_ij = 1/(sqrt|N(v_i)| sqrt|N(v_j)|).  The two other aggregators of message-passing layers the paper's
    closing section alludes to: "mean" (A_hat = D^-1 A, the mean over N(v_i)) and "sum" (A_hat = A).
    rows= limits the gather form to a list of output rows (used for sampled checks on large graphs)."""
    code = AGGREGATORS[norm]
    x = np.ascontiguousarray(x, dtype=np.float64)
    if x.ndim == 1:
        return spmm(g, x[:, None], transpose, rows, threads, norm)[:, 0]
    n, w = x.shape
    assert n == g.n
    lib = _lib()
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    if not transpose:
        if rows is not None:
            rows = np.ascontiguousarray(rows, dtype=np.int64)
            out = np.empty((rows.size, w), dtype=np.float64)
            lib.oracle_spmm_gather(n, vp(g.rowptr), vp(g.colidx), vp(g.deg), vp(x), w, w, vp(out), w,
                                   vp(rows), rows.size, threads, code)
        else:
            out = np.empty((n, w), dtype=np.float64)
            lib.oracle_spmm_gather(n, vp(g.rowptr), vp(g.colidx), vp(g.deg), vp(x), w, w, vp(out), w,
                                   None, 0, threads, code)
        return out
    assert rows is None
    out = np.empty((n, w), dtype=np.float64)
    lib.oracle_spmm_scatter_t(n, vp(g.rowptr), vp(g.colidx), vp(g.deg), vp(x), w, w, vp(out), w, code)
    return out


# --------------------------------------------------------------------------
# bf16 storage rounding (round to nearest even), for the bf16-stored configs
# --------------------------------------------------------------------------

def round_bf16(x: np.ndarray) -> np.ndarray:
    """Value of x after a store to bfloat16 (RNE) and load back, as float64."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    out = u.astype(np.uint32).view(np.float32).astype(np.float64)
    return out.reshape(np.shape(x))


def identity(x):
    return x


# --------------------------------------------------------------------------
# Model description and parameter shapes
# --------------------------------------------------------------------------

@dataclass
class ModelDesc:
    in_d: int                       # d'
    hidden: int                     # width of the unsliced GCN; classifier hidden width
    num_layers: int                 # L
    num_classes: int                # |C|
    p: int = 1                      # number of slices (computing devices in the paper)
    scale: float = 1.0              # slice_size_scale
    use_ff: bool = False            # feature fusion (Eq. 4 / Algorithm 3)
    use_se: bool = False            # slice encoding (Eq. 7)
    use_self: bool = True           # W_self term of Eq. 6 (False: Eq. 1, plain GCN)
    use_b_self: bool = False        # second bias per layer (needed by Table III only)
    slice_rule: str = "ceil"
    aggregator: str = "sym"         # "sym" = Eq. 1 / Eq. 6 as printed; "mean" / "sum": other message-passing aggregators
    slices: List[Tuple[int, int]] = field(default_factory=list)
    slice_size: int = 0
    h_s: int = 0

    def __post_init__(self):
        self.slices, self.slice_size = slice_strategy(self.in_d, self.p, self.scale, self.slice_rule)
        # each layer is scaled down in proportion to p (Section "Analysis"); ceil pinned by Table III
        self.h_s = -(-self.hidden // self.p)

    def layer_in_ranges(self, layer: int) -> List[Tuple[int, int]]:
        """Column range each slice reads from the layer's input matrix."""
        if layer == 0:
            if self.use_ff:                   # one fused X_ff feeds every slice
                return [(0, self.slice_size)] * self.p
            return list(self.slices)
        return [(i * self.h_s, (i + 1) * self.h_s) for i in range(self.p)]


def param_shapes(m: ModelDesc) -> Dict[str, Tuple[int, ...]]:
    """Name -> shape of every learnable tensor, in a fixed order."""
    shapes: Dict[str, Tuple[int, ...]] = {}
    if m.use_ff:                              # MLP_FF(in=d', h=d', out=slice_size, layers=2)
        shapes["ff_W1"] = (m.in_d, m.in_d)
        shapes["ff_b1"] = (m.in_d,)
        shapes["ff_W2"] = (m.in_d, m.slice_size)
        shapes["ff_b2"] = (m.slice_size,)
    for l in range(m.num_layers):
        for i, (s, e) in enumerate(m.layer_in_ranges(l)):
            w_in = e - s
            shapes[f"W_agg.{l}.{i}"] = (w_in, m.h_s)
            if m.use_self:
                shapes[f"W_self.{l}.{i}"] = (w_in, m.h_s)
            shapes[f"b.{l}.{i}"] = (m.h_s,)
            if m.use_b_self:
                shapes[f"b_self.{l}.{i}"] = (m.h_s,)
    if m.use_se:
        shapes["E"] = (m.p, m.h_s)
    shapes["Wc1"] = (m.p * m.h_s, m.hidden)
    shapes["bc1"] = (m.hidden,)
    shapes["Wc2"] = (m.hidden, m.num_classes)
    shapes["bc2"] = (m.num_classes,)
    return shapes


def param_count(m: ModelDesc) -> int:
    return int(sum(int(np.prod(s)) for s in param_shapes(m).values()))


# --------------------------------------------------------------------------
# Forward (Eq. 4-10) and backward
# --------------------------------------------------------------------------

def relu(x):
    return np.maximum(x, 0.0)


# Names of the places where a bf16-stored schedule keeps a tensor in the storage type.  Which of them a
# given run uses is an INPUT of forward() / backward() (`rnd_at`), never derived here:
#   forward : "ff_act", "X_ff", "Z.<l>" (aggregate-first layer l), "T.<l>" (transform-first), "H.<l>"
#             (output of layer l, l = 1..L), "cls_act"
#   backward: "dZ.<l>" (dM W_agg^T of aggregate-first layer l, the operand of the transposed aggregation)
def forward_rounding_points(m: "ModelDesc", order: Sequence[str]) -> frozenset:
    """Every forward point of a model with the given per-layer orders (what a schedule that stores
    all activations in the storage type uses)."""
    pts = {"cls_act"} | {f"H.{l + 1}" for l in range(m.num_layers)}
    pts |= {("Z" if order[l] == "agg" else "T") + f".{l}" for l in range(m.num_layers)}
    if m.use_ff:
        pts |= {"ff_act", "X_ff"}
    return frozenset(pts)


def _check_points(rnd_at, allowed):
    unknown = set(rnd_at) - set(allowed)
    if unknown:
        raise ValueError(f"no such rounding point in this model / schedule: {sorted(unknown)}")


def forward(m: ModelDesc, g: Graph, x: np.ndarray, params: Dict[str, np.ndarray],
            labels: Optional[np.ndarray] = None, train_idx: Optional[np.ndarray] = None,
            rnd: Callable[[np.ndarray], np.ndarray] = identity,
            order: Optional[Sequence[str]] = None, threads: int = 0,
            rnd_at: Optional[Sequence[str]] = None,
            dropout: Optional[Dict[int, np.ndarray]] = None, drop_rate: float = 0.0) -> Dict[str, object]:
    """One forward pass (Eq. 4-10).

    order[l] in {"agg", "xform"} says which intermediate layer l stores (A_hat*H or H*W_agg) -- the
    two are the same mathematics.  rnd (identity for fp32 storage, round_bf16 for bf16 storage) is
    applied at the stores named in rnd_at (see forward_rounding_points; None = all of them).
    dropout: {l: 0/1 mask of shape n x (p*h_s)} for l in 1..L-1 -- the output of layer l is multiplied
    by the mask and by 1/(1 - drop_rate) before the next layer reads it (placement is a choice: the
    paper lists only a rate).  Returns every intermediate needed by backward()."""
    P = {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}
    x = np.asarray(x, dtype=np.float64)
    order = list(order) if order is not None else ["agg"] * m.num_layers
    allowed = forward_rounding_points(m, order)
    if rnd_at is None:
        rnd_at = allowed
    _check_points(rnd_at, allowed)
    r = lambda name, v: rnd(v) if name in rnd_at else v
    dropout = dropout or {}
    if any(l < 1 or l >= m.num_layers for l in dropout):
        raise ValueError("dropout masks act between layers: keys 1..L-1")
    c: Dict[str, object] = {"order": order, "dropout": dropout, "drop_rate": drop_rate}
    if m.use_ff:
        c["ff_pre"] = x @ P["ff_W1"] + P["ff_b1"]
        c["ff_act"] = r("ff_act", relu(c["ff_pre"]))
        h = r("X_ff", c["ff_act"] @ P["ff_W2"] + P["ff_b2"])
    else:
        h = x
    c["H0"] = h
    for l in range(m.num_layers):
        ranges = m.layer_in_ranges(l)
        out = np.empty((g.n, m.p * m.h_s), dtype=np.float64)
        for i, (s, e) in enumerate(ranges):
            hin = h[:, s:e]                                   # Eq. 2 / Eq. 5
            W = P[f"W_agg.{l}.{i}"]
            if order[l] == "agg":
                z = r(f"Z.{l}", spmm(g, hin, threads=threads, norm=m.aggregator))   # sum_u h_u / c_uv
                c[f"Z.{l}.{i}"] = z
                mm = z @ W + P[f"b.{l}.{i}"]
            else:
                t = r(f"T.{l}", hin @ W)
                c[f"T.{l}.{i}"] = t
                mm = spmm(g, t, threads=threads, norm=m.aggregator) + P[f"b.{l}.{i}"]
            c[f"M.{l}.{i}"] = mm
            hi = relu(mm)                                     # Eq. 6: ReLU covers the aggregation only
            if m.use_self:
                hi = hi + hin @ P[f"W_self.{l}.{i}"]
            if m.use_b_self:
                hi = hi + P[f"b_self.{l}.{i}"]
            if m.use_se and l == m.num_layers - 1:
                hi = hi + P["E"][i]                           # Eq. 7, row i of E for slice i
            out[:, i * m.h_s:(i + 1) * m.h_s] = hi            # Eq. 8: concat = adjacent columns
        if (l + 1) in dropout:
            out = out * np.asarray(dropout[l + 1], dtype=np.float64) / (1.0 - drop_rate)
        h = r(f"H.{l + 1}", out)
        c[f"H{l + 1}"] = h
    c["cls_pre"] = h @ P["Wc1"] + P["bc1"]                    # Eq. 9
    c["cls_act"] = r("cls_act", relu(c["cls_pre"]))
    logits = c["cls_act"] @ P["Wc2"] + P["bc2"]
    c["logits"] = logits
    if labels is not None:
        idx = np.arange(g.n) if train_idx is None else np.asarray(train_idx)
        zmax = logits[idx].max(axis=1, keepdims=True)
        lse = zmax[:, 0] + np.log(np.exp(logits[idx] - zmax).sum(axis=1))
        c["loss"] = float(np.mean(lse - logits[idx, labels[idx]]))   # Eq. 10
        c["train_idx"] = idx
    return c


def backward(m: ModelDesc, g: Graph, x: np.ndarray, params: Dict[str, np.ndarray], labels: np.ndarray,
             cache: Dict[str, object], threads: int = 0, relu_margin: float = 0.0,
             rnd: Callable[[np.ndarray], np.ndarray] = identity, rnd_at: Sequence[str] = ()) -> Dict[str, np.ndarray]:
    """Reverse-mode gradient of the mean cross-entropy w.r.t. every parameter
    (the forward pass's storage rounding treated as identity).  ReLU'(0) = 0.

    rnd is applied to the activation gradients named in rnd_at ("dZ.<l>": dM W_agg^T of the
    aggregate-first layer l, the operand of the transposed aggregation); nothing is rounded unless
    named.  Every other gradient tensor stays in full precision.

    relu_margin (default 0 = the definition) moves the ReLU decision threshold to
    relu_margin * max|pre-activation| of each ReLU: a positive / negative margin switches every
    pre-activation that is within rounding noise of zero off / on.  Tests use the two results to
    bound the effect of sign decisions that fp32 and fp64 arithmetic may take differently."""
    P = {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}
    x = np.asarray(x, dtype=np.float64)
    idx = cache["train_idx"]
    logits = cache["logits"]
    order = cache["order"]
    _check_points(rnd_at, {f"dZ.{l}" for l in range(m.num_layers) if order[l] == "agg"})
    G: Dict[str, np.ndarray] = {}
    dlog = np.zeros_like(logits)
    z = logits[idx] - logits[idx].max(axis=1, keepdims=True)
    sm = np.exp(z)
    sm /= sm.sum(axis=1, keepdims=True)
    sm[np.arange(idx.size), labels[idx]] -= 1.0
    dlog[idx] = sm / idx.size
    G["Wc2"] = cache["cls_act"].T @ dlog
    G["bc2"] = dlog.sum(axis=0)

    def on(pre, scale=None):
        sc = np.abs(pre).max() if scale is None else scale
        return pre > relu_margin * sc

    da = (dlog @ P["Wc2"].T) * on(cache["cls_pre"])
    hL = cache[f"H{m.num_layers}"]
    G["Wc1"] = hL.T @ da
    G["bc1"] = da.sum(axis=0)
    dh = da @ P["Wc1"].T
    c = cache
    for l in reversed(range(m.num_layers)):
        ranges = m.layer_in_ranges(l)
        hprev = c[f"H{l}"]
        dprev = np.zeros_like(hprev)
        if (l + 1) in c.get("dropout", {}):                   # the layer's output passed through a dropout mask
            dh = dh * np.asarray(c["dropout"][l + 1], dtype=np.float64) / (1.0 - c["drop_rate"])
        if m.use_se and l == m.num_layers - 1:
            G["E"] = np.stack([dh[:, i * m.h_s:(i + 1) * m.h_s].sum(axis=0) for i in range(m.p)])
        m_scale = max(np.abs(c[f"M.{l}.{i}"]).max() for i in range(m.p))
        for i, (s, e) in enumerate(ranges):
            cols = slice(i * m.h_s, (i + 1) * m.h_s)
            dhi = dh[:, cols]
            hin = hprev[:, s:e]
            dm = dhi * on(c[f"M.{l}.{i}"], m_scale)
            G[f"b.{l}.{i}"] = dm.sum(axis=0)
            if m.use_b_self:
                G[f"b_self.{l}.{i}"] = dhi.sum(axis=0)
            dhin = np.zeros_like(hin)
            if m.use_self:
                G[f"W_self.{l}.{i}"] = hin.T @ dhi
                dhin = dhin + dhi @ P[f"W_self.{l}.{i}"].T
            W = P[f"W_agg.{l}.{i}"]
            if order[l] == "agg":
                G[f"W_agg.{l}.{i}"] = c[f"Z.{l}.{i}"].T @ dm
                dz = dm @ W.T
                if f"dZ.{l}" in rnd_at:
                    dz = rnd(dz)
                dhin = dhin + spmm(g, dz, transpose=True, norm=m.aggregator)
            else:
                dt = spmm(g, dm, transpose=True, norm=m.aggregator)
                G[f"W_agg.{l}.{i}"] = hin.T @ dt
                dhin = dhin + dt @ W.T
            dprev[:, s:e] += dhin            # overlapping slices / shared X_ff: contributions add
        dh = dprev
    G["H0"] = dh
    if m.use_ff:
        G["ff_W2"] = c["ff_act"].T @ dh
        G["ff_b2"] = dh.sum(axis=0)
        dpre = (dh @ P["ff_W2"].T) * on(c["ff_pre"])
        G["ff_W1"] = x.T @ dpre
        G["ff_b1"] = dpre.sum(axis=0)
    return G


def loss_only(m, g, x, params, labels, train_idx=None, order=None) -> float:
    return forward(m, g, x, params, labels, train_idx, order=order)["loss"]


# --------------------------------------------------------------------------
# Optimiser: Adam with a cosine-annealed learning rate, one step per epoch
# --------------------------------------------------------------------------

def cosine_lr(lr0: float, epoch: int, total_epochs: int) -> float:
    """Learning rate used by the update of 0-based epoch `epoch` (eta_min = 0)."""
    return lr0 * 0.5 * (1.0 + math.cos(math.pi * epoch / total_epochs))


def adam_step(theta: np.ndarray, grad: np.ndarray, m1: np.ndarray, m2: np.ndarray, step: int, lr: float,
              beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0):
    """step is 1-based.  Returns (theta, m1, m2) after the update."""
    gth = grad + weight_decay * theta
    m1 = beta1 * m1 + (1.0 - beta1) * gth
    m2 = beta2 * m2 + (1.0 - beta2) * gth * gth
    mh = m1 / (1.0 - beta1 ** step)
    vh = m2 / (1.0 - beta2 ** step)
    return theta - lr * mh / (np.sqrt(vh) + eps), m1, m2


def apply_update(params: Dict[str, np.ndarray], grads: Dict[str, np.ndarray], opt_state: Dict[str, object],
                 lr0: float, epoch: int, total_epochs: int) -> None:
    """The update at the end of one iteration of Algorithm 3's epoch loop: the 0-based epoch index
    sets the cosine-annealed rate, the number of updates made so far plus one (epoch + 1) is Adam's
    step count.  params and opt_state ({"m1": {...}, "m2": {...}}) are updated in place."""
    lr = cosine_lr(lr0, epoch, total_epochs)
    for k in params:
        m1 = opt_state["m1"].setdefault(k, np.zeros_like(params[k], dtype=np.float64))
        m2 = opt_state["m2"].setdefault(k, np.zeros_like(params[k], dtype=np.float64))
        params[k], opt_state["m1"][k], opt_state["m2"][k] = adam_step(
            np.asarray(params[k], dtype=np.float64), grads[k], m1, m2, epoch + 1, lr)


def train_epoch(m: ModelDesc, g: Graph, x, params: Dict[str, np.ndarray], labels, opt_state: Dict[str, object],
                lr0: float, epoch: int, total_epochs: int, train_idx=None, rnd=identity, order=None,
                threads: int = 0, rnd_at=None, rnd_at_bwd=(), dropout=None, drop_rate: float = 0.0):
    """Algorithm 3, one iteration of the epoch loop: forward, loss, backward, update.
    opt_state holds {"m1": {...}, "m2": {...}}; params are updated in place.
    Returns (loss, logits, grads)."""
    cache = forward(m, g, x, params, labels, train_idx, rnd, order, threads, rnd_at, dropout, drop_rate)
    grads = backward(m, g, x, params, labels, cache, threads, rnd=rnd, rnd_at=rnd_at_bwd)
    apply_update(params, {k: grads[k] for k in params}, opt_state, lr0, epoch, total_epochs)
    return cache["loss"], cache["logits"], grads
