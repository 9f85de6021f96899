"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each expected value is either a
number printed in / hand-derived from the paper (tests/golden/*.txt), a closed
form, an invariant, or a brute-force evaluation written independently here.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import slicegcn_oracle as orc
from paper_2408_11500_b200 import synth

from conftest import GOLDEN


# ------------------------------------------------------------------ Algorithm 1

def _read_alg1():
    cases = []
    for line in open(os.path.join(GOLDEN, "alg1_slices.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        a, b, c = [t.strip() for t in line.split("|")]
        in_d, p, scale = a.split()
        sl = [tuple(int(v) for v in t.split(":")) for t in c.split()]
        cases.append((int(in_d), int(p), float(scale), int(b), sl))
    return cases


@pytest.mark.parametrize("in_d,p,scale,size,slices", _read_alg1())
def test_slice_strategy_golden(in_d, p, scale, size, slices):
    got, got_size = orc.slice_strategy(in_d, p, scale)
    assert got_size == size
    assert got == slices


def test_slice_strategy_matches_eq3_closed_form():
    # Eq. 3 is 1-based inclusive; Algorithm 1 is 0-based half-open.  For the default scale the
    # two agree whenever every slice but the last fits before in_d (Eq. 3 sends every overflowing
    # slice to the last window, exactly like the shift in Algorithm 1).
    for in_d in range(1, 140):
        for p in range(1, 12):
            sl, size = orc.slice_strategy(in_d, p)
            for i in range(1, p + 1):
                s1, e1 = orc.slice_bounds_eq3(in_d, p, i)
                assert sl[i - 1] == (s1 - 1, e1), (in_d, p, i)


def test_slice_strategy_properties_and_errors():
    for in_d, p in itertools.product([1, 7, 100, 1433], [1, 2, 3, 8]):
        if p > in_d:
            continue
        sl, size = orc.slice_strategy(in_d, p)
        assert all(e - s == size for s, e in sl)
        assert sl[0][0] == 0 and sl[-1][1] == in_d
        covered = np.zeros(in_d, bool)
        for s, e in sl:
            covered[s:e] = True
        assert covered.all()
    with pytest.raises(ValueError):
        orc.slice_strategy(8, 0)
    with pytest.raises(ValueError):
        orc.slice_strategy(8, 2, 0.1)      # int(4*0.1) = 0 columns
    with pytest.raises(ValueError):
        orc.slice_strategy(8, 2, 3.0)      # 12 columns > in_d
    # floor+1 rule differs from ceil exactly when p divides in_d
    assert orc.slice_strategy(300, 3, rule="floor_plus_1")[1] == 101
    assert orc.slice_strategy(301, 3, rule="floor_plus_1")[1] == 101 == orc.slice_strategy(301, 3)[1]


# ------------------------------------------------------------------ graph + normalisation

def _read_four_node():
    d = {}
    for line in open(os.path.join(GOLDEN, "four_node_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, rest = line.split(" ", 1)
        d[k] = rest
    mat = lambda s: np.array([[float(v) for v in r.split()] for r in s.split("|")])
    edges = [tuple(int(v) for v in e.split("-")) for e in d["edges"].split()]
    return edges, mat(d["X"]), d, mat


def test_four_node_worked_example():
    edges, X, d, mat = _read_four_node()
    src = np.array([e[0] for e in edges]); dst = np.array([e[1] for e in edges])
    for tag, loops in (("selfloops", True), ("plain", False)):
        g = orc.build_graph(4, src, dst, symmetrize=True, self_loops=loops)
        assert g.deg.tolist() == [int(v) for v in d[f"deg_{tag}"].split()]
        assert g.symmetric
        ahat = mat(d[f"Ahat_{tag}"])
        np.testing.assert_allclose(orc.spmm(g, np.eye(4)), ahat, atol=1e-6)
        np.testing.assert_allclose(orc.spmm(g, X), mat(d[f"AX_{tag}"]), atol=1e-6)
        np.testing.assert_allclose(orc.spmm(g, X, transpose=True), mat(d[f"AX_{tag}"]), atol=1e-6)
    g = orc.build_graph(4, src, dst, True, True)
    assert g.rowptr.tolist() == [0, 3, 6, 10, 12]
    assert g.colidx.tolist() == [0, 1, 2, 0, 1, 2, 0, 1, 2, 3, 2, 3]


def test_graph_canonical_form():
    # repeated pairs, both directions given, an input self-loop: A stays 0/1
    src = np.array([0, 0, 1, 2, 2, 3, 3]); dst = np.array([1, 1, 0, 0, 2, 2, 2])
    g = orc.build_graph(4, src, dst, symmetrize=True, self_loops=True)
    assert g.rowptr.tolist() == [0, 3, 5, 8, 10]
    assert g.colidx.tolist() == [0, 1, 2, 0, 1, 0, 2, 3, 2, 3]
    g2 = orc.build_graph(4, src, dst, symmetrize=False, self_loops=False)
    assert g2.colidx.tolist() == [1, 0, 0, 2, 2] and g2.deg.tolist() == [1, 1, 2, 1]
    assert not g2.symmetric
    with pytest.raises(ValueError):
        orc.build_graph(3, np.array([0]), np.array([3]))
    with pytest.raises(ValueError):
        orc.build_graph(3, np.array([-1]), np.array([0]))
    # isolated node without self-loops: empty row, zero output, dinv = 0
    g3 = orc.build_graph(3, np.array([0]), np.array([1]), True, False)
    assert g3.deg.tolist() == [1, 1, 0]
    out = orc.spmm(g3, np.ones((3, 2)))
    assert out[2].tolist() == [0.0, 0.0] and orc.dinv_f32(g3.deg)[2] == 0.0


def _dense_ahat(g):
    """Brute force, written from Eq. 1 with python loops: A_hat[i,j] = A[i,j]/(sqrt d_i sqrt d_j)."""
    A = np.zeros((g.n, g.n))
    for i in range(g.n):
        for k in range(g.rowptr[i], g.rowptr[i + 1]):
            A[i, g.colidx[k]] = 1.0
    nbr = A.sum(axis=1)
    ah = np.zeros_like(A)
    for i in range(g.n):
        for j in range(g.n):
            if A[i, j] and nbr[j] > 0:       # a neighbor with an empty neighbor set: 1/c read as 0
                ah[i, j] = 1.0 / (math.sqrt(nbr[i]) * math.sqrt(nbr[j]))
    return ah


@pytest.mark.parametrize("n,m,sym,loops,seed", [(5, 6, True, True, 0), (17, 40, True, False, 1),
                                               (64, 300, True, True, 2), (33, 90, False, True, 3),
                                               (48, 200, False, False, 4)])
def test_spmm_vs_dense_bruteforce(n, m, sym, loops, seed):
    rng = np.random.default_rng(seed)
    src = rng.integers(0, n, m); dst = rng.integers(0, n, m)
    g = orc.build_graph(n, src, dst, sym, loops)
    X = rng.standard_normal((n, 7))
    ah = _dense_ahat(g)
    np.testing.assert_allclose(orc.spmm(g, X), ah @ X, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.spmm(g, X, transpose=True), ah.T @ X, rtol=1e-12, atol=1e-12)
    assert g.symmetric == np.array_equal(ah != 0, (ah != 0).T)


@pytest.mark.parametrize("norm", ["mean", "sum"])
@pytest.mark.parametrize("n,m,sym,loops,seed", [(17, 40, True, False, 1), (33, 90, False, True, 3), (48, 200, False, False, 4)])
def test_other_aggregators_vs_dense_bruteforce(norm, n, m, sym, loops, seed):
    """Mean (D^-1 A) and sum (A) aggregation, forward and transposed, against dense matrices built with python loops;
    closed forms: the mean of a constant is that constant on every node with a neighbor, the sum of ones is the degree."""
    rng = np.random.default_rng(seed)
    g = orc.build_graph(n, rng.integers(0, n, m), rng.integers(0, n, m), sym, loops)
    A = np.zeros((n, n))
    for i in range(n):
        for k in range(g.rowptr[i], g.rowptr[i + 1]):
            A[i, g.colidx[k]] = 1.0
    if norm == "mean":
        for i in range(n):
            if A[i].sum() > 0:
                A[i] /= A[i].sum()
    X = rng.standard_normal((n, 5))
    np.testing.assert_allclose(orc.spmm(g, X, norm=norm), A @ X, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.spmm(g, X, transpose=True, norm=norm), A.T @ X, rtol=1e-12, atol=1e-12)
    rows = np.array([0, n - 1, 3], dtype=np.int64)
    assert np.array_equal(orc.spmm(g, X, rows=rows, norm=norm), orc.spmm(g, X, norm=norm)[rows])
    ones = np.ones(n)
    if norm == "mean":
        np.testing.assert_allclose(orc.spmm(g, 7.0 * ones, norm=norm), 7.0 * (g.deg > 0), rtol=1e-13)
    else:
        np.testing.assert_allclose(orc.spmm(g, ones, norm=norm), g.deg.astype(np.float64), rtol=1e-13)
    # and the model's backward under these aggregators: finite differences
    m_ = orc.ModelDesc(6, 4, 2, 3, p=2, aggregator=norm)
    P = {k: v.astype(np.float64) for k, v in synth.init_params(orc.param_shapes(m_), seed=seed, bias_scale=0.3).items()}
    Xf = rng.standard_normal((n, 6)); y = rng.integers(0, 3, n)
    for order in (["agg", "agg"], ["xform", "agg"]):
        c = orc.forward(m_, g, Xf, P, y, order=order)
        G = orc.backward(m_, g, Xf, P, y, c)
        for name in ("W_agg.0.1", "W_self.1.0", "b.0.0"):
            flat = P[name].reshape(-1)
            old = flat[0]
            flat[0] = old + 1e-6; lp = orc.loss_only(m_, g, Xf, P, y, None, order)
            flat[0] = old - 1e-6; lm = orc.loss_only(m_, g, Xf, P, y, None, order)
            flat[0] = old
            fd = (lp - lm) / 2e-6
            assert abs(fd - G[name].reshape(-1)[0]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (norm, order, name)


def test_spmm_closed_form_sqrt_degree():
    # row i of A_hat * sqrt(deg): sum_j sqrt(d_j)/(sqrt d_i sqrt d_j) = d_i/sqrt(d_i) = sqrt(d_i)
    src, dst = synth.chung_lu_powerlaw(3000, 9000, 2.2, 200, seed=3)
    g = orc.build_graph(3000, src, dst, True, True)
    v = np.sqrt(g.deg.astype(np.float64))
    np.testing.assert_allclose(orc.spmm(g, v), v, rtol=1e-12)
    np.testing.assert_allclose(orc.spmm(g, v, transpose=True), v, rtol=1e-12)


def test_spmm_adjoint_identity_directed():
    rng = np.random.default_rng(7)
    n = 200
    g = orc.build_graph(n, rng.integers(0, n, 900), rng.integers(0, n, 900), symmetrize=False, self_loops=False)
    assert not g.symmetric
    X = rng.standard_normal((n, 5)); Y = rng.standard_normal((n, 5))
    lhs = np.sum(orc.spmm(g, X) * Y)
    rhs = np.sum(X * orc.spmm(g, Y, transpose=True))
    assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs))
    ah = _dense_ahat(g)
    np.testing.assert_allclose(orc.spmm(g, Y, transpose=True), ah.T @ Y, rtol=1e-12, atol=1e-13)


def test_column_separability_is_bit_exact():
    # (A_hat X)[:, s:e] == A_hat (X[:, s:e]): slices never interact during message passing
    src, dst = synth.chung_lu_powerlaw(500, 2000, 2.2, 80, seed=5)
    g = orc.build_graph(500, src, dst, True, True)
    X = synth.gaussian_features(500, 37, seed=1).astype(np.float64)
    full = orc.spmm(g, X)
    sl, _ = orc.slice_strategy(37, 4)            # overlapping last slice
    for s, e in sl:
        assert np.array_equal(full[:, s:e], orc.spmm(g, X[:, s:e]))
    rows = np.array([0, 3, 499, 17], dtype=np.int64)
    assert np.array_equal(orc.spmm(g, X, rows=rows), full[rows])
    assert np.array_equal(orc.spmm(g, X, threads=1), orc.spmm(g, X, threads=4))


def test_dinv_f32():
    deg = np.array([0, 1, 2, 3, 4, 16, 1000003], dtype=np.int32)
    d = orc.dinv_f32(deg)
    assert d.dtype == np.float32 and d[0] == 0 and d[1] == 1 and d[4] == 0.5 and d[5] == 0.25
    np.testing.assert_allclose(d[1:].astype(np.float64) ** 2 * deg[1:], 1.0, rtol=3e-7)


# ------------------------------------------------------------------ bf16 rounding

def test_round_bf16():
    import torch
    x = np.concatenate([np.random.default_rng(0).standard_normal(4096).astype(np.float32) * 37.0,
                        np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -0.0, 3.0e38], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(orc.round_bf16(x), want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.round_bf16(np.float32(1.0 + 2 ** -8)) == 1.0
    assert orc.round_bf16(np.float32(1.0 + 3 * 2 ** -8)) == 1.0 + 2 ** -6


# ------------------------------------------------------------------ model shapes: Table III

def _fmt(n):
    return f"{n / 1e6:.2f}M" if n >= 1e6 else f"{n / 1e3:.2f}K"


def test_table3_parameter_counts():
    ds, rows = [], []
    for line in open(os.path.join(GOLDEN, "table3_param_counts.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "dataset":
            ds.append((t[1], int(t[2]), int(t[3]), int(t[4])))
        elif t[0] == "row":
            rows.append((int(t[1]), int(t[2]), int(t[3]), t[5:]))
    assert len(ds) == 6 and len(rows) == 9
    checked = 0
    for p, ff, se, vals in rows:
        for (name, in_d, classes, L), want in zip(ds, vals):
            if p == 0:   # single-GPU GCN: the same layer (W_agg, W_self, two biases), no slicing
                m = orc.ModelDesc(in_d, 512, L, classes, p=1, use_self=True, use_b_self=True)
            else:
                m = orc.ModelDesc(in_d, 512, L, classes, p=p, use_ff=bool(ff), use_se=bool(se),
                                  use_self=True, use_b_self=True, slice_rule="floor_plus_1")
            assert _fmt(orc.param_count(m)) == want, (name, p, ff, se, orc.param_count(m))
            checked += 1
    assert checked == 54


# ------------------------------------------------------------------ layer semantics

def _tiny_problem(n=40, m_edges=120, in_d=11, hidden=8, L=2, C=3, p=2, seed=0, **kw):
    src, dst = synth.chung_lu_powerlaw(n, m_edges, 2.2, 12, seed=seed)
    g = orc.build_graph(n, src, dst, True, kw.pop("self_loops", True))
    m = orc.ModelDesc(in_d, hidden, L, C, p=p, **kw)
    X = synth.gaussian_features(n, in_d, seed=seed).astype(np.float64)
    y = synth.uniform_labels(n, C, seed=seed)
    P = {k: v.astype(np.float64) for k, v in
         synth.init_params(orc.param_shapes(m), seed=seed, bias_scale=0.3, se_scale=0.5).items()}
    return g, m, X, y, P


def test_single_slice_reduces_to_plain_gcn_eq1():
    g, m, X, y, P = _tiny_problem(p=1, use_self=False)
    c = orc.forward(m, g, X, P)
    ah = _dense_ahat(g)
    h = X
    for l in range(m.num_layers):       # Eq. 1: ReLU(b + A_hat H W)
        h = np.maximum(P[f"b.{l}.0"] + ah @ h @ P[f"W_agg.{l}.0"], 0.0)
    np.testing.assert_allclose(c[f"H{m.num_layers}"], h, rtol=1e-12, atol=1e-12)


def _block_diag(blocks):
    r = sum(b.shape[0] for b in blocks); c = sum(b.shape[1] for b in blocks)
    out = np.zeros((r, c)); i = j = 0
    for b in blocks:
        out[i:i + b.shape[0], j:j + b.shape[1]] = b
        i += b.shape[0]; j += b.shape[1]
    return out


@pytest.mark.parametrize("order", [("agg", "agg"), ("xform", "xform"), ("xform", "agg")])
def test_block_diagonal_equivalence(order):
    # non-overlapping slices: SliceGCN == one plain layer stack with block-diagonal weights,
    # slice encoding == one more bias on the concatenated output (Eq. 6-8)
    g, m, X, y, P = _tiny_problem(in_d=12, p=3, hidden=9, use_se=True, use_b_self=True)
    assert m.slices == [(0, 4), (4, 8), (8, 12)] and m.h_s == 3
    c = orc.forward(m, g, X, P, order=order)
    ah = _dense_ahat(g)
    h = X
    for l in range(m.num_layers):
        Wa = _block_diag([P[f"W_agg.{l}.{i}"] for i in range(3)])
        Ws = _block_diag([P[f"W_self.{l}.{i}"] for i in range(3)])
        b = np.concatenate([P[f"b.{l}.{i}"] for i in range(3)])
        bs = np.concatenate([P[f"b_self.{l}.{i}"] for i in range(3)])
        h = np.maximum(b + ah @ h @ Wa, 0.0) + h @ Ws + bs
    h = h + P["E"].reshape(-1)
    np.testing.assert_allclose(c[f"H{m.num_layers}"], h, rtol=1e-11, atol=1e-12)
    logits = np.maximum(h @ P["Wc1"] + P["bc1"], 0.0) @ P["Wc2"] + P["bc2"]
    np.testing.assert_allclose(c["logits"], logits, rtol=1e-11, atol=1e-12)


def test_overlapping_slices_and_feature_fusion_inputs():
    g, m, X, y, P = _tiny_problem(in_d=10, p=3, hidden=6)
    assert m.slices == [(0, 4), (4, 8), (6, 10)]
    c = orc.forward(m, g, X, P)
    ah = _dense_ahat(g)
    for i, (s, e) in enumerate(m.slices):
        want = np.maximum(P[f"b.0.{i}"] + ah @ X[:, s:e] @ P[f"W_agg.0.{i}"], 0.0) + X[:, s:e] @ P[f"W_self.0.{i}"]
        np.testing.assert_allclose(c["H1"][:, i * 2:(i + 1) * 2], want, rtol=1e-12, atol=1e-12)
    # feature fusion: one MLP d' -> d' -> slice_size, the same X_ff given to every slice
    g, m, X, y, P = _tiny_problem(in_d=10, p=3, hidden=6, use_ff=True)
    c = orc.forward(m, g, X, P)
    xff = np.maximum(X @ P["ff_W1"] + P["ff_b1"], 0.0) @ P["ff_W2"] + P["ff_b2"]
    assert xff.shape == (g.n, 4)
    np.testing.assert_allclose(c["H0"], xff, rtol=1e-12)
    for i in range(3):
        want = np.maximum(P[f"b.0.{i}"] + ah @ xff @ P[f"W_agg.0.{i}"], 0.0) + xff @ P[f"W_self.0.{i}"]
        np.testing.assert_allclose(c["H1"][:, i * 2:(i + 1) * 2], want, rtol=1e-11, atol=1e-12)


def test_cross_entropy_uniform_logits():
    g, m, X, y, P = _tiny_problem(C=5)
    P["Wc2"][:] = 0.0; P["bc2"][:] = 0.0
    c = orc.forward(m, g, X, P, y)
    assert abs(c["loss"] - math.log(5)) < 1e-12
    grads = orc.backward(m, g, X, P, y, c)
    # d logits = (softmax - onehot)/|V_L|: bias gradient is (1/C - class frequency)
    freq = np.bincount(y, minlength=5) / g.n
    np.testing.assert_allclose(grads["bc2"], 1.0 / 5 - freq, atol=1e-14)
    # nodes outside the training set get no gradient
    idx = np.arange(0, g.n, 3)
    c2 = orc.forward(m, g, X, P, y, idx)
    g2 = orc.backward(m, g, X, P, y, c2)
    freq2 = np.bincount(y[idx], minlength=5) / idx.size
    np.testing.assert_allclose(g2["bc2"], 1.0 / 5 - freq2, atol=1e-14)


# ------------------------------------------------------------------ backward: finite differences

@pytest.mark.parametrize("kw", [
    dict(p=1, use_self=False),
    dict(p=2),
    dict(p=3, in_d=10, hidden=6, use_se=True),                     # overlapping slices
    dict(p=3, in_d=10, hidden=6, use_ff=True, use_se=True),        # shared X_ff: gradients add
    dict(p=2, use_b_self=True, self_loops=False),
    dict(p=2, L=3, use_ff=True),
])
@pytest.mark.parametrize("order", ["agg", "xform"])
def test_backward_matches_finite_differences(kw, order):
    g, m, X, y, P = _tiny_problem(n=24, m_edges=60, seed=11, **kw)
    idx = np.arange(0, g.n, 2)
    orders = [order] * m.num_layers
    c = orc.forward(m, g, X, P, y, idx, order=orders)
    G = orc.backward(m, g, X, P, y, c)
    rng = np.random.default_rng(0)
    eps = 1e-6
    for name in P:
        flat = P[name].reshape(-1)
        picks = rng.choice(flat.size, size=min(6, flat.size), replace=False)
        for k in picks:
            old = flat[k]
            flat[k] = old + eps; lp = orc.loss_only(m, g, X, P, y, idx, orders)
            flat[k] = old - eps; lm = orc.loss_only(m, g, X, P, y, idx, orders)
            flat[k] = old
            fd = (lp - lm) / (2 * eps)
            an = G[name].reshape(-1)[k]
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (name, k, fd, an)


def test_backward_storage_rounding_acts_only_where_named():
    """The bf16 rounding point of the backward pass (dZ of an aggregate-first layer) is an explicit input: nothing is
    rounded unless named; naming layer 1's dZ moves only what lies below it, by no more than the rounding
    (2^-8 relative per element); a name that does not exist in the schedule is an error."""
    g, m, X, y, P = _tiny_problem(p=2, L=2)
    c = orc.forward(m, g, X, P, y, order=["agg", "agg"])
    ref = orc.backward(m, g, X, P, y, c)
    # rnd alone rounds nothing
    quiet = orc.backward(m, g, X, P, y, c, rnd=orc.round_bf16)
    assert all(np.array_equal(ref[k], quiet[k]) for k in ref)
    rb = orc.backward(m, g, X, P, y, c, rnd=orc.round_bf16, rnd_at={"dZ.1"})
    # only what lies below the rounded dZ of layer 1 (the gradients of layer 0) may move
    for k in ref:
        if k.endswith(".1.0") or k.endswith(".1.1") or k in ("Wc1", "bc1", "Wc2", "bc2"):
            assert np.array_equal(ref[k], rb[k]), k
    moved = [k for k in ref if not np.array_equal(ref[k], rb[k])]
    assert any(k.startswith("W_agg.0") for k in moved) and "H0" in moved
    for k in moved:
        assert np.abs(rb[k] - ref[k]).max() <= 2.0 ** -7 * np.abs(ref[k]).max(), k
    # layer 0's dZ only reaches the input gradient
    r0 = orc.backward(m, g, X, P, y, c, rnd=orc.round_bf16, rnd_at={"dZ.0"})
    assert [k for k in ref if not np.array_equal(ref[k], r0[k])] == ["H0"]
    # transform-first: no dZ exists
    cx = orc.forward(m, g, X, P, y, order=["xform", "xform"])
    with pytest.raises(ValueError):
        orc.backward(m, g, X, P, y, cx, rnd=orc.round_bf16, rnd_at={"dZ.0"})
    with pytest.raises(ValueError):
        orc.backward(m, g, X, P, y, c, rnd=orc.round_bf16, rnd_at={"dH.1"})


def _is_bf16(a):
    return np.array_equal(orc.round_bf16(a), np.asarray(a, np.float64))


def test_forward_storage_rounding_points():
    """Which tensors a bf16-stored forward pass keeps in the storage type: exactly the named ones are
    bf16-representable afterwards, pre-activations and logits never are, and the rounding function is called once
    per named store."""
    g, m, X, y, P = _tiny_problem(p=2, L=2, use_ff=True, use_se=True)
    order = ["agg", "xform"]
    pts = orc.forward_rounding_points(m, order)
    assert pts == {"ff_act", "X_ff", "Z.0", "T.1", "H.1", "H.2", "cls_act"}
    calls = []

    def counting(v):
        calls.append(v.shape)
        return orc.round_bf16(v)

    Xr = orc.round_bf16(X)
    c = orc.forward(m, g, Xr, P, y, rnd=counting, order=order)          # default: every point of the schedule
    # ff_act, X_ff, Z.0 and T.1 once per slice (2 each), H.1, H.2, cls_act
    assert len(calls) == 2 + 2 + 2 + 3
    stored = ["ff_act", "H0", "Z.0.0", "Z.0.1", "T.1.0", "T.1.1", "H1", "H2", "cls_act"]
    full = ["ff_pre", "M.0.0", "M.1.1", "cls_pre", "logits"]
    assert all(_is_bf16(c[k]) for k in stored)
    assert not any(_is_bf16(c[k]) for k in full)
    # a subset: only H.1 is rounded, everything else keeps full precision
    c1 = orc.forward(m, g, Xr, P, y, rnd=orc.round_bf16, order=order, rnd_at={"H.1"})
    assert _is_bf16(c1["H1"]) and not any(_is_bf16(c1[k]) for k in ["ff_act", "H0", "Z.0.0", "T.1.0", "H2", "cls_act"])
    # no point named = the fp64 pass; a rounded pass differs from it by no more than a few roundings
    c0 = orc.forward(m, g, Xr, P, y, rnd=orc.round_bf16, order=order, rnd_at=())
    cf = orc.forward(m, g, Xr, P, y, order=order)
    assert np.array_equal(c0["logits"], cf["logits"])
    assert 0 < np.abs(c["logits"] - cf["logits"]).max() <= 0.05 * np.abs(cf["logits"]).max()
    with pytest.raises(ValueError):
        orc.forward(m, g, Xr, P, y, rnd=orc.round_bf16, order=order, rnd_at={"Z.1"})   # layer 1 stores T, not Z


def test_order_of_aggregate_and_transform_is_immaterial():
    g, m, X, y, P = _tiny_problem(p=2, use_se=True)
    a = orc.forward(m, g, X, P, y, order=["agg", "agg"])
    b = orc.forward(m, g, X, P, y, order=["xform", "xform"])
    np.testing.assert_allclose(a["logits"], b["logits"], rtol=1e-11, atol=1e-13)
    ga = orc.backward(m, g, X, P, y, a); gb = orc.backward(m, g, X, P, y, b)
    for k in ga:
        np.testing.assert_allclose(ga[k], gb[k], rtol=1e-9, atol=1e-13)


# ------------------------------------------------------------------ optimiser

def test_adam_first_step_and_cosine():
    g = np.array([0.3, -2.0, 1e-3]); th = np.array([1.0, 1.0, 1.0])
    new, m1, m2 = orc.adam_step(th, g, np.zeros(3), np.zeros(3), 1, lr=0.01)
    # bias-corrected first step: delta = -lr * g / (|g| + eps)
    np.testing.assert_allclose(new - th, -0.01 * g / (np.abs(g) + 1e-8), rtol=1e-12)
    np.testing.assert_allclose(m1, 0.1 * g); np.testing.assert_allclose(m2, 0.001 * g * g)
    assert orc.cosine_lr(1e-3, 0, 500) == 1e-3
    assert abs(orc.cosine_lr(1e-3, 250, 500) - 0.5e-3) < 1e-18
    assert abs(orc.cosine_lr(1e-3, 500, 500)) < 1e-18
    # weight decay enters as an L2 term added to the gradient
    new_wd, _, _ = orc.adam_step(th, np.zeros(3), np.zeros(3), np.zeros(3), 1, lr=0.01, weight_decay=0.1)
    np.testing.assert_allclose(new_wd - th, -0.01 * 0.1 / (0.1 + 1e-8), rtol=1e-12)


def _read_update_golden():
    d = {}
    for line in open(os.path.join(GOLDEN, "two_epoch_update.txt")):
        t = line.split()
        if t and not t[0].startswith("#"):
            d[t[0]] = [float(v) for v in t[1:]]
    return d


def test_epoch_update_two_epochs_worked_by_hand():
    """Which index feeds the rate and which the step count (hand-worked values): a rate taken at epoch + 1 or a step
    count taken at epoch would both miss them."""
    d = _read_update_golden()
    P = {"theta": np.array(d["theta0"])}
    st = {"m1": {}, "m2": {}}
    T = int(d["total_epochs"][0])
    assert abs(orc.cosine_lr(d["lr0"][0], 0, T) - d["lr_epoch0"][0]) < 1e-12
    assert abs(orc.cosine_lr(d["lr0"][0], 1, T) - d["lr_epoch1"][0]) < 1e-8
    orc.apply_update(P, {"theta": np.array(d["g0"])}, st, d["lr0"][0], 0, T)
    np.testing.assert_allclose(P["theta"], d["theta1"], atol=1e-7)
    orc.apply_update(P, {"theta": np.array(d["g1"])}, st, d["lr0"][0], 1, T)
    np.testing.assert_allclose(P["theta"], d["theta2"], atol=1e-7)


def test_train_epoch_is_forward_backward_update():
    """train_epoch = forward, backward, then the update pinned above, on the parameters as they were before it:
    epoch 0's step is the first-step closed form at the FULL rate lr0; epoch 1 (of 2) uses lr0/2 and step 2."""
    g, m, X, y, P = _tiny_problem(n=30, m_edges=80, p=2, use_se=True)
    P0 = {k: v.copy() for k, v in P.items()}
    st = {"m1": {}, "m2": {}}
    lr0 = 0.05
    loss0, logits0, G0 = orc.train_epoch(m, g, X, P, y, st, lr0, 0, 2)
    c = orc.forward(m, g, X, P0, y)
    assert loss0 == c["loss"] and np.array_equal(logits0, c["logits"])      # loss and logits BEFORE the update
    Gref = orc.backward(m, g, X, P0, y, c)
    for k in P0:
        assert np.array_equal(G0[k], Gref[k])
        np.testing.assert_allclose(P[k], P0[k] - lr0 * Gref[k] / (np.abs(Gref[k]) + 1e-8), rtol=0, atol=1e-12)
    P1 = {k: v.copy() for k, v in P.items()}
    _, _, G1 = orc.train_epoch(m, g, X, P, y, st, lr0, 1, 2)
    for k in P0:    # step 2 written out: 1 - 0.9^2 = 0.19, 1 - 0.999^2 = 0.001999; rate lr0/2 (cos(pi/2) = 0)
        mh = (0.09 * G0[k] + 0.1 * G1[k]) / 0.19
        vh = (0.000999 * G0[k] ** 2 + 0.001 * G1[k] ** 2) / 0.001999
        np.testing.assert_allclose(P[k], P1[k] - 0.5 * lr0 * mh / (np.sqrt(vh) + 1e-8), rtol=0, atol=1e-12)


def test_dropout_mask_between_layers():
    """Dropout as an explicit 0/1 mask on the output of layer l < L, kept units scaled by 1/(1 - rate): a mask of
    ones at rate 0 changes nothing; dropped units pass neither value nor gradient; finite differences hold."""
    g, m, X, y, P = _tiny_problem(n=24, m_edges=60, p=2, L=3, seed=4)
    base = orc.forward(m, g, X, P, y)
    ones = {1: np.ones((g.n, m.p * m.h_s), np.uint8), 2: np.ones((g.n, m.p * m.h_s), np.uint8)}
    same = orc.forward(m, g, X, P, y, dropout=ones, drop_rate=0.0)
    assert np.array_equal(same["logits"], base["logits"])
    rng = np.random.default_rng(0)
    masks = {1: (rng.random((g.n, m.p * m.h_s)) >= 0.5).astype(np.uint8), 2: (rng.random((g.n, m.p * m.h_s)) >= 0.5).astype(np.uint8)}
    c = orc.forward(m, g, X, P, y, dropout=masks, drop_rate=0.5)
    assert np.all(c["H1"][masks[1] == 0] == 0) and np.all(c["H2"][masks[2] == 0] == 0)
    kept = masks[1] == 1
    # kept units are the undropped layer output times 1/(1 - 0.5)
    np.testing.assert_allclose(c["H1"][kept], 2.0 * base["H1"][kept], rtol=1e-13)
    G = orc.backward(m, g, X, P, y, c)
    eps = 1e-6
    for name in ("W_agg.0.1", "W_self.1.0", "b.0.0", "Wc1"):
        flat = P[name].reshape(-1)
        for k in (0, flat.size // 2):
            old = flat[k]
            flat[k] = old + eps; lp = orc.forward(m, g, X, P, y, dropout=masks, drop_rate=0.5)["loss"]
            flat[k] = old - eps; lm = orc.forward(m, g, X, P, y, dropout=masks, drop_rate=0.5)["loss"]
            flat[k] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - G[name].reshape(-1)[k]) <= 1e-6 * max(1.0, abs(fd)) + 1e-8, (name, k)
    with pytest.raises(ValueError):
        orc.forward(m, g, X, P, y, dropout={3: ones[1]}, drop_rate=0.5)     # no layer reads the last layer's output


def test_train_epoch_decreases_loss():
    g, m, X, y, P = _tiny_problem(n=60, m_edges=200, p=2, use_se=True)
    st = {"m1": {}, "m2": {}}
    losses = [orc.train_epoch(m, g, X, P, y, st, 0.01, ep, 30)[0] for ep in range(30)]
    assert losses[-1] < losses[0] - 0.05
