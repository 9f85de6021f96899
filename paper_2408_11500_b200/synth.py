"""Seeded synthetic inputs: graphs, features, labels, initial parameters.

Everything here is plain random-number plumbing (numpy's counter-based Philox
generator keyed by (seed, stream)); it holds none of the method's arithmetic,
so both the CUDA path and the CPU oracle can be fed from it.  The graphs take
the sizes and degree structure of node-classification workloads (power-law
citation / co-purchase graphs, a dense log-normal social graph, R-MAT) and
stand in for the public datasets of those shapes, which are not used.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


# --------------------------------------------------------------------------
# graphs (undirected edge lists without self pairs or repeats)
# --------------------------------------------------------------------------

def _inverse_cdf(cdf: np.ndarray, q: np.ndarray) -> np.ndarray:
    """searchsorted(cdf, q, side="right") as int64, through a table of the answers at 2^20 evenly spaced points:
    the answer for q starts at the table entry of q's bucket and moves up while cdf[answer] <= q (a few vector
    passes instead of one cache-missing binary search per query; identical results)."""
    nb = 1 << 20
    table = np.searchsorted(cdf, np.arange(nb, dtype=np.float64) / nb, side="right").astype(np.int64)
    out = table[np.minimum((q * nb).astype(np.int64), nb - 1)]
    n = cdf.size
    todo = np.flatnonzero(cdf[np.minimum(out, n - 1)] <= q)
    todo = todo[out[todo] < n]
    while todo.size:
        out[todo] += 1
        nxt = out[todo]
        more = nxt < n
        more[more] = cdf[nxt[more]] <= q[todo[more]]
        todo = todo[more]
    return out


def _sample_pairs(n: int, weights: np.ndarray, m: int, rng: np.random.Generator) -> Tuple[np.ndarray, np.ndarray]:
    """m distinct unordered pairs {u, v}, u != v, endpoints drawn in proportion to weights."""
    cdf = np.cumsum(weights, dtype=np.float64)
    cdf /= cdf[-1]
    keys = np.empty(0, dtype=np.int64)
    rounds = 0
    while keys.size < m:
        need = m - keys.size
        batch = int(need * 1.15) + 1024
        u = _inverse_cdf(cdf, rng.random(batch))
        v = _inverse_cdf(cdf, rng.random(batch))
        np.minimum(u, n - 1, out=u)
        np.minimum(v, n - 1, out=v)
        ok = u != v
        lo = np.minimum(u[ok], v[ok])
        hi = np.maximum(u[ok], v[ok])
        keys = np.sort(np.concatenate([keys, lo * n + hi]))       # sorted union of the distinct pairs so far
        keys = keys[np.concatenate(([True], keys[1:] != keys[:-1]))]
        rounds += 1
        if rounds > 200:
            raise RuntimeError("edge sampler did not reach the requested edge count")
    if keys.size > m:                       # drop a seeded random subset, not the sorted tail
        keep = rng.permutation(keys.size)[:m]
        keys = keys[np.sort(keep)]
    return (keys // n).astype(np.int32), (keys % n).astype(np.int32)


def _powerlaw_weights(n: int, m: int, gamma: float, max_degree: float) -> np.ndarray:
    """w_i = (i + i0)^(-1/(gamma-1)); i0 set by bisection so the largest expected degree is max_degree."""
    expo = -1.0 / (gamma - 1.0)
    idx = np.arange(n, dtype=np.float64)

    def top(i0):
        w = (idx + i0) ** expo
        return 2.0 * m * w[0] / w.sum()

    lo, hi = 1e-3, float(n)
    if top(lo) <= max_degree:
        return (idx + lo) ** expo
    for _ in range(100):
        mid = 0.5 * (lo + hi)
        if top(mid) > max_degree:
            lo = mid
        else:
            hi = mid
    return (idx + hi) ** expo


def chung_lu_powerlaw(n: int, m_undirected: int, gamma: float = 2.2, max_degree: float = 1e4, seed: int = 0,
                      shuffle_ids: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """Chung-Lu graph with a power-law expected-degree sequence.  With shuffle_ids the node ids are
    a seeded random permutation, so hubs are not packed at low ids."""
    rng = _rng(seed, 1)
    w = _powerlaw_weights(n, m_undirected, gamma, max_degree)
    src, dst = _sample_pairs(n, w, m_undirected, rng)
    if shuffle_ids:
        perm = _rng(seed, 2).permutation(n).astype(np.int32)
        src, dst = perm[src], perm[dst]
    return src, dst


def chung_lu_lognormal(n: int, m_undirected: int, sigma: float = 1.0, seed: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Chung-Lu graph whose expected degrees are log-normal (dense social-graph shape)."""
    w = np.exp(sigma * _rng(seed, 3).standard_normal(n))
    return _sample_pairs(n, w, m_undirected, _rng(seed, 4))


def rmat(scale: int, edge_factor: int = 16, a: float = 0.57, b: float = 0.19, c: float = 0.19, seed: int = 0,
         relabel: bool = False, chunk: int = 1 << 22) -> Tuple[int, np.ndarray, np.ndarray]:
    """R-MAT edge list (n = 2^scale, edge_factor * n draws); self pairs dropped, repeats kept
    (graph construction merges them).  Returns (n, src, dst)."""
    n = 1 << scale
    m = edge_factor * n
    rng = _rng(seed, 5)
    t1, t2, t3 = a, a + b, a + b + c
    srcs, dsts = [], []
    for start in range(0, m, chunk):
        k = min(chunk, m - start)
        u = np.zeros(k, dtype=np.int64)
        v = np.zeros(k, dtype=np.int64)
        for _ in range(scale):
            r = rng.random(k, dtype=np.float32)
            right = ((r >= t1) & (r < t2)) | (r >= t3)     # quadrants b and d: column bit set
            down = r >= t2                                   # quadrants c and d: row bit set
            u = (u << 1) | down
            v = (v << 1) | right
        ok = u != v
        srcs.append(u[ok].astype(np.int32))
        dsts.append(v[ok].astype(np.int32))
    src, dst = np.concatenate(srcs), np.concatenate(dsts)
    if relabel:
        src, dst = random_relabel(n, src, dst, seed)
    return n, src, dst


def random_relabel(n: int, src: np.ndarray, dst: np.ndarray, seed: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """The same edge list under a seeded random permutation of the node ids (R-MAT's natural ids put the
    hubs at low ids, which flatters locality)."""
    perm = _rng(seed, 6).permutation(n).astype(np.int32)
    return perm[src], perm[dst]


# --------------------------------------------------------------------------
# features, labels, parameters
# --------------------------------------------------------------------------

def gaussian_features(n: int, d: int, seed: int = 0) -> np.ndarray:
    return _rng(seed, 10).standard_normal((n, d), dtype=np.float32)


def binary_features(n: int, d: int, density: float = 0.013, seed: int = 0) -> np.ndarray:
    return (_rng(seed, 11).random((n, d), dtype=np.float32) < density).astype(np.float32)


def uniform_labels(n: int, num_classes: int, seed: int = 0) -> np.ndarray:
    return _rng(seed, 12).integers(0, num_classes, size=n, dtype=np.int32)


def init_params(shapes: Dict[str, Tuple[int, ...]], seed: int = 0, bias_scale: float = 0.0,
                se_scale: float = 0.0) -> Dict[str, np.ndarray]:
    """Glorot-uniform matrices; vectors (biases) and the slice-encoding table are zero unless a
    scale is given (tests use non-zero scales so every term is exercised)."""
    rng = _rng(seed, 20)
    out = {}
    for name, shp in shapes.items():
        if name == "E":
            out[name] = (se_scale * rng.standard_normal(shp)).astype(np.float32)
        elif len(shp) == 2:
            lim = np.sqrt(6.0 / (shp[0] + shp[1]))
            out[name] = rng.uniform(-lim, lim, size=shp).astype(np.float32)
        else:
            out[name] = (bias_scale * rng.standard_normal(shp)).astype(np.float32)
    return out


# --------------------------------------------------------------------------
# the named workloads
# --------------------------------------------------------------------------

WORKLOADS = {
    # name: graph recipe + model shape (see the design notes for the full recipe)
    "tiny": dict(n=2708, m=5278, gen="powerlaw", gamma=2.2, max_degree=168, in_d=1433, feat="binary",
                 classes=7, layers=2, hidden=16, p=4, dtype="f32", use_ff=False, use_se=False),
    "citation": dict(n=169343, m=1166243, gen="powerlaw", gamma=2.2, max_degree=13000, in_d=128, feat="gauss",
                     classes=40, layers=3, hidden=256, p=8, dtype="f32", use_ff=False, use_se=False),
    "social": dict(n=232965, m=57300000, gen="lognormal", sigma=1.0, in_d=602, feat="gauss",
                   classes=41, layers=2, hidden=256, p=4, dtype="f32", use_ff=False, use_se=False),
    "copurchase": dict(n=2449029, m=61859140, gen="powerlaw", gamma=2.2, max_degree=20000, in_d=100, feat="gauss",
                       classes=47, layers=3, hidden=256, p=8, dtype="bf16", use_ff=True, use_se=True),
}


# Seeded graphs with the sizes of the paper's Table I (nodes, undirected edges, features, classes) and the layer
# count and dropout rate of its Table II; width 512 as its Table III implies.  Only the sizes are the paper's: the
# edges are Chung-Lu power-law draws like the other workloads, the features Gaussian, the labels uniform.
TABLE1_SHAPES = {
    "t1_22662": dict(n=22662, m=32927, in_d=300, classes=18, layers=3, dropout=0.5),
    "t1_24492": dict(n=24492, m=93050, in_d=300, classes=5, layers=4, dropout=0.5),
    "t1_10000": dict(n=10000, m=39402, in_d=7, classes=2, layers=7, dropout=0.5),
    "t1_11758": dict(n=11758, m=519000, in_d=10, classes=2, layers=4, dropout=0.5),
    "t1_48921": dict(n=48921, m=153540, in_d=301, classes=2, layers=6, dropout=0.5),
    "t1_169343": dict(n=169343, m=1166243, in_d=128, classes=40, layers=4, dropout=0.0),
}


def table1_workload(name: str) -> dict:
    t = TABLE1_SHAPES[name]
    mean_deg = 2.0 * t["m"] / t["n"]
    return dict(n=t["n"], m=t["m"], gen="powerlaw", gamma=2.2, max_degree=min(t["n"] / 8.0, max(64.0, 60.0 * mean_deg)),
                in_d=t["in_d"], feat="gauss", classes=t["classes"], layers=t["layers"], hidden=512, p=2, dtype="f32",
                use_ff=False, use_se=False, dropout=t["dropout"])


def make_graph(w: dict, seed: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    if w["gen"] == "powerlaw":
        return chung_lu_powerlaw(w["n"], w["m"], w["gamma"], w["max_degree"], seed)
    if w["gen"] == "lognormal":
        return chung_lu_lognormal(w["n"], w["m"], w["sigma"], seed)
    raise ValueError(w["gen"])


def make_features(w: dict, seed: int = 0) -> np.ndarray:
    if w["feat"] == "binary":
        return binary_features(w["n"], w["in_d"], seed=seed)
    return gaussian_features(w["n"], w["in_d"], seed=seed)
