"""Seeded synthetic inputs: vectors, attributes, proximity graph, queries, ranges.

Everything here is input preparation.  Random numbers come from numpy's
`Generator(PCG64)` with one independent child stream per array
(`SeedSequence(seed).spawn`), always drawn on the CPU, so the same seed gives
the same vectors, attributes, queries and ranges everywhere.  The proximity
graph is a fixture too: nearest-neighbour candidates are found by blocked brute
force with torch (on the GPU when one is present, purely as a data-preparation
tool), which for the integer-valued workloads is exact and therefore
device-independent.

Attribute cells are 4 bytes each.  A float32 column is stored bit-cast inside
the int32 matrix; `attr_types[j]` says how to read column j (0 = int32,
1 = float32).  Range bounds use the same encoding and are closed intervals.
"""
from __future__ import annotations

import math
from typing import Dict

import numpy as np
import torch

from .configs import Workload

SENTINEL = np.uint32(0xFFFFFFFF)
ATTR_I32, ATTR_F32 = 0, 1


# ----------------------------------------------------------------------------
# vectors
# ----------------------------------------------------------------------------
def _latent_mixture(w: Workload, n: int, cluster: np.ndarray, centres: np.ndarray,
                    proj: np.ndarray, rng: np.random.Generator) -> np.ndarray:
    """Points near a dz-dimensional subspace: latent cluster draw, orthonormal
    embedding into D dimensions, plus a little isotropic ambient noise."""
    out = np.empty((n, w.D), dtype=np.float32)
    step = 1 << 18
    for s in range(0, n, step):
        e = min(n, s + step)
        z = centres[cluster[s:e]] + w.sigma_l * rng.standard_normal((e - s, w.dz), dtype=np.float32)
        x = z @ proj
        x += w.sigma_n * rng.standard_normal((e - s, w.D), dtype=np.float32)
        out[s:e] = x
    return out


def _finish_vectors(w: Workload, x: np.ndarray) -> np.ndarray:
    if w.vec_kind == "int_latent":
        # per-dimension std of x is about sqrt(dz/D) * sqrt(spread^2 + sigma_l^2);
        # map it to about 40 grey levels around 128, then round and clip to 0..255
        std = math.sqrt(w.dz / w.D) * math.sqrt(w.spread ** 2 + w.sigma_l ** 2)
        x = np.clip(np.rint(128.0 + (40.0 / std) * x), 0, 255)
        return x.astype(np.uint8) if w.vec_dtype == "u8" else x.astype(np.float32)
    if w.vec_kind == "unit_latent":
        # shift away from the origin so that normalising keeps the cluster structure
        x = x + np.float32(0.5 / math.sqrt(w.D))
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        return x.astype(np.float32)
    return x.astype(np.float32)


def _make_vectors(w: Workload, ss_data, ss_query):
    rng = np.random.default_rng(ss_data)
    rq = np.random.default_rng(ss_query)
    if w.vec_kind == "gauss":
        centres = rng.standard_normal((w.n_clusters, w.D)).astype(np.float32)
        cl = rng.integers(0, w.n_clusters, size=w.N)
        x = centres[cl] + np.float32(0.3) * rng.standard_normal((w.N, w.D), dtype=np.float32)
        qcl = rq.integers(0, w.n_clusters, size=w.Q)
        q = centres[qcl] + np.float32(0.3) * rq.standard_normal((w.Q, w.D), dtype=np.float32)
        return x.astype(np.float32), q.astype(np.float32), cl.astype(np.int32), centres
    centres = (w.spread * rng.standard_normal((w.n_clusters, w.dz))).astype(np.float32)
    a = rng.standard_normal((w.D, w.dz))
    proj = np.linalg.qr(a)[0].T.astype(np.float32)          # dz x D, orthonormal rows
    cl = rng.integers(0, w.n_clusters, size=w.N)
    x = _finish_vectors(w, _latent_mixture(w, w.N, cl, centres, proj, rng))
    qcl = rq.integers(0, w.n_clusters, size=w.Q)
    q = _finish_vectors(w, _latent_mixture(w, w.Q, qcl, centres, proj, rq)).astype(np.float32)
    return x, q, cl.astype(np.int32), centres


# ----------------------------------------------------------------------------
# attributes and ranges
# ----------------------------------------------------------------------------
def _make_attr_column(kind: str, w: Workload, cl: np.ndarray, rng: np.random.Generator):
    n = w.N
    if kind == "uniform_int_1000":
        return rng.integers(0, 1000, size=n).astype(np.int32), ATTR_I32
    if kind == "uniform_int":
        return rng.integers(0, 1 << 20, size=n).astype(np.int32), ATTR_I32
    if kind == "timestamp":
        t = np.arange(n, dtype=np.float64) + np.rint(0.05 * n * rng.standard_normal(n))
        return t.astype(np.int64).astype(np.int32), ATTR_I32
    if kind == "zipf_cat":
        z = rng.zipf(1.1, size=n)
        return np.minimum(z, 10_000).astype(np.int32), ATTR_I32
    if kind == "uniform_float":
        return rng.random(n, dtype=np.float32).view(np.int32), ATTR_F32
    if kind == "cluster_corr_int":
        zc = np.random.default_rng(12345).standard_normal(w.n_clusters)
        v = 0.7 * zc[cl] + math.sqrt(0.51) * rng.standard_normal(n)
        return np.rint(1000.0 * v).astype(np.int32), ATTR_I32
    raise ValueError(kind)


def _column_values(col: np.ndarray, t: int) -> np.ndarray:
    return col.view(np.float32) if t == ATTR_F32 else col


def _make_ranges(w: Workload, attrs: np.ndarray, types: np.ndarray, rng: np.random.Generator):
    q, m, n = w.Q, w.m, w.N
    lo = np.empty((q, m), dtype=np.int32)
    hi = np.empty((q, m), dtype=np.int32)
    if w.sel_kind == "window":
        # one window of ~sel_lo of the value domain per query, placed uniformly
        for j in range(m):
            vals = _column_values(attrs[:, j], types[j])
            vmin, vmax = int(vals.min()), int(vals.max())
            width = max(1, int(round(w.sel_lo * (vmax - vmin + 1))))
            start = rng.integers(vmin, vmax - width + 2, size=q)
            lo[:, j] = start
            hi[:, j] = start + width - 1
        return lo, hi, np.full(q, w.sel_lo)
    if w.sel_kind == "loguniform":
        s = np.exp(rng.uniform(math.log(w.sel_lo), math.log(w.sel_hi), size=q))
    elif w.sel_kind == "mixture":
        easy = rng.random(q) < 0.5
        s = np.where(easy,
                     np.exp(rng.uniform(math.log(0.20), math.log(w.sel_hi), size=q)),
                     np.exp(rng.uniform(math.log(w.sel_lo), math.log(0.02), size=q)))
    else:
        raise ValueError(w.sel_kind)
    sj = s ** (1.0 / m)
    for j in range(m):
        vals = np.sort(_column_values(attrs[:, j], types[j]))
        u = rng.random(q) * (1.0 - sj)
        i0 = np.minimum((u * (n - 1)).astype(np.int64), n - 1)
        i1 = np.minimum(((u + sj) * (n - 1)).astype(np.int64), n - 1)
        l, h = vals[i0], vals[i1]
        if types[j] == ATTR_F32:
            lo[:, j] = l.astype(np.float32).view(np.int32)
            hi[:, j] = h.astype(np.float32).view(np.int32)
        else:
            lo[:, j] = l
            hi[:, j] = h
    return lo, hi, s


# ----------------------------------------------------------------------------
# proximity graph fixture
# ----------------------------------------------------------------------------
def _prep_device(device: str | None) -> torch.device:
    if device is None:
        device = "cuda" if torch.cuda.is_available() else "cpu"
    if str(device).startswith("cuda"):
        torch.backends.cuda.matmul.allow_tf32 = False
    return torch.device(device)


def _sq_dists(x: torch.Tensor, xn: torch.Tensor, y: torch.Tensor, yn: torch.Tensor) -> torch.Tensor:
    d = torch.mm(x, y.t())
    d.mul_(-2.0).add_(xn[:, None]).add_(yn[None, :])
    return d


def exact_knn_graph(vectors: np.ndarray, R: int, device: str | None = None) -> np.ndarray:
    """Exact R nearest neighbours of every point (no self), by blocked brute force."""
    dev = _prep_device(device)
    x = torch.from_numpy(np.ascontiguousarray(vectors.astype(np.float32))).to(dev)
    xn = (x * x).sum(1)
    n = x.shape[0]
    out = np.empty((n, R), dtype=np.uint32)
    blk = max(256, min(8192, (1 << 28) // max(1, n)))
    for s in range(0, n, blk):
        e = min(n, s + blk)
        d = _sq_dists(x[s:e], xn[s:e], x, xn)
        d[torch.arange(e - s, device=dev), torch.arange(s, e, device=dev)] = float("inf")
        idx = torch.topk(d, R, dim=1, largest=False, sorted=True).indices
        out[s:e] = idx.cpu().numpy().astype(np.uint32)
    return out


def _attr_cells(attrs: np.ndarray, types: np.ndarray, frac: float) -> np.ndarray:
    """Cell id of every point on a rank-quantile grid holding ~frac of the data per cell."""
    n, m = attrs.shape
    g = max(1, int(round(frac ** (-1.0 / m))))
    cell = np.zeros(n, dtype=np.int64)
    for j in range(m):
        vals = _column_values(attrs[:, j], types[j])
        order = np.argsort(vals, kind="stable")
        rank = np.empty(n, dtype=np.int64)
        rank[order] = np.arange(n)
        cell = cell * g + np.minimum(rank * g // n, g - 1)
    return cell


def mixed_graph(w: Workload, vectors: np.ndarray, attrs: np.ndarray, types: np.ndarray,
                cl: np.ndarray, centres: np.ndarray, ss_graph, device: str | None = None) -> np.ndarray:
    """Degree-R fixture: approximate kNN (exact among the points of the t_near
    nearest clusters), optional attribute-cell neighbours, and multi-scale long
    edges to random points of clusters at log-uniformly drawn centre ranks."""
    dev = _prep_device(device)
    rng = np.random.default_rng(ss_graph)
    n, R, nc = w.N, w.R, w.n_clusters
    r_long = min(w.r_long, R - 1)
    r_attr = min(w.r_attr, R - r_long - 1)
    r_knn = R - r_long - r_attr
    order = np.argsort(cl, kind="stable")
    starts = np.searchsorted(cl[order], np.arange(nc + 1))
    cdist = ((centres[:, None, :] - centres[None, :, :]) ** 2).sum(-1) if nc <= 4096 else None
    if cdist is None:
        raise ValueError("too many clusters")
    crank = np.argsort(cdist, axis=1, kind="stable")        # crank[c][0] == c
    t_near = min(w.t_near, nc)
    cells = _attr_cells(attrs, types, w.attr_frac) if r_attr > 0 else None

    graph = np.full((n, R), SENTINEL, dtype=np.uint32)
    xs = torch.from_numpy(np.ascontiguousarray(vectors[order].astype(np.float32)))
    big = 3.0e38
    for c in range(nc):
        a, b = starts[c], starts[c + 1]
        if a == b:
            continue
        cand_parts = [np.arange(starts[t], starts[t + 1]) for t in crank[c, :t_near]]
        cand = np.concatenate(cand_parts)
        x = xs[a:b].to(dev)
        y = xs[torch.from_numpy(cand)].to(dev)
        d = _sq_dists(x, (x * x).sum(1), y, (y * y).sum(1))
        # candidates begin with this cluster's own rows, so self sits on the diagonal
        d[torch.arange(b - a, device=dev), torch.arange(b - a, device=dev)] = big
        kk = min(r_knn + r_attr, cand.shape[0] - 1)
        near = torch.topk(d, kk, dim=1, largest=False, sorted=True)
        near_idx = near.indices.cpu().numpy()
        rows = order[a:b]
        take = min(r_knn, kk)
        graph[rows, :take] = order[cand[near_idx[:, :take]]].astype(np.uint32)
        if r_attr > 0:
            cx = torch.from_numpy(cells[order[a:b]]).to(dev)
            cy = torch.from_numpy(cells[order[cand]]).to(dev)
            d.scatter_(1, near.indices[:, :take], big)
            d.masked_fill_(cx[:, None] != cy[None, :], big)
            ka = min(r_attr, cand.shape[0] - 1)
            an = torch.topk(d, ka, dim=1, largest=False, sorted=True)
            a_idx = an.indices.cpu().numpy()
            a_ok = (an.values < 1.0e38).cpu().numpy()
            picked = order[cand[a_idx]].astype(np.uint32)
            # where the cell ran out of points fall back to the next plain neighbours
            spare = order[cand[near_idx[:, take:take + ka]]].astype(np.uint32) if kk > take else None
            for t in range(ka):
                col = picked[:, t].copy()
                if spare is not None and t < spare.shape[1]:
                    col = np.where(a_ok[:, t], col, spare[:, t])
                else:
                    col = np.where(a_ok[:, t], col, SENTINEL)
                graph[rows, r_knn + t] = col
    # long edges: cluster rank drawn log-uniformly in [1, nc), random point inside it
    if r_long > 0 and nc > 1:
        u = rng.random((n, r_long))
        rank = np.minimum(np.floor(np.exp(u * math.log(nc))).astype(np.int64), nc - 1)
        rank = np.maximum(rank, 1)
        tgt_cluster = crank[cl[:, None], rank]
        size = (starts[1:] - starts[:-1])[tgt_cluster]
        off = np.minimum((rng.random((n, r_long)) * size).astype(np.int64), np.maximum(size - 1, 0))
        tgt = order[np.minimum(starts[tgt_cluster] + off, n - 1)].astype(np.uint32)
        tgt = np.where(size > 0, tgt, SENTINEL)
        graph[:, R - r_long:] = tgt
    return clean_rows(graph)


def clean_rows(graph: np.ndarray) -> np.ndarray:
    """Replace self references and repeated ids inside a row by the sentinel."""
    n, R = graph.shape
    g = graph.copy()
    g[g == np.arange(n, dtype=np.uint32)[:, None]] = SENTINEL
    for j in range(1, R):
        dup = (g[:, :j] == g[:, j:j + 1]).any(axis=1)
        g[dup, j] = SENTINEL
    return g


# ----------------------------------------------------------------------------
# entry point
# ----------------------------------------------------------------------------
def make_workload(w: Workload, seed: int = 0, device: str | None = None,
                  with_graph: bool = True) -> Dict[str, np.ndarray]:
    """Build every input array of workload `w` for `seed`."""
    ss = np.random.SeedSequence(seed).spawn(5)
    vectors, queries, cl, centres = _make_vectors(w, ss[0], ss[3])
    rng_a = np.random.default_rng(ss[1])
    cols, types = [], []
    for kind in w.attrs:
        c, t = _make_attr_column(kind, w, cl, rng_a)
        cols.append(c)
        types.append(t)
    attrs = np.ascontiguousarray(np.stack(cols, axis=1).astype(np.int32))
    types = np.asarray(types, dtype=np.int32)
    lo, hi, target_sel = _make_ranges(w, attrs, types, np.random.default_rng(ss[4]))
    out = dict(vectors=np.ascontiguousarray(vectors), queries=np.ascontiguousarray(queries),
               attrs=attrs, attr_types=types, lo=np.ascontiguousarray(lo),
               hi=np.ascontiguousarray(hi), target_sel=target_sel, cluster=cl)
    if with_graph:
        if w.graph == "exact_knn":
            g = exact_knn_graph(vectors, w.R, device)
        else:
            g = mixed_graph(w, vectors, attrs, types, cl, centres, ss[2], device)
        out["graph"] = np.ascontiguousarray(g)
    return out


def reachable_fraction(graph: np.ndarray, entry: int) -> float:
    """Fraction of nodes a breadth-first walk from `entry` reaches."""
    n = graph.shape[0]
    seen = np.zeros(n, dtype=bool)
    seen[entry] = True
    frontier = np.array([entry], dtype=np.int64)
    while frontier.size:
        nb = graph[frontier].reshape(-1)
        nb = nb[nb != SENTINEL].astype(np.int64)
        nb = np.unique(nb)
        nb = nb[~seen[nb]]
        seen[nb] = True
        frontier = nb
    return float(seen.mean())
