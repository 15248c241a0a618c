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

import hashlib
import math
import os
import tempfile
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


def _rank_columns(attrs: np.ndarray, types: np.ndarray) -> np.ndarray:
    """Rank of every point in every attribute column, scaled to [0, 1)."""
    n, m = attrs.shape
    out = np.empty((n, m), dtype=np.float32)
    for j in range(m):
        vals = _column_values(attrs[:, j], types[j])
        order = np.argsort(vals, kind="stable")
        rank = np.empty(n, dtype=np.int64)
        rank[order] = np.arange(n)
        out[:, j] = rank / float(n)
    return out


def _zorder(ranks01: np.ndarray, bits: int = 7) -> np.ndarray:
    """Morton code of the attribute rank vector (bits per attribute, interleaved)."""
    n, m = ranks01.shape
    q = np.minimum((ranks01 * (1 << bits)).astype(np.int64), (1 << bits) - 1)
    code = np.zeros(n, dtype=np.int64)
    for b in range(bits - 1, -1, -1):
        for j in range(m):
            code = (code << 1) | ((q[:, j] >> b) & 1)
    return code


def _diversify(x: torch.Tensor, y_all: torch.Tensor, cand_idx: torch.Tensor, cand_d: torch.Tensor,
               keep: int, alpha: float) -> torch.Tensor:
    """Occlusion pruning of sorted candidate lists: walking a list from near to far, a
    candidate survives unless an already kept one is alpha times closer to it than the
    node itself is.  Returns, per node, candidate slots reordered so that survivors come
    first (in distance order) followed by the pruned ones (in distance order)."""
    B, K = cand_idx.shape
    yc = y_all[cand_idx]                                   # B x K x D
    yn = (yc * yc).sum(-1)
    pd = yn[:, :, None] + yn[:, None, :] - 2.0 * torch.bmm(yc, yc.transpose(1, 2))
    alive = torch.ones((B, K), dtype=torch.bool, device=x.device)
    chosen = torch.zeros((B, K), dtype=torch.bool, device=x.device)
    count = torch.zeros(B, dtype=torch.int64, device=x.device)
    for t in range(K):
        take = alive[:, t] & (count < keep)
        chosen[:, t] = take
        count += take.to(torch.int64)
        occl = (alpha * pd[:, t, :] <= cand_d) & take[:, None]
        occl[:, :t + 1] = False
        alive &= ~occl
    # stable partition: chosen first
    key = (~chosen).to(torch.int64) * K + torch.arange(K, device=x.device)[None, :]
    return torch.argsort(key, dim=1)


def _cells(vectors: np.ndarray, cl: np.ndarray, nc: int, dev: torch.device):
    """Voronoi cells of the label means in data space: returns (cell of every point,
    cell means).  A point sits in the cell of its nearest mean, whatever its label."""
    x = torch.from_numpy(np.ascontiguousarray(vectors)).to(dev)
    means = torch.zeros((nc, vectors.shape[1]), dtype=torch.float64, device=dev)
    lab = torch.from_numpy(cl.astype(np.int64)).to(dev)
    cnt = torch.bincount(lab, minlength=nc).clamp_(min=1).to(torch.float64)
    step = 1 << 18
    for s in range(0, x.shape[0], step):
        means.index_add_(0, lab[s:s + step], x[s:s + step].to(torch.float64))
    means = (means / cnt[:, None]).to(torch.float32)
    mn = (means * means).sum(1)
    cell = torch.empty(x.shape[0], dtype=torch.int64, device=dev)
    for s in range(0, x.shape[0], step):
        xb = x[s:s + step].to(torch.float32)
        cell[s:s + step] = _sq_dists(xb, (xb * xb).sum(1), means, mn).argmin(1)
    return cell.cpu().numpy(), means.cpu().numpy()


def mixed_graph(w: Workload, vectors: np.ndarray, attrs: np.ndarray, types: np.ndarray,
                cl: np.ndarray, centres: np.ndarray, ss_graph, device: str | None = None) -> np.ndarray:
    """Degree-R fixture built from four kinds of edges:
      * r_knn  approximate nearest neighbours (exact among the points of the t_near nearest
               cells), thinned by occlusion pruning so that they spread in direction;
      * r_rev  reverse copies of those edges, so that no node is left without a way in;
      * r_attr nearest neighbours among the points whose attribute ranks all lie within a
               window around the node's own, at one or more window sizes -- the role the
               threshold passes of the paper's graph construction play;
      * r_long long edges to random points of cells at log-uniformly drawn centre ranks."""
    dev = _prep_device(device)
    rng = np.random.default_rng(ss_graph)
    n, R, nc = w.N, w.R, w.n_clusters
    r_long = min(w.r_long, R - 1)
    r_attr = min(w.r_attr, R - r_long - 1)
    r_rev = min(w.r_rev, R - r_long - r_attr - 1)
    r_knn = R - r_long - r_attr - r_rev
    cell, means = _cells(vectors, cl, nc, dev)
    order = np.argsort(cell, kind="stable")
    starts = np.searchsorted(cell[order], np.arange(nc + 1))
    cdist = ((means[:, None, :].astype(np.float64) - means[None, :, :]) ** 2).sum(-1)
    crank = np.argsort(cdist, axis=1, kind="stable")        # crank[c][0] == c
    t_near = min(w.t_near, nc)
    fracs = [f for f in w.attr_fracs if f > 0] if r_attr > 0 else []
    ranks01 = _rank_columns(attrs, types)
    ranks = torch.from_numpy(ranks01[order]).to(dev) if fracs else None

    graph = np.full((n, R), SENTINEL, dtype=np.uint32)
    xs = torch.from_numpy(np.ascontiguousarray(vectors[order].astype(np.float32))).to(dev)
    order_t = torch.from_numpy(order).to(dev)
    big = 3.0e38
    k_cand = max(r_knn, min(w.k_cand, 8 * r_knn))
    blk = 2048
    for c in range(nc):
        a, b = int(starts[c]), int(starts[c + 1])
        if a == b:
            continue
        cand = torch.from_numpy(np.concatenate(
            [np.arange(starts[t], starts[t + 1]) for t in crank[c, :t_near]])).to(dev)
        y = xs[cand]
        yn = (y * y).sum(1)
        for s0 in range(a, b, blk):
            s1 = min(b, s0 + blk)
            x = xs[s0:s1]
            d = _sq_dists(x, (x * x).sum(1), y, yn)
            # candidates begin with this cell's own rows: self is at column (row - a)
            rows_local = torch.arange(s0 - a, s1 - a, device=dev)
            d[torch.arange(s1 - s0, device=dev), rows_local] = big
            kk = min(k_cand, cand.shape[0] - 1)
            near = torch.topk(d, kk, dim=1, largest=False, sorted=True)
            if w.prune_alpha > 0 and kk > r_knn:
                perm = _diversify(x, y, near.indices, near.values, r_knn, w.prune_alpha)
                sel = torch.gather(near.indices, 1, perm[:, :r_knn])
            else:
                sel = near.indices[:, :r_knn]
            take = sel.shape[1]
            out_rows = order[s0:s1]
            graph[out_rows, :take] = order_t[cand[sel]].cpu().numpy().astype(np.uint32)
            if fracs:
                d.scatter_(1, sel, big)
                per = r_attr // len(fracs)
                col0 = r_knn + r_rev
                for fi, f in enumerate(fracs):
                    cnt = per if fi + 1 < len(fracs) else r_attr - per * (len(fracs) - 1)
                    half = 0.5 * f ** (1.0 / w.m)
                    dm = d.clone()
                    for j in range(w.m):
                        diff = (ranks[s0:s1, j][:, None] - ranks[cand, j][None, :]).abs_()
                        dm.masked_fill_(diff > half, big)
                    an = torch.topk(dm, cnt, dim=1, largest=False, sorted=True)
                    picked = order_t[cand[an.indices]]
                    picked = torch.where(an.values < 1.0e38, picked, torch.full_like(picked, -1))
                    pk = picked.cpu().numpy()
                    graph[out_rows, col0:col0 + cnt] = np.where(pk >= 0, pk, 0xFFFFFFFF).astype(np.uint32)
                    d.scatter_(1, an.indices, big)
                    col0 += cnt
    # reverse edges: v gets up to r_rev of the nodes that point at it, in a seeded random order
    if r_rev > 0:
        gk = torch.from_numpy(graph[:, :r_knn].astype(np.int64)).to(dev)
        src = torch.arange(n, dtype=torch.int64, device=dev).repeat_interleave(r_knn)
        dst = gk.reshape(-1)
        ok = dst != int(SENTINEL)
        src, dst = src[ok], dst[ok]
        shuffle = torch.from_numpy(rng.permutation(int(src.shape[0]))).to(dev)
        src, dst = src[shuffle], dst[shuffle]
        o = torch.argsort(dst, stable=True)
        src, dst = src[o], dst[o]
        first = torch.searchsorted(dst, torch.arange(n, dtype=torch.int64, device=dev))
        pos = torch.arange(dst.shape[0], dtype=torch.int64, device=dev) - first[dst]
        keep = pos < r_rev
        graph[dst[keep].cpu().numpy(), (r_knn + pos[keep]).cpu().numpy()] = src[keep].cpu().numpy().astype(np.uint32)
        del gk, src, dst, ok, shuffle, o, first, pos, keep
    # long edges: cell rank drawn log-uniformly in [1, nc); inside that cell the point whose
    # attributes are nearest to the node's own along a Z-order curve over the attribute
    # ranks (plus a small random offset), so that long hops tend to stay inside a range
    if r_long > 0 and nc > 1:
        u = rng.random((n, r_long))
        rank = np.minimum(np.floor(np.exp(u * math.log(nc))).astype(np.int64), nc - 1)
        rank = np.maximum(rank, 1)
        tgt_cell = crank[cell[:, None], rank]
        size = (starts[1:] - starts[:-1])[tgt_cell]
        if w.long_attr_aware:
            zc = _zorder(ranks01)
            key = torch.from_numpy(cell.astype(np.int64) * (1 << 32) + zc).to(dev)
            korder_t = torch.argsort(key, stable=True)      # grouped by cell, Z-ordered inside
            ksorted = key[korder_t]
            want = torch.from_numpy(tgt_cell.astype(np.int64) * (1 << 32) + zc[:, None]).to(dev)
            pos = torch.searchsorted(ksorted, want.reshape(-1)).reshape(n, r_long).cpu().numpy()
            korder = korder_t.cpu().numpy()
            del key, korder_t, ksorted, want
            pos = pos + rng.integers(-2, 3, size=(n, r_long))
            pos = np.clip(pos, starts[tgt_cell], np.maximum(starts[tgt_cell + 1] - 1, starts[tgt_cell]))
            tgt = korder[np.minimum(pos, n - 1)].astype(np.uint32)
        else:
            off = np.minimum((rng.random((n, r_long)) * size).astype(np.int64), np.maximum(size - 1, 0))
            tgt = order[np.minimum(starts[tgt_cell] + off, n - 1)].astype(np.uint32)
        tgt = np.where(size > 0, tgt, SENTINEL)
        graph[:, R - r_long:] = tgt
    return clean_rows(graph, str(dev))


def clean_rows(graph: np.ndarray, device: str = "cpu") -> np.ndarray:
    """Replace self references and repeated ids inside a row by the sentinel."""
    n, R = graph.shape
    dev = torch.device(device)
    g = torch.from_numpy(np.ascontiguousarray(graph).view(np.int32).copy()).to(dev)   # sentinel == -1
    g[g == torch.arange(n, dtype=torch.int32, device=dev)[:, None]] = -1
    for j in range(1, R):
        dup = (g[:, :j] == g[:, j:j + 1]).any(dim=1)
        g[dup, j] = -1
    return g.cpu().numpy().view(np.uint32)


# ----------------------------------------------------------------------------
# entry point
# ----------------------------------------------------------------------------
_CACHED = ("vectors", "queries", "attrs", "attr_types", "lo", "hi", "target_sel", "cluster", "graph")


def _cache_dir(w: Workload, seed: int, dev: torch.device, with_graph: bool) -> str | None:
    """Where the arrays of a large workload are kept between processes on one machine, or
    None.  Building the 10M-point graph takes minutes; a test run and a benchmark run on the
    same machine then build it once.  The key covers the whole description, the seed, the
    kind of device that found the neighbours and the source of this package, so a change of
    recipe never meets old arrays.  BOA_SYNTH_CACHE=0 switches it off, another value moves it."""
    where = os.environ.get("BOA_SYNTH_CACHE", "")
    if where == "0" or w.N < 500_000 or not with_graph:
        return None
    h = hashlib.sha256()
    h.update(repr(w).encode())
    h.update(f"|{seed}|{dev.type}|".encode())
    here = os.path.dirname(os.path.abspath(__file__))
    for name in ("generate.py", "configs.py"):
        with open(os.path.join(here, name), "rb") as f:
            h.update(f.read())
    root = where or os.path.join(tempfile.gettempdir(), "boa_synth_cache")
    return os.path.join(root, f"{w.name}_{h.hexdigest()[:16]}")


def _cache_load(path: str):
    try:
        if not os.path.exists(os.path.join(path, "done")):
            return None
        return {k: np.load(os.path.join(path, k + ".npy")) for k in _CACHED}
    except Exception:
        return None


def _cache_store(path: str, out: Dict[str, np.ndarray]) -> None:
    """Written under a name of this process's own and renamed into place in one step, so that
    several ranks building the same workload at once never read each other's half-written files."""
    tmp = f"{path}.tmp{os.getpid()}"
    try:
        os.makedirs(tmp, exist_ok=True)
        for k in _CACHED:
            np.save(os.path.join(tmp, k + ".npy"), out[k])
        with open(os.path.join(tmp, "done"), "w") as f:
            f.write("ok")
        os.rename(tmp, path)      # fails when another process got there first
    except Exception:
        pass                      # a full or read-only disk, or a lost race, only costs a build
    finally:
        if os.path.isdir(tmp):
            import shutil
            shutil.rmtree(tmp, ignore_errors=True)


def make_workload(w: Workload, seed: int = 0, device: str | None = None,
                  with_graph: bool = True) -> Dict[str, np.ndarray]:
    """Build every input array of workload `w` for `seed`."""
    cache = _cache_dir(w, seed, _prep_device(device), with_graph)
    if cache:
        hit = _cache_load(cache)
        if hit is not None:
            return hit
    out = _build_workload(w, seed, device, with_graph)
    if cache:
        _cache_store(cache, out)
    return out


def _build_workload(w: Workload, seed: int, device: str | None, with_graph: bool) -> Dict[str, np.ndarray]:
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
