"""ctypes front end of the plain-C oracle (oracle/boa_oracle.c).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's CPU
baseline may import this.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, dbl = C.c_void_p, C.c_int, C.c_int64, C.c_double
        L.orc_create.restype = vp
        L.orc_create.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, i32, i64]
        L.orc_destroy.argtypes = [vp]
        L.orc_entry.restype = i64
        L.orc_entry.argtypes = [vp]
        L.orc_medoid.restype = i64
        L.orc_medoid.argtypes = [vp]
        L.orc_dist2_f64.restype = dbl
        L.orc_dist2_f64.argtypes = [vp, vp, i64]
        L.orc_dist2_lanes.restype = C.c_float
        L.orc_dist2_lanes.argtypes = [vp, vp, i64]
        L.orc_phi.restype = i32
        L.orc_phi.argtypes = [vp, vp, vp, i64]
        L.orc_bruteforce.restype = i64
        L.orc_bruteforce.argtypes = [vp, vp, vp, vp, i32, vp, vp]
        L.orc_state_new.restype = vp
        L.orc_state_new.argtypes = [vp, i32]
        L.orc_state_free.argtypes = [vp]
        L.orc_state_set_lambda.argtypes = [vp, C.c_float]
        L.orc_beam_init.argtypes = [vp, i32, vp, vp, vp, i32]
        L.orc_beam_run_w.argtypes = [vp, i32, vp, vp, vp, i32, i64, i32]
        L.orc_beam_result.restype = i32
        L.orc_beam_result.argtypes = [vp, i32, vp, vp]
        L.orc_state_size.restype = i32
        L.orc_state_size.argtypes = [vp]
        L.orc_state_expanded.restype = i64
        L.orc_state_expanded.argtypes = [vp]
        L.orc_state_scored.restype = i64
        L.orc_state_scored.argtypes = [vp]
        L.orc_state_hit_cap.restype = i32
        L.orc_state_hit_cap.argtypes = [vp]
        L.orc_state_pool.argtypes = [vp, vp, vp, vp, vp]
        L.orc_uncertain.restype = i32
        L.orc_uncertain.argtypes = [vp, i32, i32, dbl]
        L.orc_boa_search_wl.argtypes = [vp, vp, i64, vp, vp, i32, vp, i32, dbl, dbl, i32, i32,
                                        i32, i32, i32, C.c_float, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.orc_prune.restype = i32
        L.orc_prune.argtypes = [vp, vp, i32, i64, vp, i32, i32, C.c_float, vp, i32, vp]
        L.orc_build_graph.restype = i64
        L.orc_build_graph.argtypes = [vp, vp, i32, vp, i32, i32, C.c_float, vp, i32, i32, i32, i32]
        L.orc_range_penalty.restype = C.c_float
        L.orc_range_penalty.argtypes = [vp, vp, vp, i64, vp]
        L.orc_state_set_penalty.argtypes = [vp, vp]
        L.orc_set_metric.argtypes = [vp, i32]
        L.orc_cos_dist.restype = C.c_float
        L.orc_cos_dist.argtypes = [vp, vp, i64, i32]
        L.orc_unit_f32.argtypes = [vp, i32, vp]
        L.orc_pq_attach.argtypes = [vp, vp, vp, i32, i32]
        L.orc_pq_table.argtypes = [vp, vp, i32, vp]
        L.orc_pq_dist.restype = C.c_float
        L.orc_pq_dist.argtypes = [vp, vp, i32, i64]
        L.orc_state_use_pq.argtypes = [vp, i32, vp, i32]
        L.orc_beam_rerank.restype = i32
        L.orc_beam_rerank.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp, vp]
        L.orc_uncertain_reranked.restype = i32
        L.orc_uncertain_reranked.argtypes = [i32, i32, C.c_float, C.c_float, dbl]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


DEFAULT_CAP = (8, 64)      # a phase at width L stops after 8*L + 64 expansions


def default_widths(L0: int, Lmax: int, growth: int = 4):
    """Geometric schedule L0, growth*L0, ... clamped to Lmax (last phase == Lmax)."""
    w = [int(L0)]
    while w[-1] < Lmax:
        w.append(min(int(Lmax), w[-1] * growth))
    return w


class OracleIndex:
    """Holds the input arrays (no copies of the big ones) and the entry point."""

    def __init__(self, vectors, attrs, attr_types, graph, entry: int = -1):
        self.vectors = np.ascontiguousarray(vectors)
        assert self.vectors.dtype in (np.float32, np.uint8)
        self.vec_dtype = 0 if self.vectors.dtype == np.float32 else 1
        self.attrs = np.ascontiguousarray(attrs, dtype=np.int32)
        self.attr_types = np.ascontiguousarray(attr_types, dtype=np.int32)
        self.graph = np.ascontiguousarray(graph, dtype=np.uint32)
        self.N, self.D = self.vectors.shape
        self.m = self.attrs.shape[1]
        self.R = self.graph.shape[1]
        self.h = lib().orc_create(_p(self.vectors), self.vec_dtype, self.N, self.D, _p(self.attrs),
                                  _p(self.attr_types), self.m, _p(self.graph), self.R, int(entry))
        self.entry = int(lib().orc_entry(self.h))

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_destroy(self.h)
            self.h = None

    # --- elementary pieces -------------------------------------------------
    def dist2_f64(self, q, p):
        q = np.ascontiguousarray(q, dtype=np.float32)
        return float(lib().orc_dist2_f64(self.h, _p(q), int(p)))

    def dist2_lanes(self, q, p):
        q = np.ascontiguousarray(q, dtype=np.float32)
        return np.float32(lib().orc_dist2_lanes(self.h, _p(q), int(p)))

    def phi(self, lo, hi, p):
        lo = np.ascontiguousarray(lo, dtype=np.int32)
        hi = np.ascontiguousarray(hi, dtype=np.int32)
        return int(lib().orc_phi(self.h, _p(lo), _p(hi), int(p)))

    # --- graph construction -------------------------------------------------------
    @staticmethod
    def _threshold_rows(thresholds, m):
        """[T][m] float32: a scalar threshold applies to every attribute."""
        rows = [[float(t)] * m if np.isscalar(t) else [float(x) for x in t] for t in thresholds]
        assert all(len(r) == m for r in rows)
        return np.ascontiguousarray(rows, dtype=np.float32)

    def prune(self, pos, p, ids, R, alpha=1.2, thresholds=(float("inf"),)):
        pos = np.ascontiguousarray(pos, dtype=np.float32)
        ids = np.ascontiguousarray(ids, dtype=np.uint32)
        th = self._threshold_rows(thresholds, pos.shape[1])
        row = np.empty(R, dtype=np.uint32)
        n = lib().orc_prune(self.h, _p(pos), pos.shape[1], int(p), _p(ids), len(ids), int(R), float(alpha),
                            _p(th), len(th), _p(row))
        return row, n

    def build_graph(self, pos, R, Lb, alpha=1.2, thresholds=(float("inf"),), B=1024, passes=1, cap_in=64):
        """Builds the graph into a new array, which becomes this index's graph."""
        pos = np.ascontiguousarray(pos, dtype=np.float32)
        th = self._threshold_rows(thresholds, pos.shape[1])
        g = np.empty((self.N, R), dtype=np.uint32)
        self._build_pos, self._build_th = pos, th
        lib().orc_build_graph(self.h, _p(pos), pos.shape[1], _p(g), int(R), int(Lb), float(alpha), _p(th),
                              len(th), int(B), int(passes), int(cap_in))
        self.graph, self.R = g, R
        return g

    def range_penalty(self, lo, hi, p, scales):
        lo = np.ascontiguousarray(lo, dtype=np.int32)
        hi = np.ascontiguousarray(hi, dtype=np.int32)
        scales = np.ascontiguousarray(scales, dtype=np.float32)
        return np.float32(lib().orc_range_penalty(self.h, _p(lo), _p(hi), int(p), _p(scales)))

    def medoid(self):
        return int(lib().orc_medoid(self.h))

    # --- metric ----------------------------------------------------------------
    def set_metric(self, metric: str):
        """'l2' (default) or 'cosine' (float vectors; call once, right after construction)."""
        assert metric in ("l2", "cosine") and (metric == "l2" or self.vec_dtype == 0)
        lib().orc_set_metric(self.h, 1 if metric == "cosine" else 0)

    def cos_dist(self, q, p, dist_mode=0):
        q = np.ascontiguousarray(q, dtype=np.float32)
        return np.float32(lib().orc_cos_dist(self.h, _p(q), int(p), int(dist_mode)))

    # --- product quantisation ------------------------------------------------
    def attach_pq(self, pivots, codes):
        """pivots [M][K][D/M] float32, codes [N][M] uint8 (the arrays are kept, not copied)."""
        self.pq_pivots = np.ascontiguousarray(pivots, dtype=np.float32)
        self.pq_codes = np.ascontiguousarray(codes, dtype=np.uint8)
        M, K, dsub = self.pq_pivots.shape
        assert M * dsub == self.D and self.pq_codes.shape == (self.N, M) and K <= 256
        self.pq_M, self.pq_K = M, K
        lib().orc_pq_attach(self.h, _p(self.pq_pivots), _p(self.pq_codes), M, K)

    def pq_table(self, q, dist_mode=0):
        q = np.ascontiguousarray(q, dtype=np.float32)
        t = np.empty((self.pq_M, self.pq_K), dtype=np.float32)
        lib().orc_pq_table(self.h, _p(q), int(dist_mode), _p(t))
        return t

    def pq_dist(self, table, p, dist_mode=0):
        table = np.ascontiguousarray(table, dtype=np.float32)
        return np.float32(lib().orc_pq_dist(self.h, _p(table), int(dist_mode), int(p)))

    # --- exact filtered top-k ------------------------------------------------
    def bruteforce(self, queries, lo, hi, k):
        queries = np.ascontiguousarray(queries, dtype=np.float32)
        lo = np.ascontiguousarray(lo, dtype=np.int32)
        hi = np.ascontiguousarray(hi, dtype=np.int32)
        Q = queries.shape[0]
        ids = np.empty((Q, k), dtype=np.uint32)
        d2 = np.empty((Q, k), dtype=np.float64)
        nvalid = np.empty(Q, dtype=np.int64)
        for i in range(Q):
            nvalid[i] = lib().orc_bruteforce(self.h, _p(queries[i]), _p(lo[i]), _p(hi[i]), k,
                                             _p(ids[i]), _p(d2[i]))
        return ids, d2, nvalid

    # --- one beam search, step-wise ------------------------------------------
    def beam(self, q, lo, hi, L, C=None, dist_mode=0, max_expand=1 << 40, expand_w=1,
             lam=float("inf"), pq=False, penalty_scales=None):
        return OracleBeam(self, q, lo, hi, L, C if C is not None else L, dist_mode, max_expand,
                          expand_w, lam, pq, penalty_scales)

    # --- the multi-phase batch driver ----------------------------------------
    def search(self, queries, lo, hi, k, widths, eps=0.05, tau=0.0, mode="restart",
               dist_mode=0, cap=DEFAULT_CAP, expand_w=1, lam=float("inf"), pq=False, penalty_scales=None):
        queries = np.ascontiguousarray(queries, dtype=np.float32)
        ps = None if penalty_scales is None else np.ascontiguousarray(penalty_scales, dtype=np.float32)
        lo = np.ascontiguousarray(lo, dtype=np.int32)
        hi = np.ascontiguousarray(hi, dtype=np.int32)
        Q = queries.shape[0]
        w = np.ascontiguousarray(widths, dtype=np.int32)
        ids = np.empty((Q, k), dtype=np.uint32)
        d2 = np.empty((Q, k), dtype=np.float32)
        final_L = np.empty(Q, dtype=np.int32)
        n_expand = np.empty(Q, dtype=np.int32)
        n_scored = np.empty(Q, dtype=np.int32)
        flags = np.empty(Q, dtype=np.int32)
        phase_active = np.zeros(len(w), dtype=np.int64)
        lib().orc_boa_search_wl(self.h, _p(queries), Q, _p(lo), _p(hi), k, _p(w), len(w),
                               float(eps), float(tau), 1 if mode == "resume" else 0, int(dist_mode),
                               int(cap[0]), int(cap[1]), int(expand_w), float(lam), 1 if pq else 0,
                               None if ps is None else _p(ps), _p(ids), _p(d2), _p(final_L),
                               _p(n_expand), _p(n_scored), _p(flags), _p(phase_active))
        return dict(ids=ids, d2=d2, final_L=final_L, n_expand=n_expand, n_scored=n_scored,
                    flags=flags, phase_active=phase_active)


class OracleBeam:
    """One query's Algorithm-2 state, for tests that look inside a search."""

    def __init__(self, index, q, lo, hi, L, C, dist_mode, max_expand, expand_w=1, lam=float("inf"),
                 pq=False, penalty_scales=None):
        self.ix = index
        self.pq = bool(pq)
        self.pen = None if penalty_scales is None else np.ascontiguousarray(penalty_scales, dtype=np.float32)
        self.expand_w = int(expand_w)
        self.q = np.ascontiguousarray(q, dtype=np.float32)
        self.lo = np.ascontiguousarray(lo, dtype=np.int32)
        self.hi = np.ascontiguousarray(hi, dtype=np.int32)
        self.dist_mode = dist_mode
        self.st = lib().orc_state_new(index.h, int(C))
        lib().orc_state_set_lambda(self.st, float(lam))
        if self.pen is not None:
            lib().orc_state_set_penalty(self.st, _p(self.pen))
        if self.pq:
            lib().orc_state_use_pq(self.st, 1, _p(self.q), dist_mode)
        lib().orc_beam_init(self.st, int(C), _p(self.q), _p(self.lo), _p(self.hi), dist_mode)
        self.run(L, max_expand)

    def run(self, L, max_expand=1 << 40):
        self.L = int(L)
        lib().orc_beam_run_w(self.st, int(L), _p(self.q), _p(self.lo), _p(self.hi), self.dist_mode,
                             int(max_expand), self.expand_w)
        return self

    def result(self, k):
        ids = np.empty(k, dtype=np.uint32)
        d2 = np.empty(k, dtype=np.float32)
        n = lib().orc_beam_result(self.st, k, _p(ids), _p(d2))
        return ids, d2, n

    def rerank(self, k, L=None):
        """End of a PQ search: (ids, exact d2, |V|, d2_k, d2_max) over the valid beam entries."""
        ids = np.empty(k, dtype=np.uint32)
        d2 = np.empty(k, dtype=np.float32)
        dk, dm = C.c_float(0), C.c_float(0)
        nv = lib().orc_beam_rerank(self.st, int(self.L if L is None else L), int(k), _p(self.q),
                                   self.dist_mode, _p(ids), _p(d2), C.byref(dk), C.byref(dm))
        return ids, d2, nv, np.float32(dk.value), np.float32(dm.value)

    def pool(self):
        n = lib().orc_state_size(self.st)
        ids = np.empty(n, dtype=np.uint32)
        d2 = np.empty(n, dtype=np.float32)
        phi = np.empty(n, dtype=np.int32)
        ex = np.empty(n, dtype=np.int32)
        lib().orc_state_pool(self.st, _p(ids), _p(d2), _p(phi), _p(ex))
        return ids, d2, phi, ex

    def uncertain(self, k, eps=0.05, L=None):
        return bool(lib().orc_uncertain(self.st, int(self.L if L is None else L), int(k), float(eps)))

    @property
    def n_expand(self):
        return int(lib().orc_state_expanded(self.st))

    @property
    def n_scored(self):
        return int(lib().orc_state_scored(self.st))

    @property
    def hit_cap(self):
        return bool(lib().orc_state_hit_cap(self.st))

    def __del__(self):
        if getattr(self, "st", None):
            lib().orc_state_free(self.st)
            self.st = None
