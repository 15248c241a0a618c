"""Thin ctypes binding of include/boa.h.

Argument marshalling only: tensors are passed as device pointers, every step of
the search runs in the CUDA library.  There is no CPU fallback; if the shared
library is missing or no CUDA device is present, calls fail loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

PARAM = dict(eps=0, growth=1, tau=2, mode=3, plus_k=4, cap_mult=5, cap_add=6, table_kb=7,
             max_warps_per_sm=8, expand_w=9, table_tags=10, lam=11, pq=12, host_in_place=13, plus_min_sub=14, chains=15)
F32, U8 = 0, 1
NO_ID = 0xFFFFFFFF


class BoaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        lib = load_library()
        msg = lib.boa_strerror(status).decode()
        cuda = lib.boa_last_cuda_error()
        super().__init__(f"{what}: {msg} (status {status}, last CUDA error {cuda})")


def library_path() -> str:
    return os.path.join(HERE, "libboa.so")


def load_library():
    """Load libboa.so (built in-tree by build.py); raises if it is not there."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} is missing: build it with `python -m paper_2609_16175_b200.build` "
            "(there is no fallback implementation)")
    L = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
    L.boa_index_create.restype = i32
    L.boa_index_create.argtypes = [C.POINTER(vp), vp, i32, i64, i32, vp, C.POINTER(i32), i32, vp, i32,
                                   i64, vp]
    L.boa_index_share.restype = i32
    L.boa_index_share.argtypes = [C.POINTER(vp), vp]
    L.boa_index_destroy.restype = i32
    L.boa_index_destroy.argtypes = [vp]
    L.boa_index_entry.restype = i64
    L.boa_index_entry.argtypes = [vp]
    L.boa_search.restype = i32
    L.boa_search.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, vp, vp, vp]
    L.boa_search_noalloc.restype = i32
    L.boa_search_noalloc.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, vp, vp, vp]
    L.boa_search_host.restype = i32
    L.boa_search_host.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, vp, vp, vp]
    L.boa_set_param.restype = i32
    L.boa_set_param.argtypes = [vp, i32, C.c_double]
    L.boa_set_schedule.restype = i32
    L.boa_set_schedule.argtypes = [vp, C.POINTER(i32), i32]
    L.boa_get_stats.restype = i32
    L.boa_get_stats.argtypes = [vp, vp, vp, vp, vp, vp]
    L.boa_get_phase_counts.restype = i32
    L.boa_get_phase_counts.argtypes = [vp, C.POINTER(i64), i32, C.POINTER(i32), vp]
    L.boa_workspace_bytes.restype = i32
    L.boa_workspace_bytes.argtypes = [vp, i64, i32, C.POINTER(C.c_size_t)]
    L.boa_set_range_penalty.restype = i32
    L.boa_set_range_penalty.argtypes = [vp, C.POINTER(C.c_float), vp]
    L.boa_index_set_metric.restype = i32
    L.boa_index_set_metric.argtypes = [vp, i32, vp]
    L.boa_index_attach_pq.restype = i32
    L.boa_index_attach_pq.argtypes = [vp, vp, vp, i32, i32, vp]
    L.boa_get_rerank_counts.restype = i32
    L.boa_get_rerank_counts.argtypes = [vp, vp, vp]
    L.boa_last_launch_count.restype = i32
    L.boa_last_launch_count.argtypes = [vp]
    L.boa_device_status.restype = i32
    L.boa_device_status.argtypes = [vp, C.POINTER(i32), vp]
    L.boa_graph_build.restype = i32
    L.boa_graph_build.argtypes = [vp, i32, i64, i32, vp, i32, i32, i32, C.c_float, C.POINTER(C.c_float), i32, i32,
                                  i32, i32, i64, vp, C.POINTER(i64), vp]
    L.boa_last_cuda_error.restype = i32
    L.boa_strerror.restype = C.c_char_p
    L.boa_strerror.argtypes = [i32]
    _LIB = L
    return L


def _check(status: int, what: str):
    if status != 0:
        raise BoaError(status, what)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return t.contiguous()


def build_graph(vectors: torch.Tensor, attr_pos: torch.Tensor, R: int, Lb: int, alpha: float = 1.2,
                thresholds: Sequence = (float("inf"),), B: int = 1024, passes: int = 1, cap_in: int = 64,
                entry: int = -1, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """boa_graph_build: returns the [N][R] graph (int32 storage of node ids) on the vectors' device.
    Every entry of `thresholds` is one number (the same threshold in every attribute) or a
    sequence of one number per attribute."""
    lib = load_library()
    vectors = _dev(vectors, "vectors")
    attr_pos = _dev(attr_pos, "attr_pos")
    if attr_pos.dtype != torch.float32 or attr_pos.dim() != 2:
        raise ValueError("attr_pos must be float32 [N][m]")
    dt = F32 if vectors.dtype == torch.float32 else U8
    N, D = vectors.shape
    out = torch.empty((N, R), dtype=torch.int32, device=vectors.device)
    m_pos = attr_pos.shape[1]
    flat = []
    for t in thresholds:
        row = [float(x) for x in t] if hasattr(t, "__len__") else [float(t)] * m_pos
        if len(row) != m_pos:
            raise ValueError("a threshold needs one value per attribute")
        flat += row
    th = (C.c_float * len(flat))(*flat)
    nb = C.c_int64(0)
    _check(lib.boa_graph_build(vectors.data_ptr(), dt, N, D, attr_pos.data_ptr(), attr_pos.shape[1], R, Lb,
                               float(alpha), th, len(thresholds), B, passes, cap_in, int(entry), out.data_ptr(),
                               C.byref(nb), _stream_ptr(stream)), "boa_graph_build")
    return out


class BoaIndex:
    """boa_index_create / boa_search / ... with torch tensors as the device buffers."""

    def __init__(self, vectors: torch.Tensor, attrs: torch.Tensor, attr_types: Sequence[int],
                 graph: torch.Tensor, entry: int = -1, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("BoaIndex needs a CUDA device; there is no CPU path")
        self._lib = load_library()
        vectors = _dev(vectors, "vectors")
        attrs = _dev(attrs, "attrs")
        graph = _dev(graph, "graph")
        if vectors.dtype == torch.float32:
            dt = F32
        elif vectors.dtype == torch.uint8:
            dt = U8
        else:
            raise ValueError("vectors must be float32 or uint8")
        if attrs.dtype not in (torch.int32, torch.float32):
            raise ValueError("attrs must hold 4-byte cells (int32 storage)")
        if graph.dtype not in (torch.int32, torch.uint32):
            raise ValueError("graph must be int32/uint32 storage of node ids")
        self.N, self.D = vectors.shape
        self.m = attrs.shape[1]
        self.R = graph.shape[1]
        types = (C.c_int * self.m)(*[int(t) for t in attr_types])
        h = C.c_void_p()
        _check(self._lib.boa_index_create(C.byref(h), vectors.data_ptr(), dt, self.N, self.D,
                                          attrs.data_ptr(), types, self.m, graph.data_ptr(), self.R,
                                          int(entry), _stream_ptr(stream)), "boa_index_create")
        self._h = h
        self.device = vectors.device

    def share(self) -> "BoaIndex":
        """boa_index_share: another handle on the same index data with scratch of its own, for a
        search that runs at the same time as this handle's (on another stream).  This object must
        stay open while the shared one is in use."""
        other = object.__new__(BoaIndex)
        other._lib = self._lib
        other.N, other.D, other.m, other.R, other.device = self.N, self.D, self.m, self.R, self.device
        other._owner = self                       # keeps the data alive
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self._lib.boa_index_share(C.byref(h), self._h), "boa_index_share")
        other._h = h
        return other

    def close(self):
        if getattr(self, "_h", None):
            self._lib.boa_index_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def entry(self) -> int:
        return int(self._lib.boa_index_entry(self._h))

    def set_range_penalty(self, scales: Optional[Sequence[float]], stream: Optional[torch.cuda.Stream] = None):
        """boa_set_range_penalty: per-attribute scales (None: back to the violation count)."""
        arr = None if scales is None else (C.c_float * self.m)(*[float(x) for x in scales])
        _check(self._lib.boa_set_range_penalty(self._h, arr, _stream_ptr(stream)), "boa_set_range_penalty")

    def set_metric(self, metric: str, stream: Optional[torch.cuda.Stream] = None):
        """boa_index_set_metric: 'l2' (default) or 'cosine' (float vectors, one way)."""
        _check(self._lib.boa_index_set_metric(self._h, {"l2": 0, "cosine": 1}[metric], _stream_ptr(stream)),
               "boa_index_set_metric")

    def attach_pq(self, pivots: torch.Tensor, codes: torch.Tensor,
                  stream: Optional[torch.cuda.Stream] = None):
        """boa_index_attach_pq: pivots [M][K][D/M] float32, codes [N][M] uint8 (device tensors)."""
        pivots = _dev(pivots, "pivots")
        codes = _dev(codes, "codes")
        if pivots.dtype != torch.float32 or codes.dtype != torch.uint8 or pivots.dim() != 3:
            raise ValueError("pivots must be float32 [M][K][D/M], codes uint8 [N][M]")
        M, K = int(pivots.shape[0]), int(pivots.shape[1])
        if tuple(codes.shape) != (self.N, M) or int(pivots.shape[2]) * M != self.D:
            raise ValueError("codebook shape does not match the index")
        _check(self._lib.boa_index_attach_pq(self._h, pivots.data_ptr(), codes.data_ptr(), M, K,
                                             _stream_ptr(stream)), "boa_index_attach_pq")

    def rerank_counts(self, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        out = torch.zeros(getattr(self, "_last_Q", 0), dtype=torch.int32, device=self.device)
        _check(self._lib.boa_get_rerank_counts(self._h, out.data_ptr(), _stream_ptr(stream)),
               "boa_get_rerank_counts")
        return out

    def set_param(self, name: str, value: float):
        _check(self._lib.boa_set_param(self._h, PARAM[name], float(value)), f"boa_set_param({name})")

    def set_schedule(self, widths: Sequence[int]):
        arr = (C.c_int * max(1, len(widths)))(*[int(w) for w in widths])
        _check(self._lib.boa_set_schedule(self._h, arr, len(widths)), "boa_set_schedule")

    def search(self, queries: torch.Tensor, lo: torch.Tensor, hi: torch.Tensor, k: int, L0: int,
               Lmax: int, out_ids: Optional[torch.Tensor] = None,
               out_dists: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
        queries = _dev(queries, "queries")
        lo = _dev(lo, "lo")
        hi = _dev(hi, "hi")
        Q = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty((Q, k), dtype=torch.int32, device=queries.device)
        if out_dists is None:
            out_dists = torch.empty((Q, k), dtype=torch.float32, device=queries.device)
        _check(self._lib.boa_search(self._h, queries.data_ptr(), Q, lo.data_ptr(), hi.data_ptr(), k,
                                    L0, Lmax, out_ids.data_ptr(), out_dists.data_ptr(),
                                    _stream_ptr(stream)), "boa_search")
        self._last_Q = Q
        return out_ids, out_dists

    def search_host(self, queries: torch.Tensor, lo: torch.Tensor, hi: torch.Tensor, k: int, L0: int,
                    Lmax: int, out_ids: Optional[torch.Tensor] = None,
                    out_dists: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
        """boa_search_host: HOST tensors in (pinned for full copy speed), HOST tensors out; the
        library does the transfers and returns when the results are readable."""
        for name, t in (("queries", queries), ("lo", lo), ("hi", hi)):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError(f"{name} must be a contiguous CPU tensor")
        Q = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty((Q, k), dtype=torch.int32)
        if out_dists is None:
            out_dists = torch.empty((Q, k), dtype=torch.float32)
        for name, t in (("out_ids", out_ids), ("out_dists", out_dists)):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError(f"{name} must be a contiguous CPU tensor")
        with torch.cuda.device(self.device):
            _check(self._lib.boa_search_host(self._h, queries.data_ptr(), Q, lo.data_ptr(), hi.data_ptr(), k,
                                             L0, Lmax, out_ids.data_ptr(), out_dists.data_ptr(),
                                             _stream_ptr(stream)), "boa_search_host")
        self._last_Q = Q
        return out_ids, out_dists

    def search_noalloc(self, queries: torch.Tensor, lo: torch.Tensor, hi: torch.Tensor, k: int,
                       L0: int, Lmax: int, out_ids: torch.Tensor, out_dists: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None):
        """boa_search_noalloc: for callers that may not allocate device memory.  The caller
        passes every buffer, outputs included; the library's scratch is a fixed array in its
        own image (batches up to 1024 queries, widths up to 512).  Calls that overlap on the
        GPU race on that array, so keep them ordered."""
        for name, t in (("queries", queries), ("lo", lo), ("hi", hi), ("out_ids", out_ids),
                        ("out_dists", out_dists)):
            if not (t.is_cuda and t.is_contiguous()):
                raise ValueError(f"{name} must be a contiguous CUDA tensor")
        _check(self._lib.boa_search_noalloc(self._h, queries.data_ptr(), queries.shape[0],
                                            lo.data_ptr(), hi.data_ptr(), k, L0, Lmax,
                                            out_ids.data_ptr(), out_dists.data_ptr(),
                                            _stream_ptr(stream)), "boa_search_noalloc")
        return out_ids, out_dists

    def stats(self, stream: Optional[torch.cuda.Stream] = None):
        Q = getattr(self, "_last_Q", 0)
        out = [torch.zeros(Q, dtype=torch.int32, device=self.device) for _ in range(4)]
        _check(self._lib.boa_get_stats(self._h, *[t.data_ptr() for t in out], _stream_ptr(stream)),
               "boa_get_stats")
        return dict(final_L=out[0], n_expand=out[1], n_scored=out[2], flags=out[3])

    def phase_counts(self, stream: Optional[torch.cuda.Stream] = None):
        buf = (C.c_int64 * 8)()
        n = C.c_int(0)
        _check(self._lib.boa_get_phase_counts(self._h, buf, 8, C.byref(n), _stream_ptr(stream)),
               "boa_get_phase_counts")
        return [int(buf[i]) for i in range(n.value)]

    def workspace_bytes(self, Q: int, Lmax: int) -> int:
        b = C.c_size_t(0)
        _check(self._lib.boa_workspace_bytes(self._h, Q, Lmax, C.byref(b)), "boa_workspace_bytes")
        return int(b.value)

    def device_status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        v = C.c_int(0)
        _check(self._lib.boa_device_status(self._h, C.byref(v), _stream_ptr(stream)), "boa_device_status")
        return int(v.value)

    @property
    def last_launch_count(self) -> int:
        return int(self._lib.boa_last_launch_count(self._h))
