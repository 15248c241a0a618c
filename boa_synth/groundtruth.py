"""Exact range-filtered top-k by blocked brute force with torch -- a harness tool that
scores recall for large batches.  It is not part of the search path; tests compare
it with the CPU oracle's own brute force on sampled queries."""
from __future__ import annotations

import numpy as np
import torch

from .generate import ATTR_F32


def filtered_topk(vectors: torch.Tensor, attrs: torch.Tensor, attr_types, queries: torch.Tensor,
                  lo: torch.Tensor, hi: torch.Tensor, k: int, block: int = 256):
    """Returns (ids [Q,k] int64 with -1 padding, d2 [Q,k] float64-accurate for integer data
    / float32 otherwise, n_valid [Q]) on the device of `vectors`."""
    dev = vectors.device
    x = vectors.to(torch.float32)
    xn = (x.double() ** 2).sum(1)
    n, Q = x.shape[0], queries.shape[0]
    ids = torch.full((Q, k), -1, dtype=torch.int64, device=dev)
    d2 = torch.full((Q, k), float("inf"), dtype=torch.float64, device=dev)
    nvalid = torch.zeros(Q, dtype=torch.int64, device=dev)
    if str(dev).startswith("cuda"):
        torch.backends.cuda.matmul.allow_tf32 = False
    for s in range(0, Q, block):
        e = min(Q, s + block)
        q = queries[s:e].to(torch.float32)
        ok = torch.ones((e - s, n), dtype=torch.bool, device=dev)
        for j, t in enumerate(attr_types):
            col = attrs[:, j]
            l, h = lo[s:e, j], hi[s:e, j]
            if int(t) == ATTR_F32:
                col, l, h = col.view(torch.float32), l.view(torch.float32), h.view(torch.float32)
            ok &= (col[None, :] >= l[:, None]) & (col[None, :] <= h[:, None])
        d = (xn[None, :] + (q.double() ** 2).sum(1)[:, None]).to(torch.float64)
        d -= 2.0 * torch.mm(q, x.t()).double()
        d.masked_fill_(~ok, float("inf"))
        # the expansion |x|^2 + |q|^2 - 2xq in fp32 loses digits on small distances: take a
        # few candidates more than k, recompute their distances directly in double, re-rank
        kk = min(k, n)
        kc = min(k + 16, n)
        cand = torch.topk(d, kc, dim=1, largest=False, sorted=True)
        fin = torch.isfinite(cand.values)
        diff = x[cand.indices].double() - q.double()[:, None, :]
        exact = (diff * diff).sum(-1)
        exact.masked_fill_(~fin, float("inf"))
        # order by (distance, id)
        order = torch.argsort(cand.indices, dim=1, stable=True)
        exact_o = torch.gather(exact, 1, order)
        idx_o = torch.gather(cand.indices, 1, order)
        order2 = torch.argsort(exact_o, dim=1, stable=True)
        exact_s = torch.gather(exact_o, 1, order2)[:, :kk]
        idx_s = torch.gather(idx_o, 1, order2)[:, :kk]
        fin_s = torch.isfinite(exact_s)
        ids[s:e, :kk] = torch.where(fin_s, idx_s, torch.full_like(idx_s, -1))
        d2[s:e, :kk] = exact_s
        nvalid[s:e] = ok.sum(1)
    return ids, d2, nvalid


def recall_against(ids_found: np.ndarray, d2_found: np.ndarray, gt_d2: np.ndarray, gt_nvalid: np.ndarray,
                   k: int, rel: float = 1e-6):
    """Per-query tie-aware recall: a returned point counts when its squared distance does
    not exceed the exact k-th one.  Queries with an empty valid set get NaN."""
    Q = ids_found.shape[0]
    den = np.minimum(k, gt_nvalid).astype(np.float64)
    kth = gt_d2[np.arange(Q), np.maximum(den.astype(np.int64) - 1, 0)]
    ok = (ids_found != 0xFFFFFFFF) & (d2_found.astype(np.float64) <= kth[:, None] * (1.0 + rel) + 1e-30)
    hit = np.minimum(ok.sum(1), den)
    with np.errstate(invalid="ignore", divide="ignore"):
        r = hit / den
    r[den == 0] = np.nan
    return r
