"""Product-quantisation codebooks for the synthetic workloads: a fixture, like the graph.

The search library and the oracle both take the codebook (centroids per subspace) and the
codes (nearest centroid of every point in every subspace) as inputs; this module trains
them with a few seeded Lloyd iterations per subspace.  It holds no part of the search.
"""
from __future__ import annotations

import numpy as np
import torch


def _assign(x: torch.Tensor, cent: torch.Tensor, block: int = 1 << 16) -> torch.Tensor:
    """Index of the nearest centroid (squared L2, lower index on ties) for every row of x."""
    cn = (cent * cent).sum(1)
    out = torch.empty(x.shape[0], dtype=torch.int64, device=x.device)
    for s in range(0, x.shape[0], block):
        xb = x[s:s + block]
        d = cn[None, :] - 2.0 * (xb @ cent.t())
        out[s:s + block] = d.argmin(1)
    return out


def train_pq(vectors: np.ndarray, M: int, K: int = 256, iters: int = 8, seed: int = 0,
             sample: int = 1 << 16, device: str | None = None):
    """Returns (pivots [M][K][D/M] float32, codes [N][M] uint8).

    Subspace m covers dimensions [m*D/M, (m+1)*D/M).  Centroids start from a seeded random
    sample of the points and are refined by `iters` Lloyd iterations on a seeded sample; a
    centroid that loses all its points keeps its place.  Every point is then encoded by its
    nearest centroid."""
    if device is None:
        device = "cuda" if torch.cuda.is_available() else "cpu"
    if str(device).startswith("cuda"):
        torch.backends.cuda.matmul.allow_tf32 = False
    dev = torch.device(device)
    N, D = vectors.shape
    assert D % M == 0 and 1 <= K <= 256
    dsub = D // M
    rng = np.random.default_rng(np.random.SeedSequence([seed, 0x5051]))
    pick = rng.choice(N, size=min(sample, N), replace=False)
    xs = torch.from_numpy(np.ascontiguousarray(vectors[np.sort(pick)]).astype(np.float32)).to(dev)
    pivots = np.empty((M, K, dsub), dtype=np.float32)
    codes = np.empty((N, M), dtype=np.uint8)
    step = 1 << 20
    for m in range(M):
        sub = xs[:, m * dsub:(m + 1) * dsub].contiguous()
        first = rng.choice(sub.shape[0], size=K, replace=sub.shape[0] < K)
        cent = sub[torch.from_numpy(first).to(dev)].clone()
        for _ in range(iters):
            a = _assign(sub, cent)
            tot = torch.zeros_like(cent).index_add_(0, a, sub)
            cnt = torch.bincount(a, minlength=K).to(torch.float32)
            keep = cnt > 0
            cent[keep] = tot[keep] / cnt[keep, None]
        pivots[m] = cent.cpu().numpy()
        for s in range(0, N, step):
            xb = torch.from_numpy(np.ascontiguousarray(vectors[s:s + step, m * dsub:(m + 1) * dsub])
                                  .astype(np.float32)).to(dev)
            codes[s:s + step, m] = _assign(xb, cent).cpu().numpy().astype(np.uint8)
    return pivots, codes
