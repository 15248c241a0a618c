"""Evaluation arithmetic of the benchmark harness: recall@k, average beamwidth,
per-phase split.  These describe how results are scored, not how they are found."""
from __future__ import annotations

import numpy as np

SENTINEL = 0xFFFFFFFF


def recall_plain(ids: np.ndarray, gt_ids: np.ndarray, gt_nvalid: np.ndarray, k: int) -> float:
    """Mean of |returned ∩ exact| / min(k, |valid set|) over queries with a non-empty valid set."""
    tot, cnt = 0.0, 0
    for i in range(ids.shape[0]):
        den = min(k, int(gt_nvalid[i]))
        if den == 0:
            continue
        g = set(int(x) for x in gt_ids[i][:den])
        tot += len(g & set(int(x) for x in ids[i] if int(x) != SENTINEL)) / den
        cnt += 1
    return tot / max(cnt, 1)


def recall_tie_aware(ids: np.ndarray, d2: np.ndarray, gt_d2: np.ndarray, gt_nvalid: np.ndarray,
                     k: int, rel: float = 0.0) -> float:
    """As recall_plain, but a returned (valid) point also counts when its squared
    distance does not exceed the exact k-th one: at ties several answers are exact."""
    tot, cnt = 0.0, 0
    for i in range(ids.shape[0]):
        den = min(k, int(gt_nvalid[i]))
        if den == 0:
            continue
        kth = float(gt_d2[i][den - 1])
        ok = (ids[i] != SENTINEL) & (d2[i].astype(np.float64) <= kth * (1.0 + rel))
        tot += min(int(ok.sum()), den) / den
        cnt += 1
    return tot / max(cnt, 1)


def l_avg(final_L: np.ndarray) -> float:
    """Average beamwidth: mean over queries of the width of the last phase each one ran."""
    return float(np.mean(final_L))


def l_avg_from_split(percent_by_width: dict) -> float:
    """Same quantity from a table of 'percent of queries resolved at width L'."""
    tot = sum(percent_by_width.values())
    return sum(L * p for L, p in percent_by_width.items()) / tot


def phase_split(final_L: np.ndarray, widths) -> dict:
    """Percent of queries whose last phase ran at each width."""
    n = max(1, final_L.shape[0])
    return {int(w): 100.0 * float(np.sum(final_L == w)) / n for w in widths}
