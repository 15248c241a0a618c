"""Pins for the oracle's graph construction: a hand-worked three-point build and a hand-worked
pruning call, the pruning rule's defining properties, the limit of no pruning (R nearest), the
threshold passes, and the built graph's structure and search quality."""
import os

import numpy as np
import pytest

from boa_synth import C2, SENTINEL, make_workload
from oracle.boa_oracle import OracleIndex
from tests.test_oracle_pins import _read_golden

INF = float("inf")


def _points(x, R=2, entry=-1):
    x = np.asarray(x, dtype=np.float32)
    if x.ndim == 1:
        x = np.stack([x, np.zeros_like(x), np.zeros_like(x), np.zeros_like(x)], 1)
    n = x.shape[0]
    g = np.full((n, R), SENTINEL, dtype=np.uint32)
    return OracleIndex(x, np.zeros((n, 1), np.int32), np.zeros(1, np.int32), g, entry=entry)


def test_hand_worked_build_and_prune():
    rows = _read_golden("build_trace_three_points.txt")
    ix = _points([0.0, 1.0, 3.0])
    assert ix.entry == 1
    g = ix.build_graph(np.zeros((3, 1), np.float32), R=2, Lb=4, alpha=1.2, B=1)
    for r in rows:
        if r[0] == "row":
            want = [SENTINEL if v == "-" else int(v) for v in r[2:]]
            assert g[int(r[1])].tolist() == want
    xs = [0.0, 1.0, 2.0, 3.0, 10.0, -1.5]
    ix2 = _points(xs)
    row, n = ix2.prune(np.zeros((6, 1), np.float32), 0, [4, 3, 2, 1, 5, 5, 0], R=4, alpha=1.0)
    want = [xs.index(float(v)) for v in [r for r in rows if r[0] == "prune_selected"][0][1:]]
    assert n == 2 and row[:2].tolist() == want and (row[2:] == SENTINEL).all()


@pytest.fixture(scope="module")
def data():
    w = C2.scaled(3000, 50, name="c2_build")
    d = make_workload(w, seed=13, device="cpu")
    n = w.N
    pos = np.empty((n, 2), np.float32)
    for j in range(2):
        o = np.argsort(d["attrs"][:, j], kind="stable")
        pos[o, j] = np.arange(n, dtype=np.float32) / n
    return w, d, pos


def test_pruning_rule_properties(data):
    w, d, pos = data
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    x = d["vectors"].astype(np.float64)
    rng = np.random.default_rng(0)
    for p in (0, 17, 2999):
        ids = rng.choice(w.N, size=90, replace=False).astype(np.uint32)
        dp = ((x[ids] - x[p]) ** 2).sum(1)
        order = ids[np.lexsort((ids, dp))]
        order = order[order != p]
        # no pruning in the limit of a huge alpha: the R nearest candidates, in order
        row, n = ix.prune(pos, p, ids, R=16, alpha=1e9)
        assert n == 16 and row.tolist() == order[:16].tolist()
        # alpha = 1.2: a selected neighbour is never dominated by an earlier one, and whatever was
        # passed over while there was budget is dominated by an earlier selected one
        row, n = ix.prune(pos, p, ids, R=16, alpha=1.2)
        sel = row[:n].tolist()
        a2 = np.float32(1.2) * np.float32(1.2)
        dd = lambda a, b: np.float32(((x[a] - x[b]) ** 2).sum())
        for i, c in enumerate(sel):
            assert not any(np.float32(a2 * dd(e, c)) <= dd(p, c) for e in sel[:i])
        last = order.tolist().index(sel[-1]) if n == 16 else len(order)
        for c in order[:last]:
            if c not in sel:
                earlier = [e for e in sel if (dd(p, e), e) < (dd(p, c), c)]
                assert any(np.float32(a2 * dd(e, c)) <= dd(p, c) for e in earlier)
        # two threshold passes: half the budget for anything, half for attribute-near candidates
        row2, n2 = ix.prune(pos, p, ids, R=16, alpha=1.2, thresholds=(INF, 0.2))
        first, n1 = ix.prune(pos, p, ids, R=8, alpha=1.2)
        assert n2 >= n1 and row2[:n1].tolist() == first[:n1].tolist()
        assert n2 - n1 <= 8
        for c in row2[n1:n2]:
            assert np.abs(pos[c] - pos[p]).max() <= 0.2
        # a threshold that binds one attribute only: the second half is near in that attribute and
        # free in the others, and it is what a one-attribute position table gives
        if pos.shape[1] >= 2:
            one = (INF,) * (pos.shape[1] - 1) + (0.1,)
            row3, n3 = ix.prune(pos, p, ids, R=16, alpha=1.2, thresholds=(INF, one))
            assert row3[:n1].tolist() == first[:n1].tolist()
            assert all(abs(pos[c, -1] - pos[p, -1]) <= 0.1 for c in row3[n1:n3])
            row4, n4 = ix.prune(np.ascontiguousarray(pos[:, -1:]), p, ids, R=16, alpha=1.2, thresholds=(INF, 0.1))
            assert n3 == n4 and row3.tolist() == row4.tolist()


def test_built_graph_structure_and_quality(data):
    w, d, pos = data
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], np.zeros((w.N, 1), np.uint32))
    R = 16
    g = ix.build_graph(pos, R=R, Lb=32, alpha=1.2, thresholds=(INF, 0.15), B=256, passes=2)
    g2 = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], np.zeros((w.N, 1), np.uint32)).build_graph(
        pos, R=R, Lb=32, alpha=1.2, thresholds=(INF, 0.15), B=256, passes=2)
    assert (g == g2).all()                                               # deterministic
    real = g != SENTINEL
    assert (g[real] < w.N).all() and (g != np.arange(w.N, dtype=np.uint32)[:, None]).all()
    for r in range(0, w.N, 37):
        row = g[r][real[r]]
        assert len(set(row.tolist())) == len(row)
        assert (real[r][:-1] >= real[r][1:]).all()                       # padding only at the tail
    assert real.sum(1).mean() > R / 2
    # every point can be reached from the entry, and an unfiltered search finds the true neighbours
    seen = np.zeros(w.N, bool); seen[ix.entry] = True
    front = [ix.entry]
    while front:
        nb = np.unique(g[front][real[front]])
        nb = nb[~seen[nb]]
        seen[nb] = True
        front = nb.tolist()
    assert seen.mean() > 0.995
    full_lo = np.full((w.Q, 2), np.iinfo(np.int32).min, np.int32)
    full_hi = np.full((w.Q, 2), np.iinfo(np.int32).max, np.int32)
    r = ix.search(d["queries"], full_lo, full_hi, 10, [48])
    b_ids, _, _ = ix.bruteforce(d["queries"], full_lo, full_hi, 10)
    rec = np.mean([len(set(r["ids"][i].tolist()) & set(b_ids[i].tolist())) / 10 for i in range(w.Q)])
    assert rec > 0.9
    # the second threshold pass leaves its mark: far more attribute-near neighbours than the same
    # build without it (reverse edges that fit are appended without a pruning run, so a row can
    # hold more than R/2 attribute-far ones)
    plain = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], np.zeros((w.N, 1), np.uint32)).build_graph(
        pos, R=R, Lb=32, alpha=1.2, B=256, passes=2)
    def near_share(gr):
        rl = gr != SENTINEL
        return np.mean([(np.abs(pos[gr[r][rl[r]]] - pos[r]).max(1) <= 0.15).mean() for r in range(0, w.N, 11) if rl[r].any()])
    assert near_share(g) > near_share(plain) + 0.15
