"""Pins for the oracle's product-quantised search: the distance table and the look-up sum
against a hand-worked example and plain numpy, a lossless codebook (PQ distance equals the
exact distance, so the PQ search must equal the exact search), a full-width beam (the final
exact ranking must equal brute force whatever the codebook loses), and the properties of the
final ranking."""
import math
import os

import numpy as np
import pytest

from boa_synth import C2, C3, SENTINEL, clean_rows, exact_knn_graph, make_workload
from boa_synth.pq import train_pq
from oracle.boa_oracle import OracleIndex, default_widths

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FULL_LO, FULL_HI = np.iinfo(np.int32).min, np.iinfo(np.int32).max


def _tiny_index(x, pivots, codes, R=2):
    n = x.shape[0]
    g = ((np.arange(n)[:, None] + np.arange(1, R + 1)[None, :]) % n).astype(np.uint32)
    ix = OracleIndex(x, np.zeros((n, 1), np.int32), np.zeros(1, np.int32), g, entry=0)
    ix.attach_pq(pivots, codes)
    return ix


def test_table_and_lookup_sum_hand_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "pq_table_hand.txt")) if l.strip() and l[0] != "#"]
    pivots = np.array([[[0, 0], [1, 2]], [[3, 1], [-1, 0.5]]], dtype=np.float32)
    codes = np.array([[0, 1], [1, 0], [0, 0], [1, 1]], dtype=np.uint8)
    ix = _tiny_index(np.zeros((4, 4), np.float32), pivots, codes)
    q = np.array([1, 1, 2, 0], dtype=np.float32)
    for mode in (0, 1):
        t = ix.pq_table(q, mode)
        for r in rows:
            if r[0] == "table":
                assert t[int(r[1]), int(r[2])] == np.float32(r[3])
        for r in rows:
            if r[0] == "dist":
                p = int(np.nonzero((codes == [int(r[1]), int(r[2])]).all(1))[0][0])
                assert ix.pq_dist(t, p, mode) == np.float32(r[3])


def test_table_matches_numpy_and_fp32_order_is_sequential():
    w = C3.scaled(3000, 10, name="c3_pq_tab")
    d = make_workload(w, seed=9, device="cpu")
    piv, codes = train_pq(d["vectors"], M=12, K=64, iters=3, seed=1, device="cpu")
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    ix.attach_pq(piv, codes)
    q = d["queries"][0]
    dsub = w.D // 12
    want = ((q.reshape(12, 1, dsub).astype(np.float64) - piv.astype(np.float64)) ** 2).sum(-1)
    np.testing.assert_allclose(ix.pq_table(q, 0), want, rtol=2e-7)
    np.testing.assert_allclose(ix.pq_table(q, 1), want, rtol=(dsub + 1) * 2.0 ** -23)
    t0 = ix.pq_table(q, 0)
    for p in (0, 7, 2999):
        s = t0[np.arange(12), codes[p]].astype(np.float64).sum()
        assert abs(float(ix.pq_dist(t0, p, 0)) - s) <= 1e-6 * s
        assert abs(float(ix.pq_dist(t0, p, 1)) - s) <= 13 * 2.0 ** -23 * s
    # the fp32 sum runs over the subspaces in ascending order: 2^24 + 1 + 1 stays 2^24 that way,
    # any order that adds the two ones first gives 2^24 + 2
    piv2 = np.array([[[4096.0]], [[1.0]], [[1.0]]], dtype=np.float32)
    ix2 = _tiny_index(np.zeros((3, 3), np.float32), piv2, np.zeros((3, 3), np.uint8))
    t = ix2.pq_table(np.zeros(3, np.float32), 1)
    assert t[:, 0].tolist() == [16777216.0, 1.0, 1.0]
    assert ix2.pq_dist(t, 0, 1) == np.float32(16777216.0)
    assert ix2.pq_dist(t, 0, 0) == np.float32(16777218.0)


def _lossless_case(seed=0, N=700, Q=24):
    """Integer vectors whose 2-d subvectors take at most 64 values: a codebook holding every
    one of them loses nothing, so the PQ distance is the exact distance."""
    rng = np.random.default_rng(seed)
    D, M = 8, 4
    x = rng.integers(0, 8, size=(N, D)).astype(np.float32)
    a, b = np.meshgrid(np.arange(8), np.arange(8), indexing="ij")
    book = np.stack([a.ravel(), b.ravel()], 1).astype(np.float32)            # code = 8*a + b
    pivots = np.repeat(book[None], M, 0)
    codes = (x[:, 0::2] * 8 + x[:, 1::2]).astype(np.uint8)
    attrs = rng.integers(0, 100, size=(N, 2)).astype(np.int32)
    lo = rng.integers(0, 40, size=(Q, 2)).astype(np.int32)
    hi = (lo + rng.integers(30, 70, size=(Q, 2))).astype(np.int32)
    q = rng.integers(0, 8, size=(Q, D)).astype(np.float32)
    g = clean_rows(np.concatenate([exact_knn_graph(x, 6, device="cpu"),
                                   rng.integers(0, N, size=(N, 2)).astype(np.uint32)], 1))
    ix = OracleIndex(x, attrs, np.zeros(2, np.int32), g)
    ix.attach_pq(pivots, codes)
    return ix, q, lo, hi, x


def test_lossless_codebook_makes_pq_search_equal_exact_search():
    ix, q, lo, hi, x = _lossless_case()
    t = ix.pq_table(q[0], 1)
    for p in range(0, 700, 37):
        assert ix.pq_dist(t, p, 1) == np.float32(((x[p] - q[0]) ** 2).sum())
    for mode_d in (0, 1):
        for widths in ([12], [10, 40], [10, 30, 90]):
            a = ix.search(q, lo, hi, 5, widths, eps=0.1, mode="restart", dist_mode=mode_d)
            b = ix.search(q, lo, hi, 5, widths, eps=0.1, mode="restart", dist_mode=mode_d, pq=True)
            for key in ("ids", "d2", "final_L", "n_expand", "n_scored", "flags", "phase_active"):
                assert (a[key] == b[key]).all(), (widths, key)
    # finite lambda and expansion width 2 go through the same keys
    a = ix.search(q, lo, hi, 5, [10, 40], mode="restart", dist_mode=1, lam=3.0, expand_w=2)
    b = ix.search(q, lo, hi, 5, [10, 40], mode="restart", dist_mode=1, lam=3.0, expand_w=2, pq=True)
    assert (a["ids"] == b["ids"]).all() and (a["n_expand"] == b["n_expand"]).all()


def _lossy_case():
    w = C2.scaled(5000, 40, name="c2_pq_small")
    d = make_workload(w, seed=6, device="cpu")
    piv, codes = train_pq(d["vectors"], M=16, K=32, iters=4, seed=2, device="cpu")
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    ix.attach_pq(piv, codes)
    return w, d, ix


@pytest.fixture(scope="module")
def lossy():
    return _lossy_case()


def test_full_width_pq_search_is_exact_whatever_the_codebook_loses():
    rng = np.random.default_rng(3)
    N, D = 300, 8
    x = rng.standard_normal((N, D)).astype(np.float32)
    piv, codes = train_pq(x, M=2, K=4, iters=3, seed=0, device="cpu")       # a very coarse codebook
    ring = ((np.arange(N)[:, None] + np.array([1, N - 1])[None, :]) % N).astype(np.uint32)
    g = clean_rows(np.concatenate([exact_knn_graph(x, 4, device="cpu"), ring], 1))
    attrs = rng.integers(0, 10, size=(N, 1)).astype(np.int32)
    ix = OracleIndex(x, attrs, np.zeros(1, np.int32), g)
    ix.attach_pq(piv, codes)
    q = rng.standard_normal((12, D)).astype(np.float32)
    lo = np.full((12, 1), 2, np.int32)
    hi = np.full((12, 1), 6, np.int32)
    r = ix.search(q, lo, hi, 7, [N], mode="restart", dist_mode=0, cap=(8, 10 ** 6), pq=True)
    b_ids, b_d2, b_nv = ix.bruteforce(q, lo, hi, 7)
    assert (r["n_expand"] == N).all()
    assert (r["ids"] == b_ids).all()
    assert (r["d2"] == b_d2.astype(np.float32)).all()
    # and the coarse codebook really does lose something: the PQ order differs from the exact one
    t = ix.pq_table(q[0], 0)
    pqd = np.array([ix.pq_dist(t, p, 0) for p in range(N)])
    ex = ((x - q[0]) ** 2).sum(1)
    assert (np.argsort(pqd)[:20] != np.argsort(ex)[:20]).any()


def test_final_ranking_properties(lossy):
    w, d, ix = lossy
    k, L = 10, 24
    seen_unc = set()
    for i in range(w.Q):
        b = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=L, dist_mode=0, pq=True)
        ids, pq_d, phi, ex = b.pool()
        assert (np.diff(pq_d[phi == 0]) >= 0).all()                     # the pool is ordered by PQ distance
        t = ix.pq_table(d["queries"][i], 0)
        assert pq_d[0] == ix.pq_dist(t, ids[0], 0)
        valid = ids[:L][phi[:L] == 0]
        exact = np.array([np.float32(ix.dist2_f64(d["queries"][i], p)) for p in valid], dtype=np.float32)
        order = np.lexsort((valid, exact))
        r_ids, r_d2, nv, dk, dm = b.rerank(k)
        assert nv == len(valid)
        n = min(k, nv)
        assert (r_ids[:n] == valid[order][:n]).all() and (r_d2[:n] == exact[order][:n]).all()
        assert (r_ids[n:] == SENTINEL).all() and np.isinf(r_d2[n:]).all()
        if nv >= k:
            assert dk == exact[order][k - 1]
        if nv > 0:
            assert dm == exact.max()
        if nv > k:
            gamma = (math.sqrt(dm) - math.sqrt(dk)) / math.sqrt(dm) if dm > 0 else 0.0
            for eps in (0.02, 0.1, 0.3):
                if abs(gamma - eps) > 1e-4:
                    from oracle.boa_oracle import lib
                    u = bool(lib().orc_uncertain_reranked(nv, k, float(dk), float(dm), eps))
                    assert u == (gamma > eps)
                    seen_unc.add(u)
    assert seen_unc == {True, False}


def test_pq_driver_relations(lossy):
    w, d, ix = lossy
    q, lo, hi = d["queries"], d["lo"], d["hi"]
    widths = [16, 64, 128]
    # results are valid, sorted by exact distance, unique; distances are exact ones
    for mode in ("restart", "resume"):
        r = ix.search(q, lo, hi, 10, widths, eps=0.05, mode=mode, dist_mode=0, pq=True)
        for i in range(w.Q):
            got = r["ids"][i][r["ids"][i] != SENTINEL]
            assert len(set(got.tolist())) == len(got)
            for p in got:
                assert ix.phi(lo[i], hi[i], p) == 0
            dd = r["d2"][i][: len(got)]
            assert (np.diff(dd) >= 0).all()
            assert all(dd[j] == np.float32(ix.dist2_f64(q[i], got[j])) for j in range(len(got)))
    # resume carries the whole PQ search: one beam never saved or put back gives the same
    r = ix.search(q, lo, hi, 10, widths, eps=-1.0, mode="resume", dist_mode=1, pq=True)
    for i in range(0, w.Q, 3):
        b = ix.beam(q[i], lo[i], hi[i], L=16, C=128, dist_mode=1, max_expand=8 * 16 + 64, pq=True)
        b.run(64, 8 * 64 + 64)
        b.run(128, 8 * 128 + 64)
        ids, d2, nv, dk, dm = b.rerank(10, L=128)
        assert (ids == r["ids"][i]).all() and (d2 == r["d2"][i]).all()
        assert b.n_expand == r["n_expand"][i] and b.n_scored == r["n_scored"][i]
    # first phase of resume == first phase of restart; eps >= 1 resolves whoever has > k valid
    a = ix.search(q, lo, hi, 10, [16], mode="restart", dist_mode=1, pq=True)
    b2 = ix.search(q, lo, hi, 10, [16], mode="resume", dist_mode=1, pq=True)
    assert (a["ids"] == b2["ids"]).all() and (a["n_expand"] == b2["n_expand"]).all()
    e1 = ix.search(q, lo, hi, 10, widths, eps=1.0, mode="restart", dist_mode=1, pq=True)
    for i in range(w.Q):
        bb = ix.beam(q[i], lo[i], hi[i], L=16, dist_mode=1, pq=True)
        assert (e1["final_L"][i] == 16) == (bb.rerank(10)[2] > 10)
    # a wider beam on PQ keys does not lose recall against exact brute force (soft: half a point)
    b_ids, b_d2, b_nv = ix.bruteforce(q, lo, hi, 10)
    def rec(r):
        tot = 0.0
        for i in range(w.Q):
            den = min(10, int(b_nv[i]))
            if den:
                tot += len(set(r["ids"][i].tolist()) & set(b_ids[i][:den].tolist())) / den
        return tot / w.Q
    rs = [rec(ix.search(q, lo, hi, 10, [L], mode="restart", dist_mode=0, pq=True)) for L in (16, 64, 256)]
    assert rs[1] >= rs[0] - 0.005 and rs[2] >= rs[1] - 0.005 and rs[2] > 0.8
