"""Pins for the CPU oracle: each test ties one oracle function to something the
paper or plain mathematics fixes, independent of the oracle's own code."""
import math
import os

import numpy as np
import pytest
import torch

from boa_synth import C1, C2, C3, SENTINEL, clean_rows, exact_knn_graph, make_workload
from boa_synth.metrics import l_avg, l_avg_from_split, recall_tie_aware
from oracle.boa_oracle import OracleIndex, default_widths

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FULL_LO, FULL_HI = np.iinfo(np.int32).min, np.iinfo(np.int32).max


def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ----------------------------------------------------------------------------
# small shared inputs
# ----------------------------------------------------------------------------
@pytest.fixture(scope="module")
def small():
    w = C2.scaled(6000, 60, name="c2_small")
    d = make_workload(w, seed=3, device="cpu")
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    return w, d, ix


@pytest.fixture(scope="module")
def small_float():
    w = C3.scaled(5000, 40, name="c3_small")
    d = make_workload(w, seed=4, device="cpu")
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    return w, d, ix


def _valid_mask(d, i):
    a = d["attrs"]
    ok = np.ones(a.shape[0], dtype=bool)
    for j, t in enumerate(d["attr_types"]):
        if t == 1:
            col, l, h = a[:, j].view(np.float32), d["lo"][i, j:j + 1].view(np.float32)[0], \
                d["hi"][i, j:j + 1].view(np.float32)[0]
        else:
            col, l, h = a[:, j], d["lo"][i, j], d["hi"][i, j]
        ok &= (col >= l) & (col <= h)
    return ok


# ----------------------------------------------------------------------------
# P1: exact filtered top-k against an independent sort-everything, and against
#     a library k-NN when every predicate is the full range (g == 1)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["small", "small_float"])
def test_bruteforce_matches_sort_everything(which, request):
    w, d, ix = request.getfixturevalue(which)
    k = 10
    ids, d2, nvalid = ix.bruteforce(d["queries"], d["lo"], d["hi"], k)
    x = d["vectors"].astype(np.float64)
    for i in range(d["queries"].shape[0]):
        ok = _valid_mask(d, i)
        assert nvalid[i] == ok.sum()
        dist = ((x - d["queries"][i].astype(np.float64)) ** 2).sum(1)
        cand = np.nonzero(ok)[0]
        order = cand[np.lexsort((cand, dist[cand]))][:k]
        n = len(order)
        assert list(ids[i][:n]) == list(order)
        np.testing.assert_allclose(d2[i][:n], dist[order], rtol=1e-12)
        assert (ids[i][n:] == SENTINEL).all() and np.isinf(d2[i][n:]).all()


def test_bruteforce_full_range_is_plain_knn(small_float):
    w, d, ix = small_float
    q = d["queries"]
    lo = np.full((q.shape[0], w.m), FULL_LO, dtype=np.int32)
    hi = np.full((q.shape[0], w.m), FULL_HI, dtype=np.int32)
    for j, t in enumerate(d["attr_types"]):
        if t == 1:
            lo[:, j] = np.array([-np.inf], dtype=np.float32).view(np.int32)[0]
            hi[:, j] = np.array([np.inf], dtype=np.float32).view(np.int32)[0]
    ids, d2, nvalid = ix.bruteforce(q, lo, hi, 10)
    assert (nvalid == w.N).all()
    dist = torch.cdist(torch.from_numpy(q).double(), torch.from_numpy(d["vectors"]).double()) ** 2
    ref = torch.topk(dist, 10, dim=1, largest=False)
    np.testing.assert_allclose(d2, ref.values.numpy(), rtol=1e-9)
    assert (np.sort(ids, 1) == np.sort(ref.indices.numpy().astype(np.uint32), 1)).all()


# ----------------------------------------------------------------------------
# distances and filter distance
# ----------------------------------------------------------------------------
def test_dist2_integer_data_is_exact_in_both_modes(small):
    w, d, ix = small
    rng = np.random.default_rng(0)
    for _ in range(200):
        p = int(rng.integers(w.N))
        q = d["queries"][int(rng.integers(w.Q))]
        exact = int(((d["vectors"][p].astype(np.int64) - q.astype(np.int64)) ** 2).sum())
        assert exact < 2 ** 24
        assert ix.dist2_f64(q, p) == float(exact)
        assert float(ix.dist2_lanes(q, p)) == float(exact)


def test_dist2_lanes_close_to_double_on_float_data(small_float):
    w, d, ix = small_float
    rng = np.random.default_rng(1)
    for _ in range(200):
        p = int(rng.integers(w.N))
        q = d["queries"][int(rng.integers(w.Q))]
        ref = ix.dist2_f64(q, p)
        # each of the ~D/8+3 roundings on a path contributes at most 2^-24 relative
        assert abs(float(ix.dist2_lanes(q, p)) - ref) <= ref * (w.D / 8 + 8) * 2.0 ** -24


def test_dist2_lanes_order_on_a_cancellation_probe():
    """The fp32 order is observable: with one huge and many tiny terms the result
    depends on which partial sum the huge term joins.  Element i lives in 16-byte
    chunk i//4, chunk c in partial sum c%8; partial sums meet as
    ((p0+p4)+(p2+p6)) + ((p1+p5)+(p3+p7))."""
    D = 64
    x = np.zeros((2, D), dtype=np.float32)
    q = np.zeros(D, dtype=np.float32)
    big = np.float32(4096.0)         # big^2 = 2^24: adding 1.0 to it is lost in fp32
    x[0, 0] = big                    # chunk 0 -> partial 0
    x[0, 1:4] = 1.0                  # same chunk, same partial: three 1s are absorbed one by one
    x[0, 4:8] = 1.0                  # chunk 1 -> partial 1: sums to 4 exactly
    g = np.full((2, 1), SENTINEL, dtype=np.uint32)
    ix = OracleIndex(x, np.zeros((2, 1), np.int32), np.zeros(1, np.int32), g, entry=0)
    got = float(ix.dist2_lanes(q, 0))
    # partial 0: 2^24 (+1 three times, each rounded away); partial 1: 4; then 2^24 + 4 = exact
    assert got == 2.0 ** 24 + 4.0
    assert ix.dist2_f64(q, 0) == 2.0 ** 24 + 7.0


def test_phi_counts_violated_closed_ranges():
    x = np.zeros((4, 4), dtype=np.float32)
    attrs = np.zeros((4, 3), dtype=np.int32)
    attrs[:, 0] = [5, 10, 15, 20]
    attrs[:, 1] = np.array([0.25, 0.5, 0.75, np.nan], dtype=np.float32).view(np.int32)
    attrs[:, 2] = [-3, 0, 3, 7]
    types = np.array([0, 1, 0], dtype=np.int32)
    g = np.full((4, 1), SENTINEL, dtype=np.uint32)
    ix = OracleIndex(x, attrs, types, g, entry=0)
    lo = np.array([10, 0, -3], dtype=np.int32)
    hi = np.array([15, 0, 3], dtype=np.int32)
    lo[1] = np.array([0.5], dtype=np.float32).view(np.int32)[0]
    hi[1] = np.array([0.75], dtype=np.float32).view(np.int32)[0]
    # closed on both ends; NaN violates; counts, not a flag
    assert [ix.phi(lo, hi, p) for p in range(4)] == [2, 0, 0, 3]
    # lo > hi: empty interval, every point violates it
    lo2, hi2 = lo.copy(), hi.copy()
    lo2[0], hi2[0] = 16, 9
    assert [ix.phi(lo2, hi2, p) for p in range(4)] == [2, 1, 1, 3]


def test_medoid_closed_form():
    # points on a line: mean is 3.2, nearest point is x=3 (id 2); ties go to the lower id
    x = np.array([[0.0], [1.0], [3.0], [4.0], [8.0]], dtype=np.float32)
    g = np.full((5, 1), SENTINEL, dtype=np.uint32)
    z = np.zeros((5, 1), np.int32)
    assert OracleIndex(x, z, np.zeros(1, np.int32), g).entry == 2
    x2 = np.array([[0.0], [2.0], [4.0], [6.0]], dtype=np.float32)   # mean 3: ids 1 and 2 tie
    assert OracleIndex(x2, z[:4], np.zeros(1, np.int32), g[:4]).entry == 1
    # uint8 rows
    x3 = np.array([[10, 0], [20, 0], [90, 0]], dtype=np.uint8)      # mean 40 -> id 1
    assert OracleIndex(x3, z[:3], np.zeros(1, np.int32), g[:3]).entry == 1


# ----------------------------------------------------------------------------
# P11: the hand trace
# ----------------------------------------------------------------------------
def _ring():
    x = np.arange(8, dtype=np.float32)[:, None]
    attrs = (np.arange(8) % 2).astype(np.int32)[:, None]
    g = np.stack([(np.arange(8) - 1) % 8, (np.arange(8) + 1) % 8], 1).astype(np.uint32)
    return OracleIndex(x, attrs, np.zeros(1, np.int32), g, entry=0)


def test_ring_hand_trace():
    gold = {r[0]: r[1:] for r in _read_golden("ring_trace.txt")}
    ix = _ring()
    q = np.array([5.2], dtype=np.float32)
    lo = np.array([1], dtype=np.int32)
    hi = np.array([1], dtype=np.int32)
    b2 = ix.beam(q, lo, hi, L=3, C=3)
    assert b2.n_expand == len(gold["expansion_order"]) == 5
    assert b2.n_scored == len(gold["scored_order"]) == 6
    ids, d2, phi, ex = b2.pool()
    assert [int(i) for i in ids] == [int(v) for v in gold["final_pool"]]
    assert ex.all()
    rid, rd2, n = b2.result(2)
    assert n == 2 and [int(i) for i in rid] == [int(v) for v in gold["result_ids"]]
    np.testing.assert_allclose(rd2, [float(v) for v in gold["result_d2"]], rtol=1e-5)
    assert b2.uncertain(2, eps=0.05)
    gamma = 1.0 - math.sqrt(float(d2[1]) / float(d2[2]))
    assert abs(gamma - float(gold["gamma"][0])) < 1e-5
    # node 3 is never scored: not in any pool, and total scored + entry == 7 nodes
    assert int(gold["never_seen"][0]) not in [int(i) for i in ids]
    # step-wise: one expansion per step, five steps, scored counts 2,3,4,5,6
    b3 = ix.beam(q, lo, hi, L=3, C=3, max_expand=0)
    want_pools = [[7, 1, 0], [7, 1, 6], [7, 1, 6], [5, 7, 1], [5, 7, 1]]
    want_scored = [2, 3, 4, 5, 6]
    for s in range(5):
        b3.run(3, max_expand=1)
        ids3 = [int(i) for i in b3.pool()[0]]
        assert ids3 == want_pools[s]
        assert b3.n_scored == want_scored[s]
    b3.run(3, max_expand=1)
    assert not b3.hit_cap and b3.n_expand == 5


def test_ring_walk_passes_through_invalid_nodes():
    """Invalid candidates are demoted, not removed: valid node 5 is reachable from
    valid node 7 only through invalid node 6."""
    ix = _ring()
    b = ix.beam(np.array([5.2], np.float32), np.array([1], np.int32), np.array([1], np.int32), L=3)
    assert 5 in [int(i) for i in b.result(2)[0]]


# ----------------------------------------------------------------------------
# finite lambda: the score dist + lambda*phi as the paper states it
# ----------------------------------------------------------------------------
def test_ring_hand_traces_with_finite_lambda():
    gold = {r[0]: [int(v) for v in r[1:]] for r in _read_golden("ring_trace_finite_lambda.txt")}
    ix = _ring()
    q = np.array([5.2], dtype=np.float32)
    one = np.array([1], dtype=np.int32)
    for lam, tag in ((2.0, "l2"), (0.5, "l05")):
        b = ix.beam(q, one, one, L=3, C=3, lam=lam)
        assert b.n_expand == len(gold[tag + "_expansions"])
        assert b.n_scored == len(gold[tag + "_scored"])
        ids, d2, phi, ex = b.pool()
        assert [int(i) for i in ids] == gold[tag + "_final_pool"]
        rid, rd2, n = b.result(2)
        assert [int(i) for i in rid[:n]] == gold[tag + "_result_ids"]
        assert (rid[n:] == SENTINEL).all()
    # the lexicographic order expands node 1, lambda = 2 does not
    assert ix.beam(q, one, one, L=3, C=3).n_expand == 5


def test_lambda_zero_walks_like_an_unfiltered_search(small):
    """With lambda = 0 the predicates cannot steer the walk: the pool is that of a search
    whose ranges admit everything, and the answer is its filter-valid part."""
    w, d, ix = small
    everything_lo = np.full(w.m, np.iinfo(np.int32).min, dtype=np.int32)
    everything_hi = np.full(w.m, np.iinfo(np.int32).max, dtype=np.int32)
    for i in range(8):
        a = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=32, lam=0.0)
        b = ix.beam(d["queries"][i], everything_lo, everything_hi, L=32)
        assert (a.pool()[0] == b.pool()[0]).all() and a.n_scored == b.n_scored
        ok = _valid_mask(d, i)
        want = [int(v) for v in b.pool()[0] if ok[int(v)]][:w.k]
        got = a.result(w.k)
        assert [int(v) for v in got[0][:got[2]]] == want


def test_large_exact_lambda_equals_the_lexicographic_order():
    """Integer data with every d2 < 1024 and lambda = 1024: the score d2 + 1024*phi is exact
    in fp32 and orders like (phi, d2), so the two searches are the same search."""
    rng = np.random.default_rng(5)
    N, D, R, k = 400, 4, 6, 5
    x = rng.integers(0, 16, size=(N, D)).astype(np.float32)          # d2 <= 4*15^2 = 900
    attrs = rng.integers(0, 10, size=(N, 3)).astype(np.int32)
    g = rng.integers(0, N, size=(N, R)).astype(np.uint32)
    g[:, 0] = (np.arange(N) + 1) % N
    ix = OracleIndex(x, attrs, np.zeros(3, np.int32), g)
    q = rng.integers(0, 16, size=(12, D)).astype(np.float32)
    lo = rng.integers(0, 5, size=(12, 3)).astype(np.int32)
    hi = (lo + rng.integers(0, 5, size=(12, 3))).astype(np.int32)
    a = ix.search(q, lo, hi, k, [6, 24], mode="resume", lam=1024.0)
    b = ix.search(q, lo, hi, k, [6, 24], mode="resume")
    for key in ("ids", "d2", "final_L", "n_expand", "n_scored"):
        assert (a[key] == b[key]).all(), key
    c = ix.search(q, lo, hi, k, [6, 24], mode="resume", lam=8.0)      # a small lambda does differ
    assert (c["n_scored"] != b["n_scored"]).any()


# ----------------------------------------------------------------------------
# expansion width W > 1 (an extension of Algorithm 2): a second hand trace
# ----------------------------------------------------------------------------
def _stride_line():
    n = 16
    x = np.arange(n, dtype=np.float32)[:, None]
    attrs = np.zeros((n, 1), dtype=np.int32)
    g = np.full((n, 4), SENTINEL, dtype=np.uint32)
    for i in range(n):
        for c, o in enumerate((-2, -1, 1, 2)):
            if 0 <= i + o < n:
                g[i, c] = i + o
    return OracleIndex(x, attrs, np.zeros(1, np.int32), g, entry=0)


def test_stride_line_hand_trace_width_1_and_2():
    gold = {r[0]: [int(v) for v in r[1:]] for r in _read_golden("stride_trace_width2.txt")}
    ix = _stride_line()
    q = np.array([10.1], dtype=np.float32)
    z = np.zeros(1, dtype=np.int32)
    for w, tag in ((1, "w1"), (2, "w2"), (3, "w2")):     # the beam holds two entries: W = 3 picks two
        b = ix.beam(q, z, z, L=2, C=8, expand_w=w)
        ids, d2, phi, ex = b.pool()
        assert [int(i) for i in ids] == gold["final_pool"]
        assert [int(e) for e in ex] == gold[tag + "_expanded_flags"]
        assert b.n_expand == len(gold[tag + "_expansions"])
        assert b.n_scored == len(gold["scored_order"])
        assert not b.hit_cap
        assert [int(i) for i in b.result(2)[0]] == [10, 11]
    # the cap is counted in nodes, not in iterations
    b = ix.beam(q, z, z, L=2, C=8, expand_w=2, max_expand=4)
    ids, d2, phi, ex = b.pool()
    assert b.n_expand == 4 and b.hit_cap
    assert [int(i) for i in ids] == gold["w2_cap4_pool"]
    assert [int(e) for e in ex] == gold["w2_cap4_flags"]
    # the order in which nodes become expanded: a cap of c nodes leaves exactly the first c
    # of the hand-derived order expanded (capacity 16 keeps every scored node in the pool)
    for c in range(1, 13):
        b = ix.beam(q, z, z, L=2, C=16, expand_w=2, max_expand=c)
        ids, _, _, ex = b.pool()
        assert sorted(int(i) for i, e in zip(ids, ex) if e) == sorted(gold["w2_expansions"][:c])
        assert b.hit_cap == (c < 12)


@pytest.mark.parametrize("w", [2, 3, 7])
def test_any_expansion_width_at_full_beam_equals_bruteforce(w):
    rng = np.random.default_rng(11)
    N, D, R, k = 200, 6, 5, 8
    x = rng.integers(0, 32, size=(N, D)).astype(np.float32)
    attrs = rng.integers(0, 100, size=(N, 2)).astype(np.int32)
    g = rng.integers(0, N, size=(N, R)).astype(np.uint32)
    g[:, 0] = (np.arange(N) + 1) % N
    ix = OracleIndex(x, attrs, np.zeros(2, np.int32), g)
    q = rng.integers(0, 32, size=(10, D)).astype(np.float32)
    lo = rng.integers(0, 50, size=(10, 2)).astype(np.int32)
    hi = (lo + rng.integers(20, 60, size=(10, 2))).astype(np.int32)
    gt_ids, gt_d2, nvalid = ix.bruteforce(q, lo, hi, k)
    for i in range(10):
        b = ix.beam(q[i], lo[i], hi[i], L=N, C=N, expand_w=w)
        assert b.n_expand == N and b.n_scored == N - 1      # every node once, whatever W
        assert (b.result(k)[0] == gt_ids[i]).all()
    r1 = ix.search(q, lo, hi, k, [8, 32], eps=0.05, mode="resume", expand_w=1)
    rw = ix.search(q, lo, hi, k, [8, 32], eps=0.05, mode="resume", expand_w=w)
    # narrow beams: whatever W, answers are no better than exact and the cap holds per phase
    for r in (r1, rw):
        for i in range(10):
            n = int((r["ids"][i] != SENTINEL).sum())
            assert (r["d2"][i][:n].astype(np.float64) >= gt_d2[i][:n]).all()
            assert (r["n_expand"][i] <= 2 * (8 * 32 + 64)).all()


# ----------------------------------------------------------------------------
# P4: on a graph connected from s with L = C >= N the search sees every node,
#     so its answer is the exact filtered top-k
# ----------------------------------------------------------------------------
def test_full_width_search_equals_bruteforce():
    rng = np.random.default_rng(7)
    N, D, R, k = 300, 8, 6, 10
    x = rng.integers(0, 32, size=(N, D)).astype(np.float32)
    attrs = rng.integers(0, 100, size=(N, 2)).astype(np.int32)
    g = exact_knn_graph(x, R - 1, device="cpu")
    ring = ((np.arange(N) + 1) % N).astype(np.uint32)[:, None]      # makes it strongly connected
    g = clean_rows(np.concatenate([g, ring], 1))
    ix = OracleIndex(x, attrs, np.zeros(2, np.int32), g)
    q = rng.integers(0, 32, size=(25, D)).astype(np.float32)
    lo = rng.integers(0, 50, size=(25, 2)).astype(np.int32)
    hi = (lo + rng.integers(20, 60, size=(25, 2))).astype(np.int32)
    gt_ids, gt_d2, nvalid = ix.bruteforce(q, lo, hi, k)
    for i in range(25):
        b = ix.beam(q[i], lo[i], hi[i], L=N, C=N)
        assert b.n_expand == N and b.n_scored == N - 1
        ids, d2, n = b.result(k)
        assert n == min(k, nvalid[i])
        assert (ids == gt_ids[i]).all()
        assert (d2[:n].astype(np.float64) == gt_d2[i][:n]).all()   # integer data: exact


# ----------------------------------------------------------------------------
# P2, P3: validity, order, uniqueness, padding of every returned list
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["restart", "resume"])
@pytest.mark.parametrize("which", ["small", "small_float"])
def test_results_valid_sorted_unique(which, mode, request):
    w, d, ix = request.getfixturevalue(which)
    r = ix.search(d["queries"], d["lo"], d["hi"], 10, default_widths(16, 128), mode=mode)
    for i in range(w.Q):
        ids, d2 = r["ids"][i], r["d2"][i]
        n = int((ids != SENTINEL).sum())
        assert (ids[n:] == SENTINEL).all() and np.isinf(d2[n:]).all()
        ok = _valid_mask(d, i)
        assert ok[ids[:n].astype(np.int64)].all()
        assert len(set(ids[:n].tolist())) == n
        keys = list(zip(d2[:n].tolist(), ids[:n].tolist()))
        assert keys == sorted(keys)


# ----------------------------------------------------------------------------
# P5, P6: restart / resume relations
# ----------------------------------------------------------------------------
def test_resume_first_phase_equals_restart_first_phase(small):
    w, d, ix = small
    a = ix.search(d["queries"], d["lo"], d["hi"], 10, [16], mode="restart")
    b = ix.search(d["queries"], d["lo"], d["hi"], 10, [16], mode="resume")
    assert (a["ids"] == b["ids"]).all() and (a["d2"] == b["d2"]).all()
    assert (a["n_expand"] == b["n_expand"]).all() and (a["n_scored"] == b["n_scored"]).all()


def test_resume_kth_distance_never_grows(small):
    w, d, ix = small
    prev = None
    for n in range(1, 4):
        r = ix.search(d["queries"], d["lo"], d["hi"], 10, [16, 64, 128][:n], eps=-1.0, mode="resume")
        kth = r["d2"][:, 9]
        if prev is not None:
            assert (kth <= prev).all()
        prev = kth


def test_resume_continues_the_same_search(small):
    """What resume mode carries from phase to phase is the whole search: one beam that is
    never saved or put back, run at 16, then on at 64, then on at 128 with the pool capacity
    of the last width, must give the driver's resume-mode results, and the same cumulative
    expansion and scoring counts (a restore that lost the expanded flags would expand nodes
    again; one that lost part of the seen set would score nodes again)."""
    w, d, ix = small
    widths = [16, 64, 128]
    r = ix.search(d["queries"], d["lo"], d["hi"], 10, widths, eps=-1.0, mode="resume")
    assert (r["final_L"] == 128).all()
    grew = 0
    for i in range(w.Q):
        b = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=16, C=128, max_expand=8 * 16 + 64)
        e0 = b.n_expand
        b.run(64, 8 * 64 + 64)
        e1 = b.n_expand
        b.run(128, 8 * 128 + 64)
        ids, d2, _ = b.result(10)
        assert (ids == r["ids"][i]).all() and (d2 == r["d2"][i]).all()
        assert b.n_expand == r["n_expand"][i]
        assert b.n_scored == r["n_scored"][i]
        _, _, _, ex = b.pool()
        assert ex[:128].all()
        # later phases do continue, and do not start over: they expand more nodes, fewer
        # than a fresh search at that width would
        grew += int(e1 > e0)
        fresh = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=128, C=128)
        assert b.n_expand - e1 <= fresh.n_expand
    assert grew > w.Q // 2
    # two phases: the same relation with one hand-over
    r2 = ix.search(d["queries"], d["lo"], d["hi"], 10, [16, 64], eps=-1.0, mode="resume")
    for i in range(0, w.Q, 3):
        b = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=16, C=64, max_expand=8 * 16 + 64)
        b.run(64, 8 * 64 + 64)
        assert (b.result(10)[0] == r2["ids"][i]).all()
        assert b.n_expand == r2["n_expand"][i] and b.n_scored == r2["n_scored"][i]


def test_single_width_schedule_is_plain_fixed_L(small):
    w, d, ix = small
    a = ix.search(d["queries"], d["lo"], d["hi"], 10, [64], mode="restart")
    b = ix.search(d["queries"], d["lo"], d["hi"], 10, [64], mode="resume")
    assert (a["ids"] == b["ids"]).all() and (a["final_L"] == 64).all()
    for i in range(0, w.Q, 7):
        one = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=64)
        assert (one.result(10)[0] == a["ids"][i]).all()
        assert one.n_expand == a["n_expand"][i]


# ----------------------------------------------------------------------------
# P7: queries are independent
# ----------------------------------------------------------------------------
def test_batch_permutation_permutes_outputs(small):
    w, d, ix = small
    perm = np.random.default_rng(5).permutation(w.Q)
    a = ix.search(d["queries"], d["lo"], d["hi"], 10, default_widths(16, 128))
    b = ix.search(d["queries"][perm], d["lo"][perm], d["hi"][perm], 10, default_widths(16, 128))
    assert (a["ids"][perm] == b["ids"]).all() and (a["final_L"][perm] == b["final_L"]).all()


# ----------------------------------------------------------------------------
# P8 and Eq. 3: the confidence test
# ----------------------------------------------------------------------------
def test_uncertainty_matches_gamma_formula_away_from_the_boundary(small):
    w, d, ix = small
    k = 10
    seen_both = set()
    for L in (16, 32):
        for i in range(w.Q):
            b = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=L)
            ids, d2, phi, ex = b.pool()
            v = d2[:L][phi[:L] == 0].astype(np.float64)
            for eps in (0.02, 0.05, 0.2, 0.5):
                if len(v) <= k:
                    assert b.uncertain(k, eps)
                    continue
                dk, dmax = math.sqrt(v[k - 1]), math.sqrt(v[-1])
                gamma = (dmax - dk) / dmax if dmax > 0 else 0.0
                if abs(gamma - eps) < 1e-4:
                    continue
                assert b.uncertain(k, eps) == (gamma > eps)
                seen_both.add(gamma > eps)
    assert seen_both == {True, False}


def test_eps_special_cases(small):
    w, d, ix = small
    widths = default_widths(16, 128)
    # eps >= 1: whoever has more than k valid beam entries is done after phase 0
    r = ix.search(d["queries"], d["lo"], d["hi"], 10, widths, eps=1.0)
    for i in range(w.Q):
        b = ix.beam(d["queries"][i], d["lo"][i], d["hi"][i], L=16)
        nv = int((b.pool()[2][:16] == 0).sum())
        assert (r["final_L"][i] == 16) == (nv > 10)
    # eps < 0: nobody is ever confident; restart mode then equals fixed L = Lmax
    r2 = ix.search(d["queries"], d["lo"], d["hi"], 10, widths, eps=-1.0)
    fixed = ix.search(d["queries"], d["lo"], d["hi"], 10, [128])
    assert (r2["final_L"] == 128).all() and (r2["phase_active"] == w.Q).all()
    assert (r2["ids"] == fixed["ids"]).all()
    # all candidates at one distance: gamma = 0, confident
    x = np.ones((40, 4), dtype=np.float32)
    g = ((np.arange(40)[:, None] + np.arange(1, 5)[None, :]) % 40).astype(np.uint32)
    ix2 = OracleIndex(x, np.zeros((40, 1), np.int32), np.zeros(1, np.int32), g, entry=0)
    b = ix2.beam(np.zeros(4, np.float32), np.array([0], np.int32), np.array([0], np.int32), L=16)
    assert not b.uncertain(10, 0.05) and not b.uncertain(10, 0.0)
    assert b.uncertain(15, 0.05) is False and b.uncertain(16, 0.05) is True   # needs > k valid


def test_tau_stops_the_loop(small):
    w, d, ix = small
    widths = default_widths(16, 128)
    r0 = ix.search(d["queries"], d["lo"], d["hi"], 10, widths, tau=0.0)
    act = r0["phase_active"]
    assert act[0] == w.Q and act[1] < act[0]
    tau = (act[1] + 0.5) / w.Q          # |A| after phase 0 is not > tau*Q: phase 1 must not run
    r1 = ix.search(d["queries"], d["lo"], d["hi"], 10, widths, tau=tau)
    assert r1["phase_active"][1] == 0 and (r1["final_L"] == 16).all()


def test_tau_boundary_is_strict(small):
    """Algorithm 1 loops while |A| > tau * rho: with tau * rho equal to |A| exactly the next
    phase must not run, with one query fewer it must.  The batch has a power-of-two size so
    that tau = |A| / rho is exact in floating point."""
    w, d, ix = small
    Q = 32
    q, lo, hi = d["queries"][:Q], d["lo"][:Q], d["hi"][:Q]
    widths = default_widths(16, 128)
    seen = set()
    for eps in (0.05, 0.1):
        act = ix.search(q, lo, hi, 10, widths, eps=eps, tau=0.0)["phase_active"]
        a1 = int(act[1])
        assert 1 < a1 < Q
        assert (a1 / Q) * Q == a1
        stop = ix.search(q, lo, hi, 10, widths, eps=eps, tau=a1 / Q)
        assert stop["phase_active"][1] == 0 and (stop["final_L"] == 16).all()
        go = ix.search(q, lo, hi, 10, widths, eps=eps, tau=(a1 - 1) / Q)
        assert go["phase_active"][1] == a1 and (go["final_L"] > 16).sum() == a1
        seen.add(a1)
    assert len(seen) == 2


# ----------------------------------------------------------------------------
# P9: the average-beamwidth metric reproduces the paper's printed ranges
# ----------------------------------------------------------------------------
def test_l_avg_definition_reproduces_printed_ranges():
    rows = _read_golden("table3_phase_split.txt")
    widths = [10, 100, 200]
    by_m = {}
    ranges = {}
    for r in rows:
        if r[0] == "range":
            ranges[int(r[1])] = (float(r[2]), float(r[3]))
            continue
        split = {L: float(p) for L, p in zip(widths, r[2:5]) if p != "-"}
        by_m.setdefault(int(r[1]), []).append(l_avg_from_split(split))
    for m, (lo, hi) in ranges.items():
        assert abs(min(by_m[m]) - lo) <= 1.0, (m, min(by_m[m]), lo)
        assert abs(max(by_m[m]) - hi) <= 1.0, (m, max(by_m[m]), hi)
    # and the per-query form agrees with the table form
    final_L = np.array([10] * 861 + [100] * 139)
    assert abs(l_avg(final_L) - l_avg_from_split({10: 86.1, 100: 13.9})) < 1e-9


# ----------------------------------------------------------------------------
# P10: a wider beam does not lose recall (batch mean, soft)
# ----------------------------------------------------------------------------
def test_recall_does_not_drop_as_beam_widens(small):
    w, d, ix = small
    gt_ids, gt_d2, nvalid = ix.bruteforce(d["queries"], d["lo"], d["hi"], 10)
    prev = -1.0
    for L in (16, 32, 64, 128, 256):
        r = ix.search(d["queries"], d["lo"], d["hi"], 10, [L])
        rec = recall_tie_aware(r["ids"], r["d2"], gt_d2, nvalid, 10)
        assert rec >= prev - 0.005
        prev = rec
    assert prev > 0.9


def test_expansion_cap_is_honoured(small):
    w, d, ix = small
    r = ix.search(d["queries"], d["lo"], d["hi"], 10, [64], cap=(0, 5))
    assert (r["n_expand"] <= 5).all() and (r["flags"] & 1).any()


# ----------------------------------------------------------------------------
# the harness's blocked brute force (used for recall on large batches) against the oracle's
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["small", "small_float"])
def test_harness_ground_truth_equals_oracle_bruteforce(which, request):
    from boa_synth.groundtruth import filtered_topk, recall_against
    w, d, ix = request.getfixturevalue(which)
    t = {k: torch.from_numpy(d[k]) for k in ("vectors", "attrs", "queries", "lo", "hi")}
    ids, d2, nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"], t["lo"],
                                t["hi"], 10, block=16)
    o_ids, o_d2, o_nv = ix.bruteforce(d["queries"], d["lo"], d["hi"], 10)
    assert (nv.numpy() == o_nv).all()
    fin = o_ids != SENTINEL
    np.testing.assert_allclose(d2.numpy()[fin], o_d2[fin], rtol=1e-12)
    assert (ids.numpy()[fin] == o_ids[fin].astype(np.int64)).all()
    # an exact answer scores recall 1, a shifted one less
    rec = recall_against(o_ids, o_d2.astype(np.float32), d2.numpy(), nv.numpy(), 10, rel=1e-5)
    assert np.nanmin(rec) == 1.0
    worse = recall_against(o_ids, (o_d2 * 4.0 + 1.0).astype(np.float32), d2.numpy(), nv.numpy(), 10)
    assert np.nanmean(worse) < 0.5


# ----------------------------------------------------------------------------
# the same closed forms on many random tiny inputs
# ----------------------------------------------------------------------------
def test_random_tiny_graphs_full_width_is_exact_and_narrow_is_valid():
    from hypothesis import given, settings, strategies as st

    @settings(max_examples=60, deadline=None)
    @given(st.integers(0, 10 ** 6), st.integers(8, 60), st.integers(2, 5), st.integers(1, 3))
    def check(seed, N, R, m):
        rng = np.random.default_rng(seed)
        x = rng.integers(0, 16, size=(N, 4)).astype(np.float32)
        attrs = rng.integers(0, 10, size=(N, m)).astype(np.int32)
        g = rng.integers(0, N, size=(N, R)).astype(np.uint32)
        g[:, 0] = (np.arange(N) + 1) % N                       # a ring keeps it strongly connected
        g[rng.random((N, R)) < 0.2] = SENTINEL
        g[:, 0] = (np.arange(N) + 1) % N
        ix = OracleIndex(x, attrs, np.zeros(m, np.int32), g, entry=int(rng.integers(N)))
        q = rng.integers(0, 16, size=(3, 4)).astype(np.float32)
        lo = rng.integers(0, 6, size=(3, m)).astype(np.int32)
        hi = (lo + rng.integers(0, 8, size=(3, m))).astype(np.int32)
        k = int(rng.integers(1, 6))
        gt_ids, gt_d2, nvalid = ix.bruteforce(q, lo, hi, k)
        for mode in ("restart", "resume"):
            full = ix.search(q, lo, hi, k, [max(k, 4), N], eps=-1.0, mode=mode)
            assert (full["ids"] == gt_ids).all()
            narrow = ix.search(q, lo, hi, k, [max(k, 4)], mode=mode)
            for i in range(3):
                ids = narrow["ids"][i]
                n = int((ids != SENTINEL).sum())
                assert n <= min(k, nvalid[i]) and (ids[n:] == SENTINEL).all()
                a = attrs[ids[:n].astype(np.int64)]
                assert ((a >= lo[i]) & (a <= hi[i])).all()
                keys = list(zip(narrow["d2"][i][:n].tolist(), ids[:n].tolist()))
                assert keys == sorted(keys) and len(set(ids[:n].tolist())) == n
                # what the narrow search returns can never beat the exact answer
                assert (narrow["d2"][i][:n].astype(np.float64) >= gt_d2[i][:n]).all()

    check()
