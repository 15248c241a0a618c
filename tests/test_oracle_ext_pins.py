"""Pins for the two filter extensions of the oracle: membership (subset / equality) predicates
and the distance-to-range penalty as the score's filter term in place of the violation count."""
import numpy as np
import pytest

from boa_synth import C2, SENTINEL, make_workload
from oracle.boa_oracle import OracleIndex
from tests.test_oracle_pins import _read_golden, _ring

I32, F32, SET = 0, 1, 2


def _index(attrs, types, n=None):
    attrs = np.asarray(attrs, dtype=np.int64).astype(np.uint32).view(np.int32) if not isinstance(attrs, np.ndarray) else attrs.astype(np.int32)
    n = attrs.shape[0]
    x = np.arange(n, dtype=np.float32)[:, None] * np.ones((1, 4), np.float32)
    g = ((np.arange(n)[:, None] + np.arange(1, 3)[None, :]) % n).astype(np.uint32)
    return OracleIndex(x, attrs, np.asarray(types, np.int32), g, entry=0)


def test_membership_predicate_cases():
    cells = [0b0000, 0b0001, 0b0110, 0b1111, -1]                 # -1: every tag
    ix = _index([[c] for c in cells], [SET])
    def phi(mask, mode, p):
        return ix.phi(np.array([mask], np.int32), np.array([mode], np.int32), p)
    # any-of (hi == 0): valid iff the point carries at least one wanted tag
    assert [phi(0b0110, 0, p) for p in range(5)] == [1, 1, 0, 0, 0]
    assert [phi(0b0001, 0, p) for p in range(5)] == [1, 0, 1, 0, 0]
    # all-of (hi != 0): valid iff it carries every wanted tag
    assert [phi(0b0110, 1, p) for p in range(5)] == [1, 1, 0, 0, 0]
    assert [phi(0b0111, 1, p) for p in range(5)] == [1, 1, 1, 0, 0]
    # an empty wish: nothing can have "one of nothing"; everything has "all of nothing"
    assert [phi(0, 0, p) for p in range(5)] == [1, 1, 1, 1, 1]
    assert [phi(0, 1, p) for p in range(5)] == [0, 0, 0, 0, 0]
    # equality on a categorical attribute: one-hot cells, a one-bit mask
    onehot = _index([[1 << c] for c in (0, 3, 3, 7, 31)], [SET])
    want3 = [onehot.phi(np.array([1 << 3], np.int32), np.array([0], np.int32), p) for p in range(5)]
    assert want3 == [1, 0, 0, 1, 1]
    top = [onehot.phi(np.array([-2 ** 31], np.int32), np.array([0], np.int32), p) for p in range(5)]
    assert top == [1, 1, 1, 1, 0]                                 # bit 31 works like any other


def test_membership_search_is_valid_and_full_width_is_exact():
    rng = np.random.default_rng(4)
    n = 400
    attrs = np.stack([rng.integers(0, 2 ** 12, n), rng.integers(0, 100, n)], 1).astype(np.int32)
    x = rng.standard_normal((n, 8)).astype(np.float32)
    g = ((np.arange(n)[:, None] + np.arange(1, 7)[None, :] * 53) % n).astype(np.uint32)
    ix = OracleIndex(x, attrs, np.array([SET, I32], np.int32), g, entry=0)
    q = rng.standard_normal((10, 8)).astype(np.float32)
    lo = np.stack([rng.integers(1, 2 ** 12, 10), np.full(10, 10)], 1).astype(np.int32)
    hi = np.stack([rng.integers(0, 2, 10), np.full(10, 80)], 1).astype(np.int32)
    r = ix.search(q, lo, hi, 5, [n], cap=(8, 10 ** 6))
    b_ids, b_d2, b_nv = ix.bruteforce(q, lo, hi, 5)
    assert (r["ids"] == b_ids).all()
    for i in range(10):
        have = attrs[:, 0] & lo[i, 0]
        ok = ((have != 0) if hi[i, 0] == 0 else (have == lo[i, 0])) & (attrs[:, 1] >= 10) & (attrs[:, 1] <= 80)
        assert b_nv[i] == ok.sum()
        assert all(ok[p] for p in r["ids"][i] if p != SENTINEL)


def test_range_penalty_hand_values_and_order():
    f = lambda v: np.array([v], np.float32).view(np.int32)[0]
    attrs = [[5, f(0.25), 0b01], [25, f(0.75), 0b10], [15, f(np.nan), 0b11], [-2 ** 31, f(2.0), 0]]
    ix = _index(attrs, [I32, F32, SET])
    lo = np.array([10, f(0.5), 0b10], np.int32)
    hi = np.array([20, f(1.0), 0], np.int32)
    one = np.ones(3, np.float32)
    assert ix.range_penalty(lo, hi, 0, one) == np.float32(5 + 0.25 + 1)
    assert ix.range_penalty(lo, hi, 1, one) == np.float32(5 + 0 + 0)
    assert np.isinf(ix.range_penalty(lo, hi, 2, one))                       # NaN cell: infinitely far
    assert ix.range_penalty(lo, hi, 3, one) == np.float32(2.0 ** 31 + 10 + 1.0 + 1)   # no int overflow
    w = np.array([0.5, 4.0, 10.0], np.float32)
    assert ix.range_penalty(lo, hi, 0, w) == np.float32(2.5 + 1.0 + 10.0)
    assert ix.range_penalty(lo, hi, 1, w) == np.float32(2.5)
    # zero exactly when the point is valid
    inside = _index([[12, f(0.6), 0b10]], [I32, F32, SET])
    assert inside.range_penalty(lo, hi, 0, w) == 0.0 and inside.phi(lo, hi, 0) == 0
    # the attributes are added in ascending order in fp32: 2^24 + 1 + 1 stays 2^24 that way
    big = _index([[0, 9, 9]], [I32, I32, I32])
    lo3 = np.array([2 ** 24, 10, 10], np.int32)
    hi3 = np.array([2 ** 25, 20, 20], np.int32)
    assert big.range_penalty(lo3, hi3, 0, one) == np.float32(2.0 ** 24)
    rev = _index([[9, 9, 0]], [I32, I32, I32])
    assert rev.range_penalty(lo3[::-1].copy(), hi3[::-1].copy(), 0, one) == np.float32(2.0 ** 24 + 2)


def test_penalty_equals_count_when_every_violation_is_one_unit_out():
    # the ring example: attribute 0 / 1, range [1, 1]: an invalid point is exactly 1 away, so
    # the penalty is the violation count and the finite-lambda hand traces must come out the same
    gold = {r[0]: [int(v) for v in r[1:]] for r in _read_golden("ring_trace_finite_lambda.txt")}
    ix = _ring()
    q = np.array([5.2], dtype=np.float32)
    one = np.array([1], dtype=np.int32)
    for lam, tag in ((2.0, "l2"), (0.5, "l05")):
        b = ix.beam(q, one, one, L=3, C=3, lam=lam, penalty_scales=[1.0])
        assert b.n_expand == len(gold[tag + "_expansions"]) and b.n_scored == len(gold[tag + "_scored"])
        assert [int(i) for i in b.pool()[0]] == gold[tag + "_final_pool"]
    # a scale of two is a lambda twice as large
    a = ix.beam(q, one, one, L=3, C=3, lam=1.0, penalty_scales=[2.0])
    b = ix.beam(q, one, one, L=3, C=3, lam=2.0)
    assert (a.pool()[0] == b.pool()[0]).all() and a.n_expand == b.n_expand


def test_penalty_search_relations():
    w = C2.scaled(5000, 40, name="c2_pen")
    d = make_workload(w, seed=8, device="cpu")
    ix = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    q, lo, hi = d["queries"], d["lo"], d["hi"]
    scales = np.array([1e-3, 5e-2], np.float32)
    for mode in ("restart", "resume"):
        r = ix.search(q, lo, hi, 10, [16, 64, 128], mode=mode, lam=50.0, penalty_scales=scales, dist_mode=1)
        for i in range(w.Q):
            got = r["ids"][i][r["ids"][i] != SENTINEL]
            assert all(ix.phi(lo[i], hi[i], p) == 0 for p in got)             # validity is decided by phi
            assert (np.diff(r["d2"][i][: len(got)]) >= 0).all()
    # the pool is ordered by d2 + lambda * penalty
    b = ix.beam(q[0], lo[0], hi[0], L=32, lam=50.0, penalty_scales=scales, dist_mode=1)
    ids, d2, phi, ex = b.pool()
    sc = [np.float32(np.float32(50.0) * ix.range_penalty(lo[0], hi[0], p, scales) + dd) for p, dd in zip(ids, d2)]
    assert all(sc[i] <= sc[i + 1] * (1 + 1e-6) for i in range(len(sc) - 1))
    # zero scales: the penalty vanishes, the walk is the unfiltered one (lambda = 0)
    a = ix.search(q, lo, hi, 10, [32], lam=7.0, penalty_scales=np.zeros(2, np.float32), dist_mode=1)
    z = ix.search(q, lo, hi, 10, [32], lam=0.0, dist_mode=1)
    assert (a["ids"] == z["ids"]).all() and (a["n_expand"] == z["n_expand"]).all()
    # full width: exact, whatever the penalty
    sub = OracleIndex(d["vectors"][:500], d["attrs"][:500], d["attr_types"],
                      ((np.arange(500)[:, None] + np.arange(1, 9)[None, :] * 31) % 500).astype(np.uint32), entry=0)
    r = sub.search(q[:6], lo[:6], hi[:6], 5, [500], lam=3.0, penalty_scales=scales, cap=(8, 10 ** 6))
    b_ids, _, _ = sub.bruteforce(q[:6], lo[:6], hi[:6], 5)
    assert (r["ids"] == b_ids).all()
