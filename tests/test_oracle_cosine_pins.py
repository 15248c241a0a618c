"""Pins for the oracle's cosine metric (Definition 1 allows it; the paper itself uses the
Euclidean norm): hand values, plain numpy, invariance under rescaling, the identity with the
Euclidean search on unit-length data, the full-width beam, and Eq. 3 on cosine distances."""
import math

import numpy as np
import pytest

from boa_synth import C3, SENTINEL, make_workload
from oracle.boa_oracle import OracleIndex

FULL_LO, FULL_HI = np.iinfo(np.int32).min, np.iinfo(np.int32).max


def _tiny(x):
    n = x.shape[0]
    g = ((np.arange(n)[:, None] + np.arange(1, 3)[None, :]) % n).astype(np.uint32)
    ix = OracleIndex(x.astype(np.float32), np.zeros((n, 1), np.int32), np.zeros(1, np.int32), g, entry=0)
    ix.set_metric("cosine")
    return ix


def test_hand_values():
    x = np.array([[1, 0], [0, 2], [5, 5], [-1, -1], [0, 0], [3, 4]], dtype=np.float32)
    ix = _tiny(x)
    q = np.array([1, 1], dtype=np.float32)
    want = [1 - 1 / math.sqrt(2), 1 - 1 / math.sqrt(2), 0.0, 2.0, 0.5, 1 - 7 / (5 * math.sqrt(2))]
    for mode in (0, 1):
        for p, w in enumerate(want):
            assert abs(float(ix.cos_dist(q, p, mode)) - w) <= 2e-7, (mode, p)
    assert abs(float(ix.cos_dist(np.array([3, 0], np.float32), 1, 0)) - 1.0) <= 1e-7      # orthogonal
    # positive rescaling of either vector changes nothing
    assert ix.cos_dist(q * 7.5, 5, 0) == ix.cos_dist(q, 5, 0)


@pytest.fixture(scope="module")
def small():
    w = C3.scaled(4000, 40, name="c3_cos")
    d = make_workload(w, seed=21, device="cpu")
    rng = np.random.default_rng(1)
    x = (d["vectors"] * rng.uniform(0.2, 5.0, size=(w.N, 1))).astype(np.float32)      # not unit length any more
    q = (d["queries"] * rng.uniform(0.2, 5.0, size=(w.Q, 1))).astype(np.float32)
    ix = OracleIndex(x, d["attrs"], d["attr_types"], d["graph"])
    ix.set_metric("cosine")
    return w, d, x, q, ix


def test_matches_numpy_definition(small):
    w, d, x, q, ix = small
    xd, qd = x.astype(np.float64), q.astype(np.float64)
    for i in (0, 7, 33):
        cos = (xd @ qd[i]) / (np.linalg.norm(xd, axis=1) * np.linalg.norm(qd[i]))
        for p in (0, 5, 1234, 3999):
            assert abs(float(ix.cos_dist(q[i], p, 0)) - (1 - cos[p])) <= 1e-6
            assert abs(float(ix.cos_dist(q[i], p, 1)) - (1 - cos[p])) <= 1e-5 * max(1 - cos[p], 1e-3)
    b_ids, b_d, b_nv = ix.bruteforce(q[:6], d["lo"][:6], d["hi"][:6], 5)
    for i in range(6):
        cos = (xd @ qd[i]) / (np.linalg.norm(xd, axis=1) * np.linalg.norm(qd[i]))
        ok = np.ones(w.N, bool)
        for j, t in enumerate(d["attr_types"]):
            col = d["attrs"][:, j].view(np.float32) if t == 1 else d["attrs"][:, j]
            l = d["lo"][i, j:j + 1].view(np.float32)[0] if t == 1 else d["lo"][i, j]
            h = d["hi"][i, j:j + 1].view(np.float32)[0] if t == 1 else d["hi"][i, j]
            ok &= (col >= l) & (col <= h)
        cand = np.nonzero(ok)[0]
        order = cand[np.argsort(1 - cos[cand], kind="stable")][:5]
        n = min(5, len(cand))
        assert (b_ids[i][:n] == order[:n]).all()


def test_equals_euclidean_search_on_unit_vectors(small):
    """Cosine search == Euclidean search over the unit-length copies (keys differ by the exact
    factor one half), and positive rescaling of the data does not change it."""
    w, d, x, q, ix = small
    from oracle.boa_oracle import lib, _p
    xu = np.empty_like(x)
    qu = np.empty_like(q)
    for i in range(w.N):
        lib().orc_unit_f32(_p(x[i]), w.D, _p(xu[i]))
    for i in range(w.Q):
        lib().orc_unit_f32(_p(q[i]), w.D, _p(qu[i]))
    np.testing.assert_allclose(np.linalg.norm(xu.astype(np.float64), axis=1), 1.0, atol=1e-6)
    l2 = OracleIndex(xu, d["attrs"], d["attr_types"], d["graph"], entry=ix.entry)
    for L in (16, 64):
        a = ix.search(q, d["lo"], d["hi"], 10, [L], dist_mode=1)
        b = l2.search(qu, d["lo"], d["hi"], 10, [L], dist_mode=1)
        assert (a["ids"] == b["ids"]).all() and (a["n_expand"] == b["n_expand"]).all()
        fin = np.isfinite(a["d2"])
        assert (a["d2"][fin] == np.float32(0.5) * b["d2"][fin]).all()
    scaled = OracleIndex((x * np.float32(4.0)).astype(np.float32), d["attrs"], d["attr_types"], d["graph"],
                         entry=ix.entry)
    scaled.set_metric("cosine")
    a = ix.search(q, d["lo"], d["hi"], 10, [32], dist_mode=0)
    c = scaled.search(q * np.float32(0.25), d["lo"], d["hi"], 10, [32], dist_mode=0)
    assert (a["ids"] == c["ids"]).all()


def test_full_width_beam_is_exact_and_eq3_reads_cosine_distances(small):
    w, d, x, q, ix = small
    n = 600
    sub = OracleIndex(x[:n], d["attrs"][:n], d["attr_types"],
                      ((np.arange(n)[:, None] + np.arange(1, 9)[None, :] * 37) % n).astype(np.uint32), entry=0)
    sub.set_metric("cosine")
    r = sub.search(q[:8], d["lo"][:8], d["hi"][:8], 5, [n], dist_mode=0, cap=(8, 10 ** 6))
    b_ids, b_d, b_nv = sub.bruteforce(q[:8], d["lo"][:8], d["hi"][:8], 5)
    assert (r["ids"] == b_ids).all() and (r["n_expand"] == n).all()
    seen = set()
    for i in range(w.Q):
        b = ix.beam(q[i], d["lo"][i], d["hi"][i], L=24, dist_mode=0)
        ids, c, phi, ex = b.pool()
        v = c[:24][phi[:24] == 0].astype(np.float64)
        for eps in (0.05, 0.2, 0.5):
            if len(v) <= 10:
                assert b.uncertain(10, eps)
                continue
            gamma = (v[-1] - v[9]) / v[-1] if v[-1] > 0 else 0.0
            if abs(gamma - eps) > 1e-4:
                assert b.uncertain(10, eps) == (gamma > eps)
                seen.add(gamma > eps)
    assert seen == {True, False}
