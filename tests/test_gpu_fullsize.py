"""The benchmark configurations at full size: sampled queries against the oracle one by
one, properties that hold at any size on all of them, and the harness's brute-force ground
truth against the oracle's.  The 10M-point workload takes a few minutes to build the first
time on a machine (its arrays are then kept on disk)."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C4, C5, SENTINEL, make_workload
from boa_synth.groundtruth import filtered_topk, recall_against
from tests.helpers import gpu_search, make_pair

pytestmark = pytest.mark.gpu


def _check_properties(w, d, r, widths, Q):
    """Validity, order, uniqueness, padding and phase bookkeeping on every query of a run."""
    a = d["attrs"]
    ids, d2 = r["ids"], r["d2"]
    lo, hi = d["lo"][:Q], d["hi"][:Q]
    found = ids != SENTINEL
    assert (np.isinf(d2) == ~found).all()
    assert (found[:, :-1] >= found[:, 1:]).all()                         # padding only at the tail
    safe = np.where(found, ids, 0).astype(np.int64)
    for j, ty in enumerate(d["attr_types"]):
        col = a[:, j][safe]
        if ty == 1:
            ok = (col.view(np.float32) >= lo[:, j:j + 1].view(np.float32)) & \
                 (col.view(np.float32) <= hi[:, j:j + 1].view(np.float32))
        else:
            ok = (col >= lo[:, j:j + 1]) & (col <= hi[:, j:j + 1])
        assert ok[found].all()
    both = found[:, :-1] & found[:, 1:]
    assert (d2[:, :-1][both] <= d2[:, 1:][both]).all()
    srt = np.sort(np.where(found, ids, np.arange(w.k, dtype=np.uint32)[None, :] + 0xF0000000), axis=1)
    assert (srt[:, :-1] != srt[:, 1:]).all()
    assert set(np.unique(r["final_L"]).tolist()) <= set(widths)
    assert r["phase_active"][0] == Q
    for p in range(1, len(widths)):
        assert r["phase_active"][p] == int((r["final_L"] >= widths[p]).sum())


def _assert_sample_bit_parity(o, r, sample):
    assert (o["ids"] == r["ids"][sample]).all()
    assert (o["d2"].view(np.uint32) == r["d2"][sample].view(np.uint32)).all()
    assert (o["final_L"] == r["final_L"][sample]).all()
    assert (o["n_expand"] == r["n_expand"][sample]).all()
    assert (o["flags"] == r["flags"][sample]).all()
    assert (r["n_scored"][sample] >= o["n_scored"]).all()


@pytest.fixture(scope="module")
def full():
    d = make_workload(C2, seed=0)
    orc, gpu, g = make_pair(d)
    return C2, d, orc, gpu, g


@pytest.mark.parametrize("which", ["operating point", "wide"])
def test_full_size_bench_configuration(full, which):
    import bench
    w, d, orc, gpu, g = full
    op = bench.OPERATING["c2"] if which == "operating point" else bench.WIDE["c2"]
    widths, eps = list(op["schedule"]), op["eps"]
    r = gpu_search(gpu, g, w.k, widths, mode="resume", eps=eps)
    assert gpu.device_status() == 0
    Q = w.Q
    # --- sampled queries, element by element
    sample = np.random.default_rng(5).choice(Q, size=160, replace=False)
    o = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                   mode="resume", dist_mode=1)
    assert (o["ids"] == r["ids"][sample]).all()
    assert (o["d2"].view(np.uint32) == r["d2"][sample].view(np.uint32)).all()
    assert (o["final_L"] == r["final_L"][sample]).all()
    assert (o["n_expand"] == r["n_expand"][sample]).all()
    assert (r["n_scored"][sample] >= o["n_scored"]).all()
    assert len(set(o["final_L"].tolist())) == 2            # both outcomes of the confidence test
    # --- properties on every query: validity, order, uniqueness, padding
    a = d["attrs"]
    ids, d2 = r["ids"], r["d2"]
    found = ids != SENTINEL
    assert (np.isinf(d2) == ~found).all()
    assert (found[:, :-1] >= found[:, 1:]).all()                         # padding only at the tail
    safe = np.where(found, ids, 0).astype(np.int64)
    for j in range(w.m):
        col = a[:, j][safe]
        ok = (col >= d["lo"][:, j:j + 1]) & (col <= d["hi"][:, j:j + 1])
        assert ok[found].all()
    both = found[:, :-1] & found[:, 1:]
    assert (d2[:, :-1][both] <= d2[:, 1:][both]).all()
    srt = np.sort(np.where(found, ids, np.arange(w.k, dtype=np.uint32)[None, :] + 0xF0000000), axis=1)
    assert (srt[:, :-1] != srt[:, 1:]).all()
    assert set(np.unique(r["final_L"]).tolist()) <= set(widths)
    assert r["phase_active"][0] == Q and r["phase_active"][1] == int((r["final_L"] == widths[-1]).sum())
    # --- recall: harness ground truth vs the oracle's brute force, and the >= 0.95 bar
    gt_ids, gt_d2, gt_nv = filtered_topk(g["vectors"], g["attrs"], d["attr_types"], g["queries"],
                                         g["lo"], g["hi"], w.k)
    gt_d2, gt_nv = gt_d2.cpu().numpy(), gt_nv.cpu().numpy()
    few = sample[:12]
    b_ids, b_d2, b_nv = orc.bruteforce(d["queries"][few], d["lo"][few], d["hi"][few], w.k)
    assert (b_nv == gt_nv[few]).all()
    assert (b_d2 == gt_d2[few]).all()                                    # integer data: exact
    rec = recall_against(ids, d2, gt_d2, gt_nv, w.k)
    rec_o = recall_against(o["ids"], o["d2"], gt_d2[sample], gt_nv[sample], w.k)
    assert abs(np.nanmean(rec[sample]) - np.nanmean(rec_o)) <= 0.001
    assert np.nanmean(rec) >= 0.95


def test_full_size_boa_plus_and_restart_agree_with_their_definitions(full):
    w, d, orc, gpu, g = full
    a = gpu_search(gpu, g, w.k, [16, 512], mode="resume", eps=0.03)
    b = gpu_search(gpu, g, w.k, [16, 512], mode="resume", eps=0.03, plus_k=10)
    assert (a["ids"] == b["ids"]).all() and (a["d2"].view(np.uint32) == b["d2"].view(np.uint32)).all()
    assert (a["final_L"] == b["final_L"]).all() and (a["n_expand"] == b["n_expand"]).all()
    sample = np.arange(0, w.Q, 97)[:60]
    r = gpu_search(gpu, g, w.k, [16, 64, 256], mode="restart", eps=0.05, sel=torch.from_numpy(sample).to("cuda:0"))
    o = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, [16, 64, 256], eps=0.05,
                   mode="restart", dist_mode=1)
    assert (o["ids"] == r["ids"]).all() and (o["n_expand"] == r["n_expand"]).all()


def test_full_size_float_workload_c3():
    """The 1M x 96-d unit-norm float workload at full size: sampled queries bit for bit
    against the oracle's fixed-order fp32 distances, within the stated tolerance of its
    double-precision distances, and the recall bar."""
    from boa_synth import C3
    w = C3
    d = make_workload(w, seed=0)
    orc, gpu, g = make_pair(d)
    widths, eps = [16, 512], 0.03
    r = gpu_search(gpu, g, w.k, widths, mode="resume", eps=eps)
    assert gpu.device_status() == 0
    sample = np.random.default_rng(6).choice(w.Q, size=96, replace=False)
    o = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                   mode="resume", dist_mode=1)
    assert (o["ids"] == r["ids"][sample]).all()
    assert (o["d2"].view(np.uint32) == r["d2"][sample].view(np.uint32)).all()
    assert (o["final_L"] == r["final_L"][sample]).all() and (o["n_expand"] == r["n_expand"][sample]).all()
    # double accumulation: same ids except at near-ties below 1e-5 relative, distances within 1e-5
    o64 = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                     mode="resume", dist_mode=0)
    same_path = (o64["final_L"] == r["final_L"][sample]) & (o64["n_expand"] == r["n_expand"][sample])
    assert same_path.mean() > 0.9
    for t in np.nonzero(same_path)[0]:
        gi, oi = r["ids"][sample[t]], o64["ids"][t]
        gd, od = r["d2"][sample[t]], o64["d2"][t]
        fin = np.isfinite(od)
        assert (np.isfinite(gd) == fin).all()
        np.testing.assert_allclose(gd[fin], od[fin], rtol=1e-5)
        for c in np.nonzero(gi != oi)[0]:                      # a swap is allowed only at a near-tie
            assert abs(float(gd[c]) - float(od[c])) <= 1e-5 * max(float(od[c]), 1e-30)
    gt_ids, gt_d2, gt_nv = filtered_topk(g["vectors"], g["attrs"], d["attr_types"], g["queries"],
                                         g["lo"], g["hi"], w.k)
    rec = recall_against(r["ids"], r["d2"], gt_d2.cpu().numpy(), gt_nv.cpu().numpy(), w.k)
    assert np.nanmean(rec) >= 0.95
    # the benchmark's operating point on this workload
    import bench
    op = bench.OPERATING["c3"]
    r2 = gpu_search(gpu, g, w.k, op["schedule"], mode="resume", eps=op["eps"])
    o2 = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, op["schedule"], eps=op["eps"],
                    mode="resume", dist_mode=1)
    _assert_sample_bit_parity(o2, r2, sample)
    _check_properties(w, d, r2, op["schedule"], w.Q)
    assert np.nanmean(recall_against(r2["ids"], r2["d2"], gt_d2.cpu().numpy(), gt_nv.cpu().numpy(), w.k)) >= 0.95
    gpu.close()


def test_full_size_scale_workload_c4():
    """10M uint8 points of 128 dimensions, degree 64, 10,000 queries: node ids of 24 bits
    (wide tags in the table of scored ids), a 2.56 GB graph, record offsets beyond 2^32."""
    w = C4
    d = make_workload(w, seed=0)
    assert d["vectors"].dtype == np.uint8 and d["graph"].shape == (10_000_000, 64)
    orc, gpu, g = make_pair(d)
    assert orc.entry == gpu.entry
    widths, eps = [32, 512], 0.05
    r = gpu_search(gpu, g, w.k, widths, mode="resume", eps=eps)
    assert gpu.device_status() == 0
    sample = np.random.default_rng(7).choice(w.Q, size=100, replace=False)
    o = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                   mode="resume", dist_mode=1)
    _assert_sample_bit_parity(o, r, sample)
    o64 = orc.search(d["queries"][sample[:40]], d["lo"][sample[:40]], d["hi"][sample[:40]], w.k, widths, eps=eps,
                     mode="resume", dist_mode=0)
    assert (o64["ids"] == o["ids"][:40]).all() and (o64["d2"] == o["d2"][:40]).all()   # integer data: exact
    assert (o["final_L"] == 512).any() and (np.array(sample) >= 0).all()
    ids_far = r["ids"][r["ids"] != SENTINEL]
    assert ids_far.max() >= (1 << 23)                                   # answers from the upper half of the id range
    _check_properties(w, d, r, widths, w.Q)
    gt_ids, gt_d2, gt_nv = filtered_topk(g["vectors"], g["attrs"], d["attr_types"], g["queries"],
                                         g["lo"], g["hi"], w.k)
    gt_d2, gt_nv = gt_d2.cpu().numpy(), gt_nv.cpu().numpy()
    few = sample[:6]
    b_ids, b_d2, b_nv = orc.bruteforce(d["queries"][few], d["lo"][few], d["hi"][few], w.k)
    assert (b_nv == gt_nv[few]).all() and (b_d2 == gt_d2[few]).all()
    rec = recall_against(r["ids"], r["d2"], gt_d2, gt_nv, w.k)
    rec_o = recall_against(o["ids"], o["d2"], gt_d2[sample], gt_nv[sample], w.k)
    assert abs(np.nanmean(rec[sample]) - np.nanmean(rec_o)) <= 0.001
    assert np.nanmean(rec) >= 0.95
    # the benchmark's operating point on this workload
    import bench
    op = bench.OPERATING["c4"]
    r2 = gpu_search(gpu, g, w.k, op["schedule"], mode="resume", eps=op["eps"])
    o2 = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, op["schedule"], eps=op["eps"],
                    mode="resume", dist_mode=1)
    _assert_sample_bit_parity(o2, r2, sample)
    _check_properties(w, d, r2, op["schedule"], w.Q)
    assert np.nanmean(recall_against(r2["ids"], r2["d2"], gt_d2, gt_nv, w.k)) >= 0.95
    # restart mode and the overlapped schedule on the same index
    sel = torch.from_numpy(sample[:32].astype(np.int64)).to("cuda:0")
    rr = gpu_search(gpu, g, w.k, [32, 128], mode="restart", eps=eps, sel=sel)
    oo = orc.search(d["queries"][sample[:32]], d["lo"][sample[:32]], d["hi"][sample[:32]], w.k, [32, 128], eps=eps,
                    mode="restart", dist_mode=1)
    assert (oo["ids"] == rr["ids"]).all() and (oo["n_expand"] == rr["n_expand"]).all()
    b = gpu_search(gpu, g, w.k, widths, mode="resume", eps=eps, plus_k=10)
    assert (b["ids"] == r["ids"]).all() and (b["d2"].view(np.uint32) == r["d2"].view(np.uint32)).all()
    gpu.close()


def test_full_size_long_rows_c5():
    """1M points of 960 float dimensions (3,840-byte rows, the generic row loop), four
    attributes of mixed types: the first 4,000 queries of the 100,000-query batch, sampled
    ones against the oracle in both distance modes; the fixed beamwidth of 500 too."""
    w = C5
    Q = 4000
    d = make_workload(w, seed=0)
    orc, gpu, g = make_pair(d)
    sl = slice(0, Q)
    widths, eps = [16, 512], 0.03
    r = gpu_search(gpu, g, w.k, widths, mode="resume", eps=eps, sel=sl)
    assert gpu.device_status() == 0
    sample = np.random.default_rng(8).choice(Q, size=48, replace=False)
    o = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                   mode="resume", dist_mode=1)
    _assert_sample_bit_parity(o, r, sample)
    assert len(set(o["final_L"].tolist())) == 2
    o64 = orc.search(d["queries"][sample], d["lo"][sample], d["hi"][sample], w.k, widths, eps=eps,
                     mode="resume", dist_mode=0)
    same_path = (o64["final_L"] == r["final_L"][sample]) & (o64["n_expand"] == r["n_expand"][sample])
    assert same_path.mean() > 0.8
    for t in np.nonzero(same_path)[0]:
        gi, oi = r["ids"][sample[t]], o64["ids"][t]
        gd, od = r["d2"][sample[t]], o64["d2"][t]
        fin = np.isfinite(od)
        assert (np.isfinite(gd) == fin).all()
        np.testing.assert_allclose(gd[fin], od[fin], rtol=1e-5)
        for c in np.nonzero(gi != oi)[0]:                      # a swap is allowed only at a near-tie
            assert abs(float(gd[c]) - float(od[c])) <= 1e-5 * max(float(od[c]), 1e-30)
    _check_properties(w, d, r, widths, Q)
    gt_ids, gt_d2, gt_nv = filtered_topk(g["vectors"], g["attrs"], d["attr_types"], g["queries"][sl],
                                         g["lo"][sl], g["hi"][sl], w.k)
    gt_d2, gt_nv = gt_d2.cpu().numpy(), gt_nv.cpu().numpy()
    rec = recall_against(r["ids"], r["d2"], gt_d2, gt_nv, w.k)
    rec_o = recall_against(o["ids"], o["d2"], gt_d2[sample], gt_nv[sample], w.k)
    assert abs(np.nanmean(rec[sample]) - np.nanmean(rec_o)) <= 0.001
    # the configuration's comparison point: beamwidth 500 for every query
    f = gpu_search(gpu, g, w.k, [500], mode="restart", sel=sl)
    of = orc.search(d["queries"][sample[:16]], d["lo"][sample[:16]], d["hi"][sample[:16]], w.k, [500], dist_mode=1)
    assert (of["ids"] == f["ids"][sample[:16]]).all() and (of["n_expand"] == f["n_expand"][sample[:16]]).all()
    rec_f = recall_against(f["ids"], f["d2"], gt_d2, gt_nv, w.k)
    assert np.nanmean(rec_f) > np.nanmean(rec)                           # the wide fixed beam finds more
    gpu.close()


def test_more_than_2_pow_25_points():
    """Node ids of 26 bits: the table of scored ids has to double its size until 16-bit tags
    identify an id again, and keys carry ids beyond 2^25.  Tiny vectors (4 floats) and a random
    degree-4 graph keep the 33.5M-point index small; queries are exact copies of high-numbered
    points, so the answers come from the top of the id range."""
    N, D, R, Q, k = (1 << 25) + 8, 4, 4, 64, 5
    rng = np.random.default_rng(3)
    x = rng.integers(0, 64, size=(N, D)).astype(np.float32)
    x[N - 40:] = np.array([200, 210, 220, 230], np.float32) + rng.integers(0, 3, size=(40, D))   # a far-off family
    attrs = rng.integers(0, 100, size=(N, 1)).astype(np.int32)
    attrs[N - 40:] = 50
    graph = rng.integers(0, N, size=(N, R)).astype(np.uint32)
    graph[:, 0] = (np.arange(N, dtype=np.uint32) + np.uint32(1)) % np.uint32(N)      # a ring keeps it connected
    graph[0, 1] = N - 1                                                               # reach the top of the range at once
    graph[N - 40:, 1] = np.arange(N - 41, N - 1, dtype=np.uint32)                     # and walk down from there
    src = N - 1 - rng.integers(0, 32, size=Q)
    q = x[src].copy()
    lo = np.full((Q, 1), 0, np.int32)
    hi = np.full((Q, 1), 70, np.int32)
    d = dict(vectors=x, attrs=attrs, attr_types=np.zeros(1, np.int32), graph=graph, queries=q, lo=lo, hi=hi)
    orc, gpu, g = make_pair(d, entry=0)
    for mode, widths in (("resume", [16, 64, 256]), ("restart", [16, 128])):
        o = orc.search(q, lo, hi, k, widths, eps=0.1, mode=mode, dist_mode=1)
        r = gpu_search(gpu, g, k, widths, mode=mode, eps=0.1)
        assert (o["ids"] == r["ids"]).all() and (o["d2"].view(np.uint32) == r["d2"].view(np.uint32)).all()
        assert (o["final_L"] == r["final_L"]).all() and (o["n_expand"] == r["n_expand"]).all()
        assert (r["n_scored"] >= o["n_scored"]).all()
    found = r["ids"][r["ids"] != SENTINEL]
    assert found.size and found.max() >= (1 << 25)
    assert gpu.device_status() == 0
    gpu.close()
