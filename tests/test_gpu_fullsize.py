"""The benchmark's own configuration at full size (1M points, 10,000 queries, resume mode,
schedule 16 -> 512): sampled queries against the oracle one by one, properties that hold
at any size on all of them, and the harness's brute-force ground truth against the
oracle's."""
import numpy as np
import pytest
import torch

from boa_synth import C2, SENTINEL, make_workload
from boa_synth.groundtruth import filtered_topk, recall_against
from tests.helpers import gpu_search, make_pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def full():
    d = make_workload(C2, seed=0)
    orc, gpu, g = make_pair(d)
    return C2, d, orc, gpu, g


def test_full_size_bench_configuration(full):
    w, d, orc, gpu, g = full
    widths, eps = [16, 512], 0.03
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
    assert r["phase_active"][0] == Q and r["phase_active"][1] == int((r["final_L"] == 512).sum())
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
    gpu.close()
