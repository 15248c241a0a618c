"""Cosine metric: CUDA library against the oracle through the C interface."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C3, C4, SENTINEL, make_workload
from boa_synth.pq import train_pq
from oracle.boa_oracle import OracleIndex
from tests.helpers import assert_bit_parity, gpu_search, to_gpu

pytestmark = pytest.mark.gpu


def _pair(w, seed, scale=True):
    from paper_2609_16175_b200 import BoaIndex
    d = make_workload(w, seed=seed)
    if scale:                                   # rows and queries of very different lengths
        rng = np.random.default_rng(seed)
        d["vectors"] = (d["vectors"] * rng.uniform(0.1, 9.0, size=(w.N, 1))).astype(np.float32)
        d["queries"] = (d["queries"] * rng.uniform(0.1, 9.0, size=(w.Q, 1))).astype(np.float32)
        d["vectors"][7] = 0.0                   # a zero row: distance 0.5 to everything
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    orc.set_metric("cosine")
    g = to_gpu(d)
    gpu = BoaIndex(g["vectors"], g["attrs"], d["attr_types"].tolist(), g["graph"])
    gpu.set_metric("cosine")
    assert orc.entry == gpu.entry
    return d, orc, gpu, g


@pytest.mark.parametrize("which", ["c3", "c2"])
def test_cosine_search_matches_oracle(which):
    w = C3.scaled(30_000, 150, name="c3_cos") if which == "c3" else C2.scaled(30_000, 150, name="c2_cos")
    d, orc, gpu, g = _pair(w, seed=31)
    for mode in ("restart", "resume"):
        for widths, eps in (([16, 64, 256], 0.1), ([24], 0.05), ([16, 512], 0.3)):
            o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1)
            r = gpu_search(gpu, g, w.k, widths, mode=mode, eps=eps)
            assert_bit_parity(o, r, f"cosine {which}/{mode}/{widths}")
    assert len(set(o["final_L"].tolist())) == 2                      # Eq. 3 decided both ways
    # the definition in double: same ids except at near-ties, distances within 1e-5
    o64 = orc.search(d["queries"], d["lo"], d["hi"], w.k, [64], dist_mode=0)
    r = gpu_search(gpu, g, w.k, [64])
    same = (o64["n_expand"] == r["n_expand"])
    assert same.mean() > 0.85
    for t in np.nonzero(same)[0]:
        fin = np.isfinite(o64["d2"][t])
        np.testing.assert_allclose(r["d2"][t][fin], o64["d2"][t][fin], rtol=1e-5, atol=1e-7)
        for c in np.nonzero(r["ids"][t] != o64["ids"][t])[0]:
            assert abs(float(r["d2"][t][c]) - float(o64["d2"][t][c])) <= 1e-5 * max(float(o64["d2"][t][c]), 1e-6)
    assert (r["d2"][np.isfinite(r["d2"])] <= 2.0 + 1e-6).all() and (r["d2"] >= 0).all()
    # BOA+ and the other options ride on the same kernels
    a = gpu_search(gpu, g, w.k, [16, 64, 256], mode="resume", eps=0.1)
    b = gpu_search(gpu, g, w.k, [16, 64, 256], mode="resume", eps=0.1, plus_k=3)
    assert (a["ids"] == b["ids"]).all() and (a["d2"].view(np.uint32) == b["d2"].view(np.uint32)).all()
    gpu.close()


def test_cosine_with_pq_and_errors():
    from paper_2609_16175_b200 import BoaError, BoaIndex
    w = C3.scaled(20_000, 100, name="c3_cos_pq")
    d, orc, gpu, g = _pair(w, seed=32)
    unit = d["vectors"].astype(np.float64)
    nrm = np.linalg.norm(unit, axis=1, keepdims=True)
    unit = (unit / np.where(nrm > 0, nrm, 1.0)).astype(np.float32)
    piv, codes = train_pq(unit, M=16, K=64, iters=4, seed=5)
    orc.attach_pq(piv, codes)
    gpu.attach_pq(torch.from_numpy(piv).to("cuda:0"), torch.from_numpy(codes).to("cuda:0"))
    for mode in ("restart", "resume"):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 128], eps=0.1, mode=mode, dist_mode=1, pq=True)
        r = gpu_search(gpu, g, w.k, [16, 128], mode=mode, eps=0.1, pq=True)
        assert_bit_parity(o, r, f"cosine pq {mode}")
    with pytest.raises(BoaError):
        gpu.set_metric("l2")                                         # one way only
    gpu.set_metric("cosine")                                         # asking again is fine
    q = g["queries"][:8].contiguous()
    oi = torch.zeros((8, w.k), dtype=torch.int32, device="cuda:0")
    od = torch.zeros((8, w.k), dtype=torch.float32, device="cuda:0")
    with pytest.raises(BoaError):
        gpu.search_noalloc(q, g["lo"][:8].contiguous(), g["hi"][:8].contiguous(), w.k, 16, 64, oi, od)
    gpu.close()
    w8 = C4.scaled(5_000, 10, name="c4_cos")
    d8 = make_workload(w8, seed=1)
    g8 = to_gpu(d8)
    ix8 = BoaIndex(g8["vectors"], g8["attrs"], d8["attr_types"].tolist(), g8["graph"])
    with pytest.raises(BoaError):
        ix8.set_metric("cosine")                                     # byte vectors: Euclidean only
    ix8.close()
