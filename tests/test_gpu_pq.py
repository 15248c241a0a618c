"""Product-quantised traversal with exact final ranking: CUDA library against the oracle,
bit for bit (fixed-order fp32 table, look-up sums and exact distances), through the C
interface."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C3, C4, C5, SENTINEL, clean_rows, exact_knn_graph, make_workload
from boa_synth.pq import train_pq
from tests.helpers import assert_bit_parity, gpu_search, make_pair

pytestmark = pytest.mark.gpu

CASES = {
    #        workload                                M   K    queries
    "c2": (C2.scaled(40_000, 160, name="c2_pq"),     16, 256, 160),
    "c3": (C3.scaled(30_000, 120, name="c3_pq"),     16, 128, 120),     # 6 dims per subspace: scalar table build
    "c4": (C4.scaled(50_000, 120, name="c4_pq"),     32, 256, 120),     # uint8 rows, degree 64
    "c5": (C5.scaled(8_000, 60, name="c5_pq"),       48, 64,  60),      # 960 dims, 20 per subspace
}
_cache = {}


def _get(name):
    if name not in _cache:
        w, M, K, nq = CASES[name]
        d = make_workload(w, seed=2)
        piv, codes = train_pq(d["vectors"], M=M, K=K, iters=4, seed=3)
        orc, gpu, g = make_pair(d)
        orc.attach_pq(piv, codes)
        gpu.attach_pq(torch.from_numpy(piv).to("cuda:0"), torch.from_numpy(codes).to("cuda:0"))
        _cache[name] = (w, d, orc, gpu, g)
    return _cache[name]


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
@pytest.mark.parametrize("mode", ["restart", "resume"])
def test_pq_search_matches_oracle_bit_for_bit(name, mode):
    w, d, orc, gpu, g = _get(name)
    for widths, eps in (([w.L0, 64, 256], 0.05), ([w.L0, 512], 0.02), ([40], 0.05)):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1, pq=True)
        r = gpu_search(gpu, g, w.k, widths, mode=mode, eps=eps, pq=True)
        assert_bit_parity(o, r, f"pq {name}/{mode}/{widths}")
        assert gpu.device_status() == 0
    assert len(set(o["final_L"].tolist())) >= 1 and (r["ids"] != SENTINEL).any()
    # rows fetched for the final ranking: at most the beam of every phase run, at least the answers
    rr = gpu.rerank_counts().cpu().numpy()
    assert (rr >= (r["ids"] != SENTINEL).sum(1)).all() and (rr <= 40).all()


def test_pq_differs_from_exact_search_and_switches_back():
    w, d, orc, gpu, g = _get("c2")
    a = gpu_search(gpu, g, w.k, [16, 64], pq=True)
    b = gpu_search(gpu, g, w.k, [16, 64], pq=False)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 64], dist_mode=1)
    assert_bit_parity(o, b, "exact after pq")
    assert (a["n_expand"] != b["n_expand"]).any()             # a lossy codebook walks differently


def test_pq_with_boa_plus_finite_lambda_and_k_limits():
    from paper_2609_16175_b200 import BoaError
    w, d, orc, gpu, g = _get("c2")
    widths = [16, 64, 256]
    a = gpu_search(gpu, g, w.k, widths, mode="resume", eps=0.05, pq=True)
    for plus_k in (2, 5):
        b = gpu_search(gpu, g, w.k, widths, mode="resume", eps=0.05, pq=True, plus_k=plus_k)
        for key in ("ids", "final_L", "n_expand"):
            assert (a[key] == b[key]).all()
        assert (a["d2"].view(np.uint32) == b["d2"].view(np.uint32)).all()
    for lam in (0.0, 4000.0):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=0.05, mode="resume", dist_mode=1,
                       lam=lam, pq=True)
        r = gpu_search(gpu, g, w.k, widths, mode="resume", eps=0.05, lam=lam, pq=True)
        assert_bit_parity(o, r, f"pq lambda={lam}")
    for k in (1, 16, 32):
        o = orc.search(d["queries"][:40], d["lo"][:40], d["hi"][:40], k, [32, 100], dist_mode=1, pq=True)
        r = gpu_search(gpu, g, k, [32, 100], pq=True, sel=slice(0, 40))
        assert_bit_parity(o, r, f"pq k={k}")
    with pytest.raises(BoaError):                              # k beyond the final ranking's capacity
        gpu_search(gpu, g, 33, [40, 100], pq=True)
    with pytest.raises(BoaError):                              # one node per iteration only
        gpu_search(gpu, g, 10, [16, 64], pq=True, expand_w=2)
    gpu_search(gpu, g, 10, [16, 64], pq=False)


def test_lossless_codebook_on_gpu_equals_exact_search_and_errors():
    from paper_2609_16175_b200 import BoaError, BoaIndex
    rng = np.random.default_rng(0)
    N, D, M, Q = 2000, 32, 16, 64
    x = rng.integers(0, 8, size=(N, D)).astype(np.float32)
    a, b = np.meshgrid(np.arange(8), np.arange(8), indexing="ij")
    book = np.stack([a.ravel(), b.ravel()], 1).astype(np.float32)
    pivots = np.ascontiguousarray(np.repeat(book[None], M, 0))
    codes = np.ascontiguousarray((x[:, 0::2] * 8 + x[:, 1::2]).astype(np.uint8))
    attrs = rng.integers(0, 100, size=(N, 2)).astype(np.int32)
    lo = rng.integers(0, 40, size=(Q, 2)).astype(np.int32)
    hi = (lo + rng.integers(30, 70, size=(Q, 2))).astype(np.int32)
    q = rng.integers(0, 8, size=(Q, D)).astype(np.float32)
    gr = clean_rows(np.concatenate([exact_knn_graph(x, 10, device="cpu"),
                                    rng.integers(0, N, size=(N, 6)).astype(np.uint32)], 1))
    d = dict(vectors=x, attrs=attrs, attr_types=np.zeros(2, np.int32), graph=gr, queries=q, lo=lo, hi=hi)
    orc, gpu, g = make_pair(d)
    with pytest.raises(BoaError):
        gpu.set_param("pq", 1)                                  # nothing attached yet
    gpu.attach_pq(torch.from_numpy(pivots).to("cuda:0"), torch.from_numpy(codes).to("cuda:0"))
    orc.attach_pq(pivots, codes)
    for widths in ([12], [10, 40, 200]):
        e = gpu_search(gpu, g, 5, widths, mode="restart", eps=0.1)
        p = gpu_search(gpu, g, 5, widths, mode="restart", eps=0.1, pq=True)
        for key in ("ids", "final_L", "n_expand", "flags"):
            assert (e[key] == p[key]).all(), key
        assert (e["d2"] == p["d2"]).all()
        o = orc.search(q, lo, hi, 5, widths, eps=0.1, mode="restart", dist_mode=1, pq=True)
        assert_bit_parity(o, p, "lossless")
    bad = torch.zeros((24, 4, D // 24 if D % 24 == 0 else 1), dtype=torch.float32, device="cuda:0")
    with pytest.raises((BoaError, ValueError)):
        gpu.attach_pq(bad, torch.zeros((N, 24), dtype=torch.uint8, device="cuda:0"))
    gpu.close()
