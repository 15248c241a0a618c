"""CUDA library against the CPU oracle, element by element, through the C interface."""
import numpy as np
import pytest
import torch

from boa_synth import C1, C2, C3, C4, C5, SENTINEL, clean_rows, exact_knn_graph, make_workload
from oracle.boa_oracle import OracleIndex, default_widths
from tests.helpers import assert_bit_parity, gpu_search, make_pair

pytestmark = pytest.mark.gpu


def _workload(name):
    if name == "c1":
        return C1, make_workload(C1, seed=0)
    if name == "c2":
        w = C2.scaled(40_000, 300, name="c2_40k")
    elif name == "c3":
        w = C3.scaled(30_000, 200, name="c3_30k")
    elif name == "c4":
        w = C4.scaled(50_000, 200, name="c4_50k")
    elif name == "c5":
        w = C5.scaled(8_000, 100, name="c5_8k")
    return w, make_workload(w, seed=1)


_cache = {}


def _get(name):
    if name not in _cache:
        w, d = _workload(name)
        _cache[name] = (w, d) + make_pair(d)
    return _cache[name]


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
@pytest.mark.parametrize("mode", ["restart", "resume"])
def test_boa_matches_oracle_bit_for_bit(name, mode):
    w, d, orc, gpu, g = _get(name)
    assert orc.entry == gpu.entry
    widths = default_widths(w.L0, min(w.Lmax, 256))
    eps = {"c4": 0.2}.get(name, 0.05)      # chosen so that some queries stop early, some escalate
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1)
    r = gpu_search(gpu, g, w.k, widths, eps=eps, mode=mode)
    assert_bit_parity(o, r, f"{name}/{mode}")
    assert len(set(o["final_L"].tolist())) > 1 or name == "c1"


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
@pytest.mark.parametrize("mode", ["restart", "resume"])
def test_expansion_width_2_matches_oracle_bit_for_bit(name, mode):
    """Two nodes per iteration (an extension of Algorithm 2): same picks, same row order,
    same cap accounting as the oracle run at the same width."""
    w, d, orc, gpu, g = _get(name)
    widths = default_widths(w.L0, min(w.Lmax, 256))
    eps = {"c4": 0.2}.get(name, 0.05)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1,
                   expand_w=2)
    r = gpu_search(gpu, g, w.k, widths, eps=eps, mode=mode, expand_w=2)
    assert_bit_parity(o, r, f"{name}/{mode}/W=2")
    o1 = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1)
    assert (o1["n_expand"] != o["n_expand"]).any()        # the width does change the search


def test_expansion_width_2_cap_and_boa_plus():
    w, d, orc, gpu, g = _get("c2")
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 64], cap=(1, 3), dist_mode=1, expand_w=2)
    r = gpu_search(gpu, g, w.k, [16, 64], cap=(1, 3), expand_w=2)
    assert (o["flags"] & 1).any() and (o["n_expand"] % 2 == 1).any()
    assert_bit_parity(o, r, "cap/W=2")
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 128], mode="resume", dist_mode=1, expand_w=2)
    r = gpu_search(gpu, g, w.k, [16, 128], mode="resume", plus_k=3, expand_w=2)
    assert_bit_parity(o, r, "BOA+/W=2")


def test_stride_line_hand_trace_width_2_on_gpu():
    """The width-2 hand trace of tests/golden/stride_trace_width2.txt, on the GPU."""
    n = 16
    x = np.zeros((n, 4), dtype=np.float32)
    x[:, 0] = np.arange(n)
    graph = np.full((n, 4), SENTINEL, dtype=np.uint32)
    for i in range(n):
        for c, o in enumerate((-2, -1, 1, 2)):
            if 0 <= i + o < n:
                graph[i, c] = i + o
    d = dict(vectors=x, attrs=np.zeros((n, 1), np.int32), attr_types=np.zeros(1, np.int32), graph=graph,
             queries=np.array([[10.1, 0, 0, 0]], dtype=np.float32),
             lo=np.array([[0]], np.int32), hi=np.array([[0]], np.int32))
    orc, gpu, g = make_pair(d, entry=0)
    for w, n_exp in ((1, 7), (2, 12)):
        r = gpu_search(gpu, g, 2, [2], expand_w=w)
        assert r["ids"][0].tolist() == [10, 11]
        assert r["n_expand"][0] == n_exp and r["n_scored"][0] == 13
    gpu.close()


@pytest.mark.parametrize("name,lam", [("c2", 2000.0), ("c2", 0.0), ("c3", 0.05), ("c4", 30000.0),
                                      ("c5", 0.3)])
@pytest.mark.parametrize("mode", ["restart", "resume"])
def test_finite_lambda_matches_oracle_bit_for_bit(name, lam, mode):
    """Keys ordered by the score d2 + lambda*phi (the paper's stated form): same score bits
    (one fp32 fused multiply-add on both sides), same trajectories, same answers."""
    w, d, orc, gpu, g = _get(name)
    widths = default_widths(w.L0, min(w.Lmax, 256))
    eps = {"c4": 0.2}.get(name, 0.05)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1, lam=lam)
    r = gpu_search(gpu, g, w.k, widths, eps=eps, mode=mode, lam=lam)
    assert_bit_parity(o, r, f"{name}/{mode}/lambda={lam}")
    o_inf = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, mode=mode, dist_mode=1)
    assert (o_inf["n_scored"] != o["n_scored"]).any()        # the order does change the search
    # answers stay filter-valid and sorted
    for i in range(0, len(r["ids"]), 17):
        ids = r["ids"][i]
        n = int((ids != SENTINEL).sum())
        assert (ids[n:] == SENTINEL).all() and (np.diff(r["d2"][i][:n]) >= 0).all()
        a = d["attrs"][ids[:n].astype(np.int64)]
        for j, t in enumerate(d["attr_types"]):
            col = a[:, j].view(np.float32) if t == 1 else a[:, j]
            l = d["lo"][i, j:j + 1].view(np.float32)[0] if t == 1 else d["lo"][i, j]
            h = d["hi"][i, j:j + 1].view(np.float32)[0] if t == 1 else d["hi"][i, j]
            assert ((col >= l) & (col <= h)).all()


def test_finite_lambda_ring_hand_traces_width_2_and_boa_plus():
    x = np.zeros((8, 4), dtype=np.float32)
    x[:, 0] = np.arange(8)
    d = dict(vectors=x, attrs=(np.arange(8) % 2).astype(np.int32)[:, None],
             attr_types=np.zeros(1, np.int32),
             graph=np.stack([(np.arange(8) - 1) % 8, (np.arange(8) + 1) % 8], 1).astype(np.uint32),
             queries=np.array([[5.2, 0, 0, 0]], dtype=np.float32),
             lo=np.array([[1]], np.int32), hi=np.array([[1]], np.int32))
    orc, gpu, g = make_pair(d, entry=0)
    r = gpu_search(gpu, g, 2, [3], lam=2.0)              # tests/golden/ring_trace_finite_lambda.txt
    assert r["ids"][0].tolist() == [5, 7] and r["n_expand"][0] == 4 and r["n_scored"][0] == 5
    r = gpu_search(gpu, g, 2, [3], lam=0.5)
    assert r["ids"][0].tolist() == [5, SENTINEL] and r["n_expand"][0] == 5 and r["n_scored"][0] == 6
    gpu.close()
    w, d, orc, gpu, g = _get("c2")
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 128], mode="resume", dist_mode=1, lam=500.0,
                   expand_w=2)
    r = gpu_search(gpu, g, w.k, [16, 128], mode="resume", plus_k=3, lam=500.0, expand_w=2)
    assert_bit_parity(o, r, "BOA+/W=2/lambda=500")


@pytest.mark.parametrize("name", ["c2", "c4"])
def test_integer_data_matches_double_accumulation_too(name):
    """Every partial sum of integer-valued rows is below 2^24, so the fp32 order cannot
    matter: the GPU must also equal the oracle's double-precision distance mode."""
    w, d, orc, gpu, g = _get(name)
    widths = default_widths(w.L0, 128)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, mode="resume", dist_mode=0)
    r = gpu_search(gpu, g, w.k, widths, mode="resume")
    assert_bit_parity(o, r, name)


@pytest.mark.parametrize("name", ["c3", "c5"])
def test_float_data_within_tolerance_of_double_accumulation(name):
    """Against distances summed in double: ids identical except at near-ties (gap below
    1e-5 relative), distances within 1e-5 relative."""
    w, d, orc, gpu, g = _get(name)
    widths = [64]
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, dist_mode=0)
    r = gpu_search(gpu, g, w.k, widths)
    for i in range(w.Q):
        oi, ri = o["ids"][i], r["ids"][i]
        n = int((oi != SENTINEL).sum())
        assert int((ri != SENTINEL).sum()) == n
        np.testing.assert_allclose(r["d2"][i][:n], o["d2"][i][:n], rtol=1e-5)
        for t in np.nonzero(oi[:n] != ri[:n])[0]:
            near = np.abs(o["d2"][i][:n] - o["d2"][i][t]) <= 1e-5 * o["d2"][i][t]
            assert near.sum() > 1 or ri[t] in oi[:n], (i, t)


@pytest.mark.parametrize("name", ["c2", "c3"])
@pytest.mark.parametrize("plus_k", [2, 5, 10])
def test_boa_plus_equals_boa(name, plus_k):
    w, d, orc, gpu, g = _get(name)
    widths = default_widths(w.L0, 256)
    for mode in ("restart", "resume"):
        a = gpu_search(gpu, g, w.k, widths, mode=mode, plus_k=0)
        b = gpu_search(gpu, g, w.k, widths, mode=mode, plus_k=plus_k)
        assert (a["ids"] == b["ids"]).all() and (a["d2"].view(np.uint32) == b["d2"].view(np.uint32)).all()
        assert (a["final_L"] == b["final_L"]).all() and (a["n_expand"] == b["n_expand"]).all()
        assert (a["phase_active"] == b["phase_active"]).all()


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_two_chains_equal_one(name):
    """BOA_PARAM_CHAINS = 2: the halves of the batch go through their phases on two streams;
    ids, distances, statistics and phase counts are those of the one-chain schedule (and of the
    oracle), for even, odd and tiny batches, with PQ-free exact search in both modes."""
    w, d, orc, gpu, g = _get(name)
    widths = default_widths(w.L0, 256)
    for mode in ("restart", "resume"):
        a = gpu_search(gpu, g, w.k, widths, mode=mode, chains=1)
        assert gpu.last_launch_count == len(widths)
        b = gpu_search(gpu, g, w.k, widths, mode=mode, chains=2)
        assert gpu.last_launch_count == 2 * len(widths)
        for key in ("ids", "final_L", "n_expand", "n_scored", "flags", "phase_active"):
            assert (a[key] == b[key]).all(), key
        assert (a["d2"].view(np.uint32) == b["d2"].view(np.uint32)).all()
    o = orc.search(d["queries"][:31], d["lo"][:31], d["hi"][:31], w.k, widths, mode="resume", dist_mode=1)
    r = gpu_search(gpu, g, w.k, widths, mode="resume", chains=2, sel=slice(0, 31))
    assert_bit_parity(o, r, f"two chains {name}")
    for n in (1, 2, 3):
        a = gpu_search(gpu, g, w.k, widths, mode="resume", chains=1, sel=slice(0, n))
        b = gpu_search(gpu, g, w.k, widths, mode="resume", chains=2, sel=slice(0, n))
        assert (a["ids"] == b["ids"]).all() and (a["phase_active"] == b["phase_active"]).all()
    # a finite lambda, two nodes per iteration and BOA+ (which takes precedence) still work with it set
    a = gpu_search(gpu, g, w.k, widths, mode="resume", lam=500.0, expand_w=2, chains=1)
    b = gpu_search(gpu, g, w.k, widths, mode="resume", lam=500.0, expand_w=2, chains=2)
    c = gpu_search(gpu, g, w.k, widths, mode="resume", lam=500.0, expand_w=2, chains=2, plus_k=3)
    assert (a["ids"] == b["ids"]).all() and (a["ids"] == c["ids"]).all()
    assert (a["phase_active"] == b["phase_active"]).all() and (a["phase_active"] == c["phase_active"]).all()


def test_boa_plus_sub_batches_are_not_made_smaller_than_the_gpu():
    """With the default smallest sub-batch (twice the resident query warps) a batch of a few
    hundred queries runs as plain BOA whatever K says; plus_min_sub = 1 gives the K sub-batches."""
    w, d, orc, gpu, g = _get("c2")
    widths = default_widths(w.L0, 256)
    a = gpu_search(gpu, g, w.k, widths, mode="resume", plus_k=0, chains=1)
    boa_launches = gpu.last_launch_count
    b = gpu_search(gpu, g, w.k, widths, mode="resume", plus_k=5, chains=1)
    assert gpu.last_launch_count > boa_launches
    gpu.set_param("plus_min_sub", 0)
    ids, d2 = gpu.search(g["queries"], g["lo"], g["hi"], w.k, widths[0], widths[-1])
    assert gpu.last_launch_count == boa_launches
    assert (ids.cpu().numpy().view(np.uint32) == a["ids"]).all() and (a["ids"] == b["ids"]).all()
    gpu.set_param("plus_min_sub", 1)
    gpu.set_param("plus_k", 0)


def test_fixed_width_500_not_a_power_of_two():
    w, d, orc, gpu, g = _get("c2")
    o = orc.search(d["queries"][:80], d["lo"][:80], d["hi"][:80], w.k, [500], dist_mode=1)
    r = gpu_search(gpu, g, w.k, [500], sel=slice(0, 80))
    assert_bit_parity(o, r, "fixed500")


def test_eps_and_tau_special_cases():
    w, d, orc, gpu, g = _get("c2")
    widths = default_widths(16, 128)
    for eps in (-1.0, 1.0, 0.0, 0.3):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=eps, dist_mode=1)
        r = gpu_search(gpu, g, w.k, widths, eps=eps)
        assert_bit_parity(o, r, f"eps={eps}")
    o0 = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, dist_mode=1)
    for tau in ((o0["phase_active"][1] + 0.5) / w.Q, (o0["phase_active"][1] - 0.5) / w.Q, 1.0, 2.0):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, tau=tau, dist_mode=1)
        r = gpu_search(gpu, g, w.k, widths, tau=tau)
        assert_bit_parity(o, r, f"tau={tau}")
    # the boundary itself: tau * rho == |A| stops (strict > of Algorithm 1); 256 queries make
    # tau exact in floating point
    sl = slice(0, 256)
    a1 = int(orc.search(d["queries"][sl], d["lo"][sl], d["hi"][sl], w.k, widths, dist_mode=1)["phase_active"][1])
    assert 1 < a1 < 256
    for tau in (a1 / 256, (a1 - 1) / 256):
        o = orc.search(d["queries"][sl], d["lo"][sl], d["hi"][sl], w.k, widths, tau=tau, dist_mode=1)
        r = gpu_search(gpu, g, w.k, widths, tau=tau, sel=sl)
        assert_bit_parity(o, r, f"tau boundary {tau}")
    assert o["phase_active"][1] == a1


def test_expansion_cap():
    w, d, orc, gpu, g = _get("c2")
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 64], cap=(1, 3), dist_mode=1)
    r = gpu_search(gpu, g, w.k, [16, 64], cap=(1, 3))
    assert (o["flags"] & 1).any()
    assert_bit_parity(o, r, "cap")


def test_ring_hand_trace_on_gpu():
    x = np.zeros((8, 4), dtype=np.float32)
    x[:, 0] = np.arange(8)
    d = dict(vectors=x, attrs=(np.arange(8) % 2).astype(np.int32)[:, None],
             attr_types=np.zeros(1, np.int32),
             graph=np.stack([(np.arange(8) - 1) % 8, (np.arange(8) + 1) % 8], 1).astype(np.uint32),
             queries=np.array([[5.2, 0, 0, 0]], dtype=np.float32),
             lo=np.array([[1]], np.int32), hi=np.array([[1]], np.int32))
    orc, gpu, g = make_pair(d, entry=0)
    r = gpu_search(gpu, g, 2, [3])
    assert r["ids"][0].tolist() == [5, 7]
    np.testing.assert_allclose(r["d2"][0], [0.04, 3.24], rtol=1e-5)
    assert r["n_expand"][0] == 5 and r["n_scored"][0] == 6


def test_full_width_search_equals_bruteforce_on_gpu():
    rng = np.random.default_rng(7)
    N, D, R, k = 300, 8, 6, 10
    x = rng.integers(0, 32, size=(N, D)).astype(np.float32)
    g5 = exact_knn_graph(x, R - 1, device="cpu")
    ring = ((np.arange(N) + 1) % N).astype(np.uint32)[:, None]
    d = dict(vectors=x, attrs=rng.integers(0, 100, size=(N, 2)).astype(np.int32),
             attr_types=np.zeros(2, np.int32), graph=clean_rows(np.concatenate([g5, ring], 1)),
             queries=rng.integers(0, 32, size=(25, D)).astype(np.float32))
    d["lo"] = rng.integers(0, 50, size=(25, 2)).astype(np.int32)
    d["hi"] = (d["lo"] + rng.integers(20, 60, size=(25, 2))).astype(np.int32)
    orc, gpu, g = make_pair(d)
    gt_ids, gt_d2, nvalid = orc.bruteforce(d["queries"], d["lo"], d["hi"], k)
    r = gpu_search(gpu, g, k, [N], cap=(8, 64))
    assert (r["ids"] == gt_ids).all()
    assert (r["n_expand"] == N).all()
    fin = gt_ids != SENTINEL
    assert (r["d2"][fin].astype(np.float64) == gt_d2[fin]).all()


def test_dirty_graph_rows_empty_ranges_and_short_answers():
    w = C2.scaled(5000, 64, name="c2_dirty")
    d = make_workload(w, seed=9)
    rng = np.random.default_rng(0)
    gph = d["graph"].copy()
    rows = rng.integers(0, w.N, size=800)
    gph[rows, 3] = rows.astype(np.uint32)                   # self references
    gph[rows, 7] = gph[rows, 1]                             # repeats
    gph[rng.integers(0, w.N, size=500), rng.integers(0, w.R, size=500)] = SENTINEL
    d["graph"] = gph
    d["lo"][0], d["hi"][0] = d["hi"][0].copy(), d["lo"][0].copy() - 1      # lo > hi: empty
    d["hi"][1] = d["lo"][1]                                  # very few valid points
    d["lo"][2] = np.iinfo(np.int32).min
    d["hi"][2] = np.iinfo(np.int32).max                      # unconstrained
    orc, gpu, g = make_pair(d)
    widths = [16, 64, 128]
    for mode in ("restart", "resume"):
        o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, mode=mode, dist_mode=1)
        r = gpu_search(gpu, g, w.k, widths, mode=mode)
        assert_bit_parity(o, r, f"dirty/{mode}")
    assert (r["ids"][0] == SENTINEL).all() and np.isinf(r["d2"][0]).all()
    assert r["final_L"][0] == 128


def test_k_equals_L0_and_k_one():
    w, d, orc, gpu, g = _get("c2")
    for k, widths in ((16, [16, 64]), (1, [16, 64])):
        o = orc.search(d["queries"], d["lo"], d["hi"], k, widths, dist_mode=1)
        r = gpu_search(gpu, g, k, widths)
        assert_bit_parity(o, r, f"k={k}")


def test_empty_batch_and_argument_errors():
    from paper_2609_16175_b200 import BoaError
    w, d, orc, gpu, g = _get("c2")
    gpu.set_schedule([])
    q0 = g["queries"][:0]
    ids, d2 = gpu.search(q0, g["lo"][:0], g["hi"][:0], 10, 16, 64)
    assert ids.shape == (0, 10)
    for k, L0, Lmax in ((0, 16, 64), (17, 16, 64), (10, 64, 16), (10, 16, 4096)):
        with pytest.raises(BoaError):
            gpu.search(g["queries"], g["lo"], g["hi"], k, L0, Lmax)
    # a finite lambda must stay finite in fp32; infinity (the default) is accepted
    with pytest.raises(BoaError) as e:
        gpu.set_param("lam", 1e39)
    assert e.value.status == -1
    gpu.set_param("lam", 3.0e38)
    gpu.set_param("lam", float("inf"))
    bad = g["graph"].clone()
    bad[5, 2] = w.N + 3
    from paper_2609_16175_b200 import BoaIndex
    with pytest.raises(BoaError) as e:
        BoaIndex(g["vectors"], g["attrs"], d["attr_types"].tolist(), bad)
    assert e.value.status == -4


def test_explicit_entry_and_growth_schedule():
    w, d, _, _, _ = _get("c2")
    orc, gpu, g = make_pair(d, entry=123)
    assert gpu.entry == 123
    gpu.set_schedule([])
    gpu.set_param("growth", 4)
    gpu.set_param("mode", 0)
    ids, d2 = gpu.search(g["queries"], g["lo"], g["hi"], 10, 16, 100)     # 16, 64, 100
    torch.cuda.synchronize()
    o = orc.search(d["queries"], d["lo"], d["hi"], 10, [16, 64, 100], dist_mode=1)
    assert (ids.cpu().numpy().view(np.uint32) == o["ids"]).all()
    assert gpu.phase_counts() == o["phase_active"].tolist()
