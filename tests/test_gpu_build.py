"""Graph construction on the GPU against the oracle's builder: the same graph, entry by entry,
on float and byte data, with one and with several attribute thresholds and passes."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C3, C4, SENTINEL, make_workload
from oracle.boa_oracle import OracleIndex

pytestmark = pytest.mark.gpu
INF = float("inf")


def _positions(attrs, types):
    n, m = attrs.shape
    pos = np.empty((n, m), np.float32)
    for j in range(m):
        col = attrs[:, j].view(np.float32) if types[j] == 1 else attrs[:, j]
        o = np.argsort(col, kind="stable")
        pos[o, j] = np.arange(n, dtype=np.float32) / n
    return pos


def _build_both(w, seed, **kw):
    from paper_2609_16175_b200 import build_graph
    d = make_workload(w, seed=seed, with_graph=False)
    pos = _positions(d["attrs"], d["attr_types"])
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], np.zeros((w.N, 1), np.uint32))
    go = orc.build_graph(pos, **kw)
    gg = build_graph(torch.from_numpy(d["vectors"]).to("cuda:0"), torch.from_numpy(pos).to("cuda:0"), **kw)
    torch.cuda.synchronize()
    return d, pos, orc, go, gg.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("case", [
    ("c2", C2.scaled(3000, 20, name="c2_b"), dict(R=16, Lb=32, alpha=1.2, B=128, passes=1)),
    ("c2t", C2.scaled(4000, 20, name="c2_bt"), dict(R=24, Lb=48, alpha=1.2, thresholds=(INF, 0.2, 0.05), B=256, passes=2)),
    ("c3", C3.scaled(3000, 20, name="c3_b"), dict(R=16, Lb=32, alpha=1.3, thresholds=(INF, 0.1), B=64, passes=1)),
    ("c3v", C3.scaled(3000, 20, name="c3_bv"), dict(R=24, Lb=40, alpha=1.2, B=128, passes=2,
                                                    thresholds=(INF, (0.1, INF, INF), (INF, 0.05, 0.2)))),
    ("c4", C4.scaled(3000, 20, name="c4_b"), dict(R=32, Lb=40, alpha=1.2, thresholds=(INF, 0.15), B=200, passes=2, cap_in=8)),
], ids=lambda c: c[0])
def test_gpu_builds_the_oracles_graph(case):
    name, w, kw = case
    d, pos, orc, go, gg = _build_both(w, seed=51, **kw)
    bad = np.nonzero((go != gg).any(1))[0]
    assert bad.size == 0, f"{name}: rows differ, first {bad[:5]}: oracle {go[bad[:2]]} gpu {gg[bad[:2]]}"
    real = gg != SENTINEL
    assert (gg[real] < w.N).all() and real.sum(1).min() >= 1


def test_search_parity_over_the_oracles_built_graph():
    """The graph the oracle's builder made (equal to the library's, checked first) handed to both
    searches: the filter-aware search agrees bit for bit over a threshold-pruned graph too."""
    from paper_2609_16175_b200 import BoaIndex
    from tests.helpers import assert_bit_parity, gpu_search, to_gpu
    w = C2.scaled(5000, 60, name="c2_bs")
    d, pos, _, go, gg = _build_both(w, seed=53, R=24, Lb=48, alpha=1.2, thresholds=(INF, 0.2, 0.05), B=512, passes=1)
    assert (go == gg).all()
    d["graph"] = go
    t = to_gpu(d)
    gpu = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], go)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [16, 64, 256], mode="resume", dist_mode=1)
    r = gpu_search(gpu, t, w.k, [16, 64, 256], mode="resume")
    assert_bit_parity(o, r, "search over a built graph")
    gpu.close()


def test_built_graph_serves_the_search():
    """A graph built by the library, handed to boa_index_create: an unfiltered search finds the
    true neighbours and a filtered one finds more of them than over a graph built without the
    attribute thresholds (what the threshold passes are for)."""
    from paper_2609_16175_b200 import BoaIndex, build_graph
    from boa_synth.groundtruth import filtered_topk, recall_against
    from tests.helpers import to_gpu
    w = C2.scaled(60_000, 400, name="c2_built")
    d = make_workload(w, seed=52, with_graph=False)
    pos = _positions(d["attrs"], d["attr_types"])
    dev = torch.device("cuda:0")
    d["graph"] = np.zeros((w.N, 1), np.uint32)
    t = to_gpu(d)
    full_lo = torch.full_like(t["lo"], -2 ** 31)
    full_hi = torch.full_like(t["hi"], 2 ** 31 - 1)

    def recalls(thresholds):
        g = build_graph(t["vectors"], torch.from_numpy(pos).to(dev), R=32, Lb=64, alpha=1.2, thresholds=thresholds,
                        B=2048, passes=2)
        gpu = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), g)
        gpu.set_schedule([64]); gpu.set_param("mode", 0)
        out = []
        for lo, hi in ((full_lo, full_hi), (t["lo"], t["hi"])):
            ids, d2 = gpu.search(t["queries"], lo, hi, w.k, 64, 64)
            _, gt_d2, gt_nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"], lo, hi, w.k)
            rec = recall_against(ids.cpu().numpy().view(np.uint32), d2.cpu().numpy(), gt_d2.cpu().numpy(),
                                 gt_nv.cpu().numpy(), w.k)
            out.append(float(np.nanmean(rec)))
        gpu.close()
        return out

    plain, plain_f = recalls((INF,))
    mixed, mixed_f = recalls((INF, 0.3, 0.05))
    assert plain > 0.95 and mixed > 0.9
    assert mixed_f > 0.95 and mixed_f > plain_f


@pytest.mark.parametrize("n", [1, 2, 5, 40])
def test_tiny_and_degenerate_inputs(n):
    """Fewer points than the degree or the beamwidth, and repeated vectors (distance 0 to each
    other): the same graph as the oracle's, no self loops, no repeats in a row."""
    from paper_2609_16175_b200 import build_graph
    rng = np.random.default_rng(n)
    D = 16
    x = rng.standard_normal((n, D)).astype(np.float32)
    if n >= 5:
        x[n // 2:] = x[: n - n // 2]                      # every vector of the second half repeats one of the first
    attrs = rng.integers(0, 100, size=(n, 2)).astype(np.int32)
    types = np.zeros(2, np.int32)
    pos = _positions(attrs, types)
    kw = dict(R=8, Lb=16, alpha=1.2, thresholds=(INF, 0.3), B=4, passes=2)
    orc = OracleIndex(x, attrs, types, np.zeros((n, 1), np.uint32))
    go = orc.build_graph(pos, **kw)
    gg = build_graph(torch.from_numpy(x).to("cuda:0"), torch.from_numpy(pos).to("cuda:0"), **kw).cpu().numpy().view(np.uint32)
    assert (go == gg).all(), (go, gg)
    for r in range(n):
        row = gg[r][gg[r] != SENTINEL]
        assert r not in row and len(set(row.tolist())) == len(row) and (row < n).all()
