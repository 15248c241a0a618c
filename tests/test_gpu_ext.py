"""Membership (subset / equality) predicates and the distance-to-range penalty: CUDA library
against the oracle, bit for bit, through the C interface."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C3, C4, C5, SENTINEL, make_workload
from tests.helpers import assert_bit_parity, gpu_search, make_pair

pytestmark = pytest.mark.gpu
SET = 2


def _with_tags(w, seed):
    """The workload with one more attribute column: a 32-bit set of tags per point, and a
    membership predicate per query (any-of for even queries, all-of for odd ones)."""
    d = make_workload(w, seed=seed)
    rng = np.random.default_rng(seed + 100)
    tags = (rng.integers(0, 2 ** 16, size=w.N) & rng.integers(0, 2 ** 16, size=w.N) |
            (rng.integers(0, 2, size=w.N) << 31)).astype(np.uint32).view(np.int32)
    d["attrs"] = np.ascontiguousarray(np.concatenate([d["attrs"], tags[:, None]], 1))
    d["attr_types"] = np.concatenate([d["attr_types"], [SET]]).astype(np.int32)
    want = rng.integers(1, 2 ** 16, size=w.Q).astype(np.uint32)
    want[::2] |= rng.integers(1, 2 ** 16, size=want[::2].shape[0]).astype(np.uint32)      # any-of: wide wishes
    want[1::2] &= rng.integers(1, 2 ** 16, size=want[1::2].shape[0]).astype(np.uint32)    # all-of: short wishes
    want[5] = 0x80000000
    mode = (np.arange(w.Q) % 2).astype(np.int32)
    d["lo"] = np.ascontiguousarray(np.concatenate([d["lo"], want.view(np.int32)[:, None]], 1))
    d["hi"] = np.ascontiguousarray(np.concatenate([d["hi"], mode[:, None]], 1))
    return d


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_membership_predicates_match_oracle(name):
    w = {"c2": C2.scaled(30_000, 120, name="c2_set"), "c3": C3.scaled(25_000, 100, name="c3_set"),
         "c4": C4.scaled(40_000, 100, name="c4_set"), "c5": C5.scaled(6_000, 60, name="c5_set")}[name]
    d = _with_tags(w, seed=41)
    orc, gpu, g = make_pair(d)
    for mode in ("restart", "resume"):
        for widths, lam in (([w.L0, 64, 256], float("inf")), ([48], float("inf")), ([w.L0, 128], 3000.0)):
            o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=0.1, mode=mode, dist_mode=1, lam=lam)
            r = gpu_search(gpu, g, w.k, widths, mode=mode, eps=0.1, lam=lam)
            assert_bit_parity(o, r, f"set {name}/{mode}/{widths}/{lam}")
    found = r["ids"] != SENTINEL
    assert found.any()
    tags = d["attrs"][:, -1].view(np.uint32)
    for i in range(w.Q):
        have = tags[r["ids"][i][found[i]].astype(np.int64)] & np.uint32(d["lo"][i, -1])
        ok = (have != 0) if d["hi"][i, -1] == 0 else (have == np.uint32(d["lo"][i, -1]))
        assert ok.all()
    b = gpu_search(gpu, g, w.k, [w.L0, 64, 256], mode="resume", eps=0.1, plus_k=3)
    a = gpu_search(gpu, g, w.k, [w.L0, 64, 256], mode="resume", eps=0.1)
    assert (a["ids"] == b["ids"]).all()
    gpu.close()


@pytest.mark.parametrize("name", ["c2", "c3", "c4"])
def test_range_penalty_matches_oracle(name):
    from paper_2609_16175_b200 import BoaError
    w = {"c2": C2.scaled(30_000, 120, name="c2_pen"), "c3": C3.scaled(25_000, 100, name="c3_pen"),
         "c4": C4.scaled(40_000, 100, name="c4_pen")}[name]
    d = _with_tags(w, seed=43) if name == "c3" else make_workload(w, seed=43)
    orc, gpu, g = make_pair(d)
    m = d["attrs"].shape[1]
    # scales that bring each attribute's typical excess to the scale of the distances
    span = [float(np.ptp(d["attrs"][:, j].view(np.float32) if t == 1 else d["attrs"][:, j].astype(np.float64)))
            if t != SET else 1.0 for j, t in enumerate(d["attr_types"])]
    dscale = 4000.0 if name != "c3" else 0.05
    scales = [dscale / max(s, 1e-9) for s in span]
    for mode in ("restart", "resume"):
        for widths, lam in (([w.L0, 64, 256], 1.0), ([40], 10.0), ([w.L0, 512], 0.25)):
            o = orc.search(d["queries"], d["lo"], d["hi"], w.k, widths, eps=0.1, mode=mode, dist_mode=1, lam=lam,
                           penalty_scales=scales)
            r = gpu_search(gpu, g, w.k, widths, mode=mode, eps=0.1, lam=lam, penalty_scales=scales)
            assert_bit_parity(o, r, f"penalty {name}/{mode}/{widths}/{lam}")
    # it is a different walk from the count's
    c = gpu_search(gpu, g, w.k, [w.L0, 64, 256], lam=1.0)
    p = gpu_search(gpu, g, w.k, [w.L0, 64, 256], lam=1.0, penalty_scales=scales)
    assert (p["n_expand"] != c["n_expand"]).any()
    with pytest.raises(BoaError):                      # the penalty is a term of the finite-lambda score
        gpu_search(gpu, g, w.k, [w.L0, 64], penalty_scales=scales)
    with pytest.raises(BoaError):
        gpu.set_range_penalty([0.0] * m)
    with pytest.raises(BoaError):
        gpu_search(gpu, g, w.k, [w.L0, 64], lam=1.0, penalty_scales=scales, expand_w=2)
    o = orc.search(d["queries"], d["lo"], d["hi"], w.k, [w.L0, 64], dist_mode=1)
    r = gpu_search(gpu, g, w.k, [w.L0, 64])                                   # and back to the default
    assert_bit_parity(o, r, "back to the count")
    gpu.close()
