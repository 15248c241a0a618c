"""boa_index_share: two handles on one index searching at the same time on two streams give
what one handle gives alone; a shared handle keeps its own parameters and scratch."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C5, make_workload
from boa_synth.pq import train_pq
from tests.helpers import to_gpu

pytestmark = pytest.mark.gpu


def _search(ix, t, w, widths, stream=None, sel=slice(None)):
    ids, d2 = ix.search(t["queries"][sel], t["lo"][sel], t["hi"][sel], w.k, widths[0], widths[-1], stream=stream)
    return ids, d2


def test_two_handles_in_flight_equal_one_alone():
    from paper_2609_16175_b200 import BoaError, BoaIndex
    w = C2.scaled(60_000, 3000, name="c2_share")
    d = make_workload(w, seed=71)
    t = to_gpu(d)
    a = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    a.set_param("mode", 1); a.set_param("eps", 0.05); a.set_schedule([16, 64, 256])
    b = a.share()
    ref_ids, ref_d2 = _search(a, t, w, [16, 64, 256])
    ref_stats = {k: v.cpu().numpy() for k, v in a.stats().items()}
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    outs = []
    for rep in range(6):                      # alternate handles and streams without waiting in between
        ix, st = (a, s1) if rep % 2 == 0 else (b, s2)
        outs.append(_search(ix, t, w, [16, 64, 256], stream=st))
    torch.cuda.synchronize()
    for ids, d2 in outs:
        assert (ids == ref_ids).all() and (d2.view(torch.int32) == ref_d2.view(torch.int32)).all()
    for ix in (a, b):
        st = {k: v.cpu().numpy() for k, v in ix.stats().items()}
        for k in ref_stats:
            assert (st[k] == ref_stats[k]).all(), k
    # parameters are per handle: the shared one took a's at the time of sharing, later changes stay apart
    b.set_schedule([48]); b.set_param("mode", 0)
    ids_b, _ = _search(b, t, w, [48])
    ids_a, _ = _search(a, t, w, [16, 64, 256])
    assert (ids_a == ref_ids).all()
    assert int(b.stats()["final_L"].max()) == 48 and int(a.stats()["final_L"].max()) > 48
    assert not (ids_b == ref_ids).all()
    # what would change the shared data is refused on a shared handle
    with pytest.raises(BoaError):
        b.set_metric("cosine")
    piv, codes = train_pq(d["vectors"], M=16, K=16, iters=2, seed=1, device="cuda:0")
    with pytest.raises(BoaError):
        b.attach_pq(torch.from_numpy(piv).cuda(), torch.from_numpy(codes).cuda())
    # a share taken after the codebook is attached searches with it
    a.attach_pq(torch.from_numpy(piv).cuda(), torch.from_numpy(codes).cuda())
    a.set_param("pq", 1)
    c = a.share()
    pa, _ = _search(a, t, w, [16, 64, 256])
    pc, _ = _search(c, t, w, [16, 64, 256])
    assert (pa == pc).all() and (c.rerank_counts() == a.rerank_counts()).all()
    c.close(); b.close(); a.close()


def test_shared_handle_with_range_penalty_and_host_entry():
    from paper_2609_16175_b200 import BoaIndex
    w = C5.scaled(8_000, 300, name="c5_share")
    d = make_workload(w, seed=72)
    t = to_gpu(d)
    a = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    a.set_param("mode", 1); a.set_param("lam", 2.0); a.set_schedule([16, 128])
    a.set_range_penalty([1e-3] * w.m)
    b = a.share()
    a.set_range_penalty(None)                       # b keeps its own copy of the scales
    a.set_param("lam", float("inf"))
    ids_b, _ = _search(b, t, w, [16, 128])
    a.set_param("lam", 2.0); a.set_range_penalty([1e-3] * w.m)
    ids_a, _ = _search(a, t, w, [16, 128])
    assert (ids_a == ids_b).all()
    hq, hlo, hhi = (torch.from_numpy(d[k]).pin_memory() for k in ("queries", "lo", "hi"))
    ids_h, _ = b.search_host(hq, hlo, hhi, w.k, 16, 128)
    assert (ids_h.numpy() == ids_a.cpu().numpy()).all()
    b.close(); a.close()
