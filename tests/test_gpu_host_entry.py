"""boa_search_host: host buffers in and out through the C interface, same results as
boa_search on device buffers."""
import numpy as np
import pytest
import torch

from boa_synth import C2, C4, make_workload
from tests.helpers import to_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c2", "c4"])
def test_host_entry_equals_device_entry(name):
    from paper_2609_16175_b200 import BoaError, BoaIndex
    w = {"c2": C2.scaled(30_000, 300, name="c2_host"), "c4": C4.scaled(40_000, 200, name="c4_host")}[name]
    d = make_workload(w, seed=61)
    t = to_gpu(d)
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    ix.set_param("mode", 1); ix.set_param("eps", 0.05); ix.set_schedule([w.L0, 64, 256])
    hq, hlo, hhi = torch.from_numpy(d["queries"]), torch.from_numpy(d["lo"]), torch.from_numpy(d["hi"])
    # a small batch first, then the whole one (the staging buffers grow), pageable then pinned
    # pinned buffers are read in place by the kernels unless that is switched off
    for sel, pin, in_place in ((slice(0, 17), False, 1), (slice(0, w.Q), False, 1), (slice(5, 150), True, 1),
                               (slice(0, w.Q), True, 1), (slice(0, w.Q), True, 0), (slice(3, 40), True, 0)):
        ix.set_param("host_in_place", in_place)
        q, lo, hi = hq[sel].contiguous(), hlo[sel].contiguous(), hhi[sel].contiguous()
        out = (None, None)
        if pin:
            q, lo, hi = q.pin_memory(), lo.pin_memory(), hi.pin_memory()
            out = (torch.empty((q.shape[0], w.k), dtype=torch.int32).pin_memory(),
                   torch.empty((q.shape[0], w.k), dtype=torch.float32).pin_memory())
        # device buffers must start on 16 bytes (clone); the host entry has no such rule
        ids_d, d2_d = ix.search(t["queries"][sel].clone(), t["lo"][sel].clone(), t["hi"][sel].clone(), w.k, w.L0, 256)
        st_d = {k: v.cpu().numpy() for k, v in ix.stats().items()}
        ids_h, d2_h = ix.search_host(q, lo, hi, w.k, w.L0, 256, *out)
        st_h = {k: v.cpu().numpy() for k, v in ix.stats().items()}
        assert not ids_h.is_cuda and (ids_h.numpy() == ids_d.cpu().numpy()).all()
        assert (d2_h.numpy().view(np.uint32) == d2_d.cpu().numpy().view(np.uint32)).all()
        for key in st_d:
            assert (st_d[key] == st_h[key]).all(), key
    # a larger k than any before grows the output staging; an empty batch is fine
    ix.set_schedule([32, 256])
    ids_d, _ = ix.search(t["queries"], t["lo"], t["hi"], 32, 32, 256)
    ids_h, _ = ix.search_host(hq, hlo, hhi, 32, 32, 256)
    assert (ids_h.numpy() == ids_d.cpu().numpy()).all()
    e_ids, e_d2 = ix.search_host(hq[:0].contiguous(), hlo[:0].contiguous(), hhi[:0].contiguous(), 10, 32, 256)
    assert e_ids.shape == (0, 10)
    with pytest.raises(BoaError):                       # boa_search's argument checks apply
        ix.search_host(hq, hlo, hhi, 64, 32, 256)
    with pytest.raises(ValueError):
        ix.search_host(t["queries"], hlo, hhi, 10, 32, 256)
    ix.close()
