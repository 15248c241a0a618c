"""boa_search_noalloc against boa_search.

The no-allocation entry point serves callers that have given all device memory to their
own pools, or cannot afford the synchronisation an allocation may bring: its scratch is
a fixed array inside the library.  It must return exactly what boa_search returns --
here on two calls in a row, the second smaller than the first, so that anything the
first call left in the shared array would show.  This file is collected last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from boa_synth import C2, make_workload

pytestmark = pytest.mark.gpu


def _tensors(d, dev):
    return {k: torch.from_numpy(v.view(np.int32) if v.dtype == np.uint32 else v).to(dev)
            for k, v in d.items() if k in ("vectors", "attrs", "graph", "queries", "lo", "hi")}


@pytest.mark.parametrize("mode", [0, 1])
def test_noalloc_equals_boa_search_on_two_calls_in_a_row(mode):
    from paper_2609_16175_b200 import BoaError, BoaIndex
    dev = torch.device("cuda:0")
    w = C2.scaled(30_000, 700, name="c2_noalloc")
    d = make_workload(w, seed=11)
    t = _tensors(d, dev)
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    ix.set_param("mode", mode)
    ix.set_param("eps", 0.05)
    widths = [16, 64, 256]
    ix.set_schedule(widths)
    k = w.k
    for lo_q, hi_q in ((0, 700), (100, 333)):               # two calls in a row
        q = t["queries"][lo_q:hi_q].contiguous()
        lo = t["lo"][lo_q:hi_q].contiguous()
        hi = t["hi"][lo_q:hi_q].contiguous()
        ref_ids, ref_d2 = ix.search(q, lo, hi, k, widths[0], widths[-1])
        torch.cuda.synchronize()
        ids = torch.full_like(ref_ids, -7)
        d2 = torch.full_like(ref_d2, -7.0)
        free_before = torch.cuda.mem_get_info()[0]
        ix.search_noalloc(q, lo, hi, k, widths[0], widths[-1], ids, d2)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before       # no device allocation happened
        assert torch.equal(ids, ref_ids)                          # integer results: identical
        assert torch.equal(d2.view(torch.int32), ref_d2.view(torch.int32))   # fp32 bits identical
        assert (ref_ids != -1).any()
    # beyond the fixed scratch: a clear error, nothing written
    big = torch.zeros((1025, w.D), dtype=torch.float32, device=dev)
    z = torch.zeros((1025, w.m), dtype=torch.int32, device=dev)
    oi = torch.zeros((1025, k), dtype=torch.int32, device=dev)
    od = torch.zeros((1025, k), dtype=torch.float32, device=dev)
    with pytest.raises(BoaError) as e:
        ix.search_noalloc(big, z, z, k, widths[0], widths[-1], oi, od)
    assert e.value.status == -5
    torch.cuda.synchronize()
    assert not oi.any() and not od.any()                              # nothing was written
    ix.close()


def _compare(ix, t, sl, k, widths, plus_k=0):
    """boa_search, then boa_search_noalloc, on queries sl: identical bits, no allocation."""
    ix.set_param("plus_k", plus_k)
    ix.set_param("plus_min_sub", 1)
    ix.set_schedule(widths)
    q, lo, hi = (t[n][sl].contiguous() for n in ("queries", "lo", "hi"))
    ref_ids, ref_d2 = ix.search(q, lo, hi, k, widths[0], widths[-1])
    st = {n: v.clone() for n, v in ix.stats().items()}
    counts = ix.phase_counts()
    torch.cuda.synchronize()
    ids = torch.full_like(ref_ids, -7)
    d2 = torch.full_like(ref_d2, -7.0)
    free_before = torch.cuda.mem_get_info()[0]
    ix.search_noalloc(q, lo, hi, k, widths[0], widths[-1], ids, d2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert torch.equal(ids, ref_ids)
    assert torch.equal(d2.view(torch.int32), ref_d2.view(torch.int32))
    # the statistics calls still describe the boa_search before it
    st2 = ix.stats()
    assert all(torch.equal(st[n], st2[n]) for n in st) and ix.phase_counts() == counts
    return ref_ids


def test_noalloc_at_the_edges_of_the_fixed_array():
    """The largest batch and the largest width the fixed array allows, in resume mode (the
    last query's carried pool then ends exactly at the end of the array); the overlapped
    schedule, which uses the second set of survivor lists and counters in the array; and a
    first call on an index that has never run boa_search and so owns no scratch at all."""
    from paper_2609_16175_b200 import BoaIndex
    dev = torch.device("cuda:0")
    w = C2.scaled(30_000, 1024, name="c2_noalloc_edges")
    d = make_workload(w, seed=12)
    t = _tensors(d, dev)
    k = w.k
    # fresh index: the no-allocation call comes first
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    ix.set_param("mode", 1)
    ix.set_param("eps", 0.05)
    widths = [16, 512]
    ix.set_schedule(widths)
    first_ids = torch.full((1024, k), -7, dtype=torch.int32, device=dev)
    first_d2 = torch.full((1024, k), -7.0, dtype=torch.float32, device=dev)
    ix.search_noalloc(t["queries"], t["lo"], t["hi"], k, 16, 512, first_ids, first_d2)
    torch.cuda.synchronize()
    ref = _compare(ix, t, slice(0, 1024), k, widths)                  # Q = 1024, Lmax = 512, resume
    assert torch.equal(first_ids, ref)
    for plus_k in (2, 4):
        _compare(ix, t, slice(0, 1024), k, [16, 64, 512], plus_k=plus_k)
        _compare(ix, t, slice(4, 900), k, [16, 64, 256, 512], plus_k=plus_k)   # rows stay 16-byte aligned
    ix.set_param("mode", 0)
    _compare(ix, t, slice(0, 1024), k, [16, 128, 512], plus_k=4)
    ix.close()
