"""Shared plumbing of the GPU parity tests: build one workload, hand the same arrays
to the CPU oracle (numpy) and to the CUDA library (torch device tensors)."""
from __future__ import annotations

import numpy as np
import torch

from oracle.boa_oracle import OracleIndex


def to_gpu(d):
    dev = torch.device("cuda:0")
    return dict(
        vectors=torch.from_numpy(d["vectors"]).to(dev),
        attrs=torch.from_numpy(d["attrs"]).to(dev),
        graph=torch.from_numpy(d["graph"].view(np.int32)).to(dev),
        queries=torch.from_numpy(d["queries"]).to(dev),
        lo=torch.from_numpy(d["lo"]).to(dev),
        hi=torch.from_numpy(d["hi"]).to(dev),
    )


def make_pair(d, entry=-1):
    """(oracle index, GPU index, device tensors) over the same arrays."""
    from paper_2609_16175_b200 import BoaIndex
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"], entry=entry)
    g = to_gpu(d)
    gpu = BoaIndex(g["vectors"], g["attrs"], d["attr_types"].tolist(), g["graph"], entry=entry)
    return orc, gpu, g


def gpu_search(gpu, g, k, widths, mode="restart", eps=0.05, tau=0.0, plus_k=0, cap=(8, 64),
               sel=None, expand_w=1, lam=float("inf"), pq=False, penalty_scales=None, chains=0):
    gpu.set_param("mode", 1 if mode == "resume" else 0)
    gpu.set_param("eps", eps)
    gpu.set_param("tau", tau)
    gpu.set_param("plus_k", plus_k)
    gpu.set_param("plus_min_sub", 1)          # tests want K sub-batches whatever the batch size
    gpu.set_param("chains", chains)
    gpu.set_param("cap_mult", cap[0])
    gpu.set_param("cap_add", cap[1])
    gpu.set_param("expand_w", expand_w)
    gpu.set_param("lam", lam)
    gpu.set_param("pq", 1 if pq else 0)
    gpu.set_range_penalty(penalty_scales)
    gpu.set_schedule(list(widths))
    q, lo, hi = g["queries"], g["lo"], g["hi"]
    if sel is not None:
        q, lo, hi = q[sel].contiguous(), lo[sel].contiguous(), hi[sel].contiguous()
    ids, d2 = gpu.search(q, lo, hi, k, widths[0], widths[-1])
    st = gpu.stats()
    counts = gpu.phase_counts()
    torch.cuda.synchronize()
    out = dict(ids=ids.cpu().numpy().view(np.uint32), d2=d2.cpu().numpy(),
               phase_active=np.array(counts, dtype=np.int64))
    for kk, v in st.items():
        out[kk] = v.cpu().numpy()
    return out


def assert_bit_parity(o, r, what=""):
    """Oracle run `o` (dist_mode=1) against GPU run `r`: everything integer is
    identical, distances are identical bit for bit."""
    bad = np.nonzero((o["ids"] != r["ids"]).any(1))[0]
    assert bad.size == 0, f"{what}: ids differ for queries {bad[:10]} " \
                          f"oracle {o['ids'][bad[:2]]} gpu {r['ids'][bad[:2]]}"
    assert (o["d2"].view(np.uint32) == r["d2"].view(np.uint32)).all(), f"{what}: distances differ"
    assert (o["final_L"] == r["final_L"]).all(), f"{what}: final_L differs"
    assert (o["n_expand"] == r["n_expand"]).all(), f"{what}: expansion counts differ"
    assert (o["flags"] == r["flags"]).all(), f"{what}: flags differ"
    # the GPU's table of scored ids may forget: it never scores fewer than the exact set
    assert (r["n_scored"] >= o["n_scored"]).all(), f"{what}: scored fewer than the oracle"
    n = min(len(o["phase_active"]), len(r["phase_active"]))
    assert (o["phase_active"][:n] == r["phase_active"][:n]).all(), f"{what}: phase counts differ"
