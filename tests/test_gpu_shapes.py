"""Kernel variants the five benchmark shapes do not reach: row lengths that are not a
multiple of eight 16-byte chunks, long generic rows, uint8 rows of odd chunk counts, the
largest attribute count, degree and beamwidth, odd degrees.  Random small inputs, both
modes, bit parity with the oracle's fixed-order fp32 distances."""
import numpy as np
import pytest

from boa_synth import SENTINEL, clean_rows, exact_knn_graph
from tests.helpers import assert_bit_parity, gpu_search, make_pair

pytestmark = pytest.mark.gpu


def _random_case(seed, N, D, dtype, m, R, Q, float_cols=()):
    rng = np.random.default_rng(seed)
    if dtype == "u8":
        x = rng.integers(0, 256, size=(N, D)).astype(np.uint8)
        q = rng.integers(0, 256, size=(Q, D)).astype(np.float32)
    else:
        x = rng.standard_normal((N, D)).astype(np.float32)
        q = rng.standard_normal((Q, D)).astype(np.float32)
    attrs = rng.integers(0, 1000, size=(N, m)).astype(np.int32)
    types = np.zeros(m, dtype=np.int32)
    lo = rng.integers(0, 400, size=(Q, m)).astype(np.int32)
    hi = (lo + rng.integers(300, 900, size=(Q, m))).astype(np.int32)
    for j in float_cols:
        types[j] = 1
        attrs[:, j] = rng.random(N, dtype=np.float32).view(np.int32)
        l = (0.4 * rng.random(Q)).astype(np.float32)
        lo[:, j] = l.view(np.int32)
        hi[:, j] = (l + np.float32(0.5)).astype(np.float32).view(np.int32)
    near = exact_knn_graph(x.astype(np.float32), max(1, R - 2), device="cpu")
    far = rng.integers(0, N, size=(N, R - near.shape[1])).astype(np.uint32)
    g = clean_rows(np.concatenate([near, far], 1)[:, :R])
    return dict(vectors=x, attrs=attrs, attr_types=types, graph=g, queries=q, lo=lo, hi=hi)


CASES = [
    # name,           N,    D,  dtype, m, R,  k, widths,          float columns
    ("f32_5chunks",   3000, 20,  "f32", 2, 16, 5,  [8, 32, 64],    ()),
    ("f32_25chunks",  3000, 100, "f32", 3, 32, 10, [16, 64],       (1,)),
    ("f32_50chunks",  2500, 200, "f32", 2, 24, 10, [16, 128],      ()),
    ("f32_1chunk",    2000, 4,   "f32", 1, 7,  3,  [4, 16],        ()),
    ("u8_3chunks",    3000, 48,  "u8",  2, 16, 10, [16, 64],       ()),
    ("u8_17chunks",   2500, 272, "u8",  2, 40, 10, [16, 64],       ()),
    ("u8_12chunks",   2500, 192, "u8",  4, 33, 10, [12, 100],      (3,)),
    ("max_attrs_deg", 4000, 64,  "f32", 8, 64, 10, [16, 256, 1024], (0, 5)),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_shape_variants_match_oracle(case):
    name, N, D, dtype, m, R, k, widths, fcols = case
    d = _random_case(sum(map(ord, name)), N, D, dtype, m, R, 48, fcols)
    orc, gpu, g = make_pair(d)
    assert orc.entry == gpu.entry
    for mode in ("restart", "resume"):
        for eps in (0.05, 0.3):
            o = orc.search(d["queries"], d["lo"], d["hi"], k, widths, eps=eps, mode=mode, dist_mode=1)
            r = gpu_search(gpu, g, k, widths, mode=mode, eps=eps)
            assert_bit_parity(o, r, f"{name}/{mode}/eps={eps}")
        o = orc.search(d["queries"], d["lo"], d["hi"], k, widths, mode=mode, dist_mode=1, expand_w=2)
        r = gpu_search(gpu, g, k, widths, mode=mode, expand_w=2)
        assert_bit_parity(o, r, f"{name}/{mode}/W=2")
        lam = 40.0 if dtype == "f32" else 30000.0
        o = orc.search(d["queries"], d["lo"], d["hi"], k, widths, mode=mode, dist_mode=1, lam=lam)
        r = gpu_search(gpu, g, k, widths, mode=mode, lam=lam)
        assert_bit_parity(o, r, f"{name}/{mode}/lambda={lam}")
    assert (r["ids"] != SENTINEL).any()
    gpu.close()


@pytest.mark.parametrize("D", [128, 48, 256, 192, 272])
def test_byte_rows_with_queries_of_every_kind(D):
    """uint8 rows take an integer dot-product path when the query is itself byte-valued and
    the fp32 path otherwise; both must equal the oracle's fixed-order fp32 distance bit for
    bit.  The batch mixes whole-number queries, fractional ones, values outside 0..255, one
    fractional element at the very end, and the two extreme rows (all 0 against all 255: the
    largest distance, D * 255^2, still below 2^24 at D = 256)."""
    N, Q, m, R = 3000, 64, 2, 24
    d = _random_case(77 + D, N, D, "u8", m, R, Q)
    rng = np.random.default_rng(D)
    d["vectors"][0] = 0
    d["vectors"][1] = 255
    q = d["queries"]
    q[0] = 255.0
    q[1] = 0.0
    q[8:24] += rng.random((16, D)).astype(np.float32)           # fractional everywhere
    q[24, -1] += 0.25                                             # one fractional element, last lane
    q[25, 0] = 256.0                                              # just outside the byte range
    q[26, D // 2] = -1.0
    q[27] = -q[27]                                                # all negative (and -0.0)
    q[28, 3] = np.float32(1e-30)                                  # tiny, not a whole number
    q[29] = q[29] * 4.0                                           # whole numbers up to 1020
    d["lo"][:, :] = np.iinfo(np.int32).min                        # every point valid: distances decide
    d["hi"][:, :] = np.iinfo(np.int32).max
    d["hi"][32:, 0] = 500                                         # and a filtered half
    orc, gpu, g = make_pair(d, entry=0)
    for mode, widths in (("restart", [16, 64]), ("resume", [12, 300])):
        o = orc.search(q, d["lo"], d["hi"], 10, widths, eps=0.1, mode=mode, dist_mode=1)
        r = gpu_search(gpu, g, 10, widths, mode=mode, eps=0.1)
        assert_bit_parity(o, r, f"u8 D={D} {mode}")
    # the entry point alone (no expansion allowed): the all-zero row against the all-255
    # query is the largest distance there is, and must come out exactly
    r = gpu_search(gpu, g, 1, [1], cap=(0, 0), sel=slice(0, 2))
    o = orc.search(q[:2], d["lo"][:2], d["hi"][:2], 1, [1], cap=(0, 0), dist_mode=1)
    assert_bit_parity(o, r, f"u8 D={D} entry only")
    assert r["ids"][:, 0].tolist() == [0, 0]
    assert r["d2"][:, 0].tolist() == [D * 255.0 ** 2, 0.0] and orc.dist2_f64(q[0], 0) == D * 255.0 ** 2
    gpu.close()


def test_degenerate_sizes():
    """One point, two points, one query, every neighbour slot empty."""
    for N in (1, 2, 5):
        x = np.arange(N * 8, dtype=np.float32).reshape(N, 8)
        g = np.full((N, 3), SENTINEL, dtype=np.uint32)
        if N > 1:
            g[:, 0] = (np.arange(N) + 1) % N
        d = dict(vectors=x, attrs=np.arange(N, dtype=np.int32)[:, None], attr_types=np.zeros(1, np.int32),
                 graph=g, queries=np.ones((1, 8), np.float32), lo=np.array([[0]], np.int32),
                 hi=np.array([[3]], np.int32))
        orc, gpu, gg = make_pair(d)
        for mode in ("restart", "resume"):
            o = orc.search(d["queries"], d["lo"], d["hi"], 2, [2, 8], mode=mode, dist_mode=1)
            r = gpu_search(gpu, gg, 2, [2, 8], mode=mode)
            assert_bit_parity(o, r, f"N={N}/{mode}")
        assert r["ids"][0, 0] == 0
        gpu.close()


def test_many_random_small_cases():
    """Thirty seeded random shapes (dimension, element type, attribute count and types,
    degree, k, widths, ε, mode, BOA+, expansion width, λ, table format), each against the oracle
    bit for bit."""
    rng = np.random.default_rng(2024)
    for case in range(30):
        dtype = "u8" if rng.random() < 0.4 else "f32"
        D = int(rng.integers(1, 9)) * (16 if dtype == "u8" else 4)
        m = int(rng.integers(1, 9))
        R = int(rng.integers(2, 65))
        N = int(rng.integers(R + 2, 1500))
        fcols = tuple(j for j in range(m) if rng.random() < 0.3)
        d = _random_case(1000 + case, N, D, dtype, m, R, 24, fcols)
        k = int(rng.integers(1, 12))
        L0 = int(rng.integers(k, k + 20))
        widths = sorted({L0, L0 + int(rng.integers(1, 100)), L0 + int(rng.integers(100, 600))})
        mode = "resume" if rng.random() < 0.5 else "restart"
        eps = float(rng.choice([0.02, 0.1, 0.4]))
        plus_k = int(rng.choice([0, 0, 3]))
        orc, gpu, g = make_pair(d)
        gpu.set_param("table_tags", 16 if case % 2 else 0)       # both bucket formats
        for ew in (1, 2):
            if ew == 2:
                gpu.set_param("table_kb", int(rng.choice([0, 1])))   # a 1 KB table forgets at once
            lam = float(rng.choice([np.inf, np.inf, 0.0, 3.0, 20000.0]))
            o = orc.search(d["queries"], d["lo"], d["hi"], k, widths, eps=eps, mode=mode, dist_mode=1,
                           expand_w=ew, lam=lam)
            r = gpu_search(gpu, g, k, widths, mode=mode, eps=eps, plus_k=plus_k, expand_w=ew, lam=lam)
            assert_bit_parity(o, r, f"case {case}: {dtype} D={D} m={m} R={R} N={N} k={k} {widths} "
                                    f"{mode} W={ew} lambda={lam}")
        gpu.close()
