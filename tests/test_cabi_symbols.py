"""The shared library loads without a GPU, exports every function include/boa.h
declares, and rejects bad arguments on the host before touching CUDA."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_16175_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "boa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(boa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"boa_index_create", "boa_search", "boa_index_destroy", "boa_get_stats"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_null_handling(lib):
    assert lib.boa_strerror(0) == b"ok"
    assert b"invalid" in lib.boa_strerror(-1)
    assert lib.boa_index_destroy(None) == 0
    assert lib.boa_set_param(None, 0, 0.1) == -1
    assert lib.boa_search(None, None, 1, None, None, 10, 16, 64, None, None, None) == -1
    assert lib.boa_last_launch_count(None) == 0


def test_create_rejects_bad_shapes_before_any_cuda_call(lib):
    h = C.c_void_p()
    types = (C.c_int * 2)(0, 0)
    fake = C.c_void_p(4096)          # aligned, never dereferenced on these paths
    def create(N=100, D=16, m=2, R=8, dt=0, entry=-1, vec=fake, t=types):
        return lib.boa_index_create(C.byref(h), vec, dt, N, D, fake, t, m, fake, R, entry, None)
    assert create(N=0) == -1
    assert create(N=(1 << 28) + 1) == -1
    assert create(D=6) == -1                   # floats: D % 4
    assert create(D=24, dt=1) == -1            # bytes: D % 16
    assert create(m=0) == -1 and create(m=9) == -1
    assert create(R=0) == -1 and create(R=65) == -1
    assert create(dt=7) == -1
    assert create(entry=100) == -1
    assert create(vec=C.c_void_p(4100)) == -1  # misaligned
    assert create(t=(C.c_int * 2)(0, 5)) == -1
    assert lib.boa_index_create(None, fake, 0, 100, 16, fake, types, 2, fake, 8, -1, None) == -1


def test_graph_build_rejects_bad_arguments_before_any_cuda_call(lib):
    lib.boa_graph_build.restype = C.c_int
    lib.boa_graph_build.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                    C.c_float, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_void_p,
                                    C.c_void_p, C.c_void_p]
    fake = C.c_void_p(4096)
    th = (C.c_float * 6)(float("inf"), float("inf"), 0.3, 0.3, 0.05, 0.05)
    def build(vec=fake, dt=0, N=1000, D=16, pos=fake, m=2, R=16, Lb=32, alpha=1.2, t=th, T=3, B=256, passes=1,
              cap_in=16, out=fake):
        return lib.boa_graph_build(vec, dt, N, D, pos, m, R, Lb, alpha, t, T, B, passes, cap_in, -1, out, None, None)
    assert build(vec=None) == -1 and build(pos=None) == -1 and build(t=None) == -1 and build(out=None) == -1
    assert build(N=0) == -1
    assert build(R=0) == -1 and build(R=65) == -1
    assert build(Lb=0) == -1 and build(Lb=129) == -1
    assert build(T=0) == -1 and build(T=9) == -1
    assert build(m=0) == -1 and build(m=9) == -1
    assert build(B=0) == -1 and build(passes=0) == -1 and build(passes=5) == -1
    assert build(cap_in=0) == -1 and build(cap_in=65) == -1
    assert build(alpha=0.9) == -1
    assert build(Lb=96, T=3, R=32) == -1       # T*Lb + R beyond the candidate buffer
    assert build(dt=7) == -1
