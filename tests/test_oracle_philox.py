"""Pins for the oracle's Philox4x32-10 and its uniform draw (CPU only)."""
import os
import subprocess
import ctypes as C

import numpy as np
import pytest

from oracle import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_known_answer_vectors():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = O.philox(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


@pytest.fixture(scope="module")
def torch_engine(tmp_path_factory):
    """An independent Philox4x32-10: the header-only engine that ships with libtorch."""
    import torch
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    if not os.path.exists(os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")):
        pytest.skip("torch Philox header not present")
    d = tmp_path_factory.mktemp("philox")
    src = d / "pin.cpp"
    src.write_text(
        '#include <ATen/core/PhiloxRNGEngine.h>\n'
        'extern "C" void pin_block(unsigned long long seed, unsigned long long subseq,\n'
        '                          unsigned long long offset, unsigned int* out) {\n'
        '  at::Philox4_32 e(seed, subseq, offset);\n'
        '  for (int j = 0; j < 4; ++j) out[j] = e();\n'
        '}\n')
    so = d / "pin.so"
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-shared", "-fPIC", "-I", inc, str(src),
                           "-o", str(so)])
    L = C.CDLL(str(so))
    L.pin_block.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.POINTER(C.c_uint32)]
    return L


def test_against_independent_engine(torch_engine):
    # engine(seed, subsequence, offset): key = seed, counter = (offset lo, offset hi, subseq lo,
    # subseq hi). The oracle's draw for coordinate i uses counter (q lo, q hi, step, worker),
    # q = i / 4, i.e. subsequence = worker << 32 | step, offset = q.
    r = np.random.default_rng(5)
    out = (C.c_uint32 * 4)()
    for _ in range(3000):
        seed = int(r.integers(0, 2 ** 63)) * 2 + int(r.integers(0, 2))
        step = int(r.integers(0, 2 ** 32))
        worker = int(r.integers(0, 2 ** 32))
        q = int(r.integers(0, 2 ** 40))
        torch_engine.pin_block(seed, (worker << 32) | step, q, out)
        mine = O.philox([q & 0xFFFFFFFF, q >> 32, step, worker], [seed & 0xFFFFFFFF, seed >> 32])
        assert [int(x) for x in mine] == list(out)
        for j in range(4):
            u = O.uniform(seed, step, worker, 4 * q + j)
            assert u == (out[j] >> 8) * 2.0 ** -24


def test_uniform_range_and_moments():
    u = np.array([O.uniform(7, 0, 3, i) for i in range(40000)])
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 5 * (1 / 12 / u.size) ** 0.5
    assert abs(u.var() - 1 / 12) < 2e-3
    # index keyed globally: the draw does not depend on anything but (seed, step, worker, i)
    assert O.uniform(7, 0, 3, 123) == O.uniform(7, 0, 3, 123)
    assert O.uniform(7, 0, 3, 123) != O.uniform(7, 1, 3, 123)
    assert O.uniform(7, 0, 3, 123) != O.uniform(7, 0, 4, 123)
    assert O.uniform(7, 0, 3, 123) != O.uniform(8, 0, 3, 123)
