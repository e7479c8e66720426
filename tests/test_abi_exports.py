"""The C-ABI library loads and exports every symbol include/qsgd.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "qsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qsgd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_1610_02132_b200 import build, binding
    lib = ctypes.CDLL(build.build())
    names = declared_symbols()
    assert len(names) >= 9
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) == set(binding.EXPORTS)


def test_host_side_queries_and_validation():
    import paper_1610_02132_b200 as Q
    from oracle import oracle as O
    for n, d, s in [(2 ** 20, 512, 15), (61100840, 512, 255), (1, 32, 1), (4097, 4096, 3)]:
        assert Q.qsgd_fixed_layout(n, d, s) == O.fixed_layout(n, d, s)
        for kind in (0, 1, 2):
            assert Q.qsgd_message_capacity(n, d, s, kind) == O.message_capacity(n, d, s, kind)
    assert Q.qsgd_message_capacity(2 ** 20, 512, 15, 0) == 663552
    assert Q.qsgd_workspace_bytes(2 ** 20, 512, 15, 0) == 0
    assert Q.qsgd_workspace_bytes(2 ** 20, 512, 15, 1) > 663552
    L = Q.binding.lib()
    # invalid arguments are rejected before any launch (null pointers are never dereferenced)
    assert L.qsgd_encode(None, 10, 512, 15, 0, 0, 0, 0, 0, None, 0, None, None, None, None) == -1
    assert L.qsgd_sgd_step(None, None, 0.1, 4, 10, None) == -1
    assert L.qsgd_sgd_step(16, 16, 0.1, 0, 10, None) == -7
    assert L.qsgd_sgd_step(16, 20, 0.1, 4, 10, None) == -5
    assert L.qsgd_encode(16, 0, 512, 15, 0, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -2
    assert L.qsgd_encode(16, 10, 100, 15, 0, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -3
    assert L.qsgd_encode(16, 10, 512, 256, 0, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -4
    assert L.qsgd_encode(16, 10, 512, 15, 0, 7, 0, 0, 0, 16, 0, 16, None, 16, None) == -8
    assert L.qsgd_encode(16, 10, 512, 15, 5, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -8
    assert L.qsgd_encode(24, 10, 512, 15, 0, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -5
    assert L.qsgd_encode(16, 10, 512, 15, 0, 0, 0, 0, 0, 16, 8, 16, None, 16, None) == -6
    # n beyond 2^32 coordinates is refused by every shape check (16 GiB of gradient per call)
    assert L.qsgd_encode(16, 2 ** 32 + 1, 512, 15, 0, 0, 0, 0, 0, 16, 0, 16, None, 16, None) == -2
    assert Q.qsgd_message_capacity(2 ** 32 + 1, 512, 15, 0) == 0
    assert Q.qsgd_message_capacity(2 ** 32, 512, 15, 0) > 0
    assert L.qsgd_status_string(-3).decode().startswith("bucket")
    assert Q.qsgd_launch_count() == 0
