"""qsgd_encode_elias_static: the Elias Encode whose scratch is an array built into the library,
for callers that are not allowed to allocate device memory at the point where they encode (a hook
running under a locked framework allocator, a plug-in that owns no allocator, a thread that must
stay out of cudaMalloc). It must produce exactly the message qsgd_encode produces, call after
call, although every call reuses the same scratch and finds the previous call's leftovers in it.

Collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu


def encode_both(g, d, s, norm_kind, code_kind, seed, step, worker):
    n = g.numel()
    cap = Q.qsgd_message_capacity(n, d, s, code_kind)
    outs, infos = [], []
    for static in (False, True):
        out = torch.full((cap,), 0x5A, dtype=torch.uint8, device="cuda")
        bits = torch.zeros(4, dtype=torch.int64, device="cuda")
        status = Q.new_status()
        if static:
            Q.qsgd_encode_elias_static(g, d, s, norm_kind, code_kind, seed, step, worker, out, bits,
                                       status)
        else:
            ws = torch.empty(Q.qsgd_workspace_bytes(n, d, s, code_kind), dtype=torch.uint8, device="cuda")
            Q.qsgd_encode(g, d, s, norm_kind, code_kind, seed, step, worker, out, bits, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append(out)
        infos.append([int(v) for v in bits.cpu().numpy().view(np.uint64)])
    return outs, infos


def test_static_scratch_encode_matches_workspace_encode_twice_in_a_row():
    assert Q.qsgd_static_scratch_bytes() == 32 << 20
    # two calls in a row with different sizes, bucket sizes and code kinds: the second call
    # meets a scratch array full of the first call's data
    cases = [(3 * 4096 + 777, 512, 15, O.NORM_L2, O.CODE_ELIAS, "mix"),
             (50000, 128, 3, O.NORM_MAX, O.CODE_ELIAS_DENSE, "gauss"),
             (2 ** 20, 4096, 1, O.NORM_L2, O.CODE_ELIAS, "sparse")]
    for rep in range(2):
        for i, (n, d, s, norm_kind, code_kind, kind) in enumerate(cases):
            if kind == "mix":
                g = I.gaussian_mixture(n, seed=40 + i + rep)
            elif kind == "gauss":
                g = I.gaussian(n, 0.01, seed=40 + i + rep)
            else:
                g = I.sparse_laplace(n, 1e-3, 0.3, seed=40 + i + rep)
            g = torch.from_numpy(g).cuda()
            (a, b), (ia, ib) = encode_both(g, d, s, norm_kind, code_kind, 7, rep, i)
            assert ia == ib
            assert torch.equal(a[: ia[2]], b[: ib[2]])          # bit-identical messages
            assert bool((b[ib[2]:] == 0x5A).all())              # nothing written past the message


def test_static_scratch_limit_is_enforced():
    n, d, s = 64 * 2 ** 20, 512, 15                             # needs far more than 32 MiB
    assert Q.qsgd_workspace_bytes(n, d, s, O.CODE_ELIAS) > Q.qsgd_static_scratch_bytes()
    g = torch.zeros(16, dtype=torch.float32, device="cuda")     # never read: the call is refused
    L = Q.binding.lib()
    out = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = Q.new_status()
    before = Q.qsgd_launch_count()
    st = L.qsgd_encode_elias_static(g.data_ptr(), n, d, s, 0, O.CODE_ELIAS, 1, 0, 0, out.data_ptr(),
                                    1 << 40, bits.data_ptr(), status.data_ptr(), None)
    assert st == -10 and Q.qsgd_launch_count() == before
    assert b"scratch" in L.qsgd_status_string(st)
    # the fixed-width kind has no scratch and is not served by this entry point
    st = L.qsgd_encode_elias_static(g.data_ptr(), 16, 32, s, 0, O.CODE_FIXED, 1, 0, 0, out.data_ptr(),
                                    1 << 20, bits.data_ptr(), status.data_ptr(), None)
    assert st == -8
