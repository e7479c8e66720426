"""Host threads calling the library at the same time, each on its own stream: the per-device launch
caches and the process-wide settings are the only state they share."""
import threading

import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu

SHAPES = [(9 * 4096 + 100, 512, 15, O.CODE_FIXED), (7 * 4096 + 5, 4096, 1, O.CODE_ELIAS), (50000, 128, 3, O.CODE_ELIAS),
          (33000, 96, 255, O.CODE_FIXED), (40000, 1024, 64, O.CODE_ELIAS_DENSE), (5 * 4096, 256, 7, O.CODE_ELIAS)]


def one_round(shape, worker, stream):
    n, d, s, code_kind = shape
    dev = torch.device("cuda", 0)
    with torch.cuda.stream(stream):
        g = torch.from_numpy(I.gaussian_mixture(n, seed=70 + worker)).to(dev)
        out, bits, status = Q.encode_alloc(g, d, s, O.NORM_MAX, code_kind, 5, 2, worker)
        x = torch.zeros(n, dtype=torch.float32, device=dev)
        Q.qsgd_decode_sgd_step_packed([out], None if code_kind == O.CODE_FIXED else [bits], n, d, s, code_kind, x, -1.0,
                                      status)
        stream.synchronize()
        return out.cpu().numpy(), [int(v) for v in bits.cpu()], x.cpu().numpy(), int(status.item())


def test_threads_on_their_own_streams():
    results, errors = {}, []

    def work(t):
        try:
            stream = torch.cuda.Stream()
            for rep in range(6):
                shape = SHAPES[(t + rep) % len(SHAPES)]
                results[(t, rep)] = (shape, one_round(shape, 10 * t + rep, stream))
        except Exception as e:                         # pragma: no cover
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=(t,)) for t in range(4)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    for (t, rep), (shape, (out, info, x, st)) in results.items():
        n, d, s, code_kind = shape
        assert st == 0
        g = I.gaussian_mixture(n, seed=70 + 10 * t + rep)
        m, ref_info = O.encode(g, d, s, O.NORM_MAX, code_kind, 5, 2, 10 * t + rep)
        assert info == ref_info and np.array_equal(out[: m.size], m)
        tabs = None if code_kind == O.CODE_FIXED else [O.message_table(m, ref_info, n, d)]
        st2, acc = O.decode_accumulate([m], tabs, n, d, s, code_kind)
        assert st2 == 0
        assert np.array_equal(x.view(np.uint32), O.sgd_step(np.zeros(n, np.float32), acc, -1.0, 1).view(np.uint32))
