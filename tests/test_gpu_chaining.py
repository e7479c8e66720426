"""Launch chaining (programmatic dependent launch) changes when kernels are placed, never what they
compute: the same calls with chaining off and on give the same bytes, and those are the oracle's."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu


def one_step(n, d, s, code_kind, K, eta):
    dev = torch.device("cuda", 0)
    status = Q.new_status(dev)
    cap = Q.qsgd_message_capacity(n, d, s, code_kind)
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device=dev)
    msgs = [torch.zeros(cap, dtype=torch.uint8, device=dev) for _ in range(K)]
    infos = [torch.zeros(4, dtype=torch.int64, device=dev) for _ in range(K)]
    gs = [torch.from_numpy(I.gaussian_mixture(n, seed=20 + w)).to(dev) for w in range(K)]
    x = torch.from_numpy(I.gaussian(n, 1.0, seed=5)).to(dev)
    # back to back on one stream, nothing in between: the order of reads and writes (the shared
    # workspace, the messages, x) rests on every kernel's own wait for the kernel ahead of it
    for rep in range(2):
        for w in range(K):
            Q.qsgd_encode(gs[w], d, s, O.NORM_MAX, code_kind, 7, 4 + rep, w, msgs[w], infos[w], ws, status)
        Q.qsgd_decode_sgd_step_packed(msgs, None if code_kind == O.CODE_FIXED else infos, n, d, s, code_kind, x, eta,
                                      status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return [m.cpu().numpy() for m in msgs], [[int(v) for v in i.cpu()] for i in infos], x.cpu().numpy()


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE])
@pytest.mark.parametrize("d", [512, 4096])
def test_chaining_on_and_off_give_the_oracles_bytes(code_kind, d):
    n, s, K, eta = 4096 * 37 + 520, 15, 3, 0.1
    got = {}
    try:
        for on in (False, True):
            Q.qsgd_set_launch_chaining(on)
            got[on] = one_step(n, d, s, code_kind, K, eta)
    finally:
        assert Q.qsgd_set_launch_chaining(True) is True      # the last setting made above
    for a, b in zip(got[False][0], got[True][0]):
        assert np.array_equal(a, b)
    assert got[False][1] == got[True][1]
    assert np.array_equal(got[False][2].view(np.uint32), got[True][2].view(np.uint32))

    # the oracle: two steps of K encodes and one fused decode each
    x = I.gaussian(n, 1.0, seed=5)
    elias = code_kind != O.CODE_FIXED
    for rep in range(2):
        ref_msgs, ref_tabs = [], []
        for w in range(K):
            m, info = O.encode(I.gaussian_mixture(n, seed=20 + w), d, s, O.NORM_MAX, code_kind, 7, 4 + rep, w)
            ref_msgs.append(m)
            ref_tabs.append(O.message_table(m, info, n, d) if elias else None)
            if rep == 1:
                assert np.array_equal(got[True][0][w][: m.size], m)
                if elias:
                    assert got[True][1][w] == info
        st, acc = O.decode_accumulate(ref_msgs, ref_tabs if elias else None, n, d, s, code_kind)
        assert st == 0
        x = O.sgd_step(x, acc, eta, K)
    assert np.array_equal(got[True][2].view(np.uint32), x.view(np.uint32))
