"""A bounded wait that runs out: the streaming encoder must raise QSGD_DEV_TIMEOUT, stop, wait for
the copies it still has in flight and return, writing nothing outside the message buffer. The
wait is made to run out through the library's test hook (a poll bound of zero for the main-loop
waits; the final drain keeps its full bound), so nothing here faults, traps or hangs."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

from parity_util import CANARY, encode_parity

pytestmark = pytest.mark.gpu


@pytest.fixture
def zero_polls():
    Q.qsgd_test_set_wait_polls(0)
    try:
        yield
    finally:
        Q.qsgd_test_set_wait_polls(Q.qsgd_test_default_wait_polls())


# per-warp rings (d <= 512), per-warp rings with group barriers (d >= 1024, 2-norm: warps of a group
# must stop together), the CTA ring (d >= 1024, max-norm)
@pytest.mark.parametrize("d,code_kind,norm_kind", [(512, O.CODE_FIXED, O.NORM_L2), (128, O.CODE_FIXED, O.NORM_L2),
                                                   (4096, O.CODE_FIXED, O.NORM_L2), (1024, O.CODE_FIXED, O.NORM_L2),
                                                   (4096, O.CODE_FIXED, O.NORM_MAX), (2048, O.CODE_ELIAS, O.NORM_MAX),
                                                   (512, O.CODE_ELIAS, O.NORM_L2)])
def test_wait_gives_up_and_kernel_returns(zero_polls, d, code_kind, norm_kind):
    n, s = 40 * 4096 + 77, 15
    g = torch.from_numpy(I.gaussian(n, 0.01, seed=3)).cuda()
    cap = Q.qsgd_message_capacity(n, d, s, code_kind)
    big = torch.full((cap + 4096,), CANARY, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device="cuda")
    status = Q.new_status()
    Q.qsgd_encode(g, d, s, norm_kind, code_kind, 7, 0, 0, big[:cap], bits, ws, status)
    torch.cuda.synchronize()                                   # the kernels came back
    assert int(status.item()) & Q.binding.DEV_TIMEOUT
    assert bool((big[cap:] == CANARY).all()), "write past the message buffer"
    # the device still answers, and with the default bound the same call is exact again
    Q.qsgd_test_set_wait_polls(Q.qsgd_test_default_wait_polls())
    encode_parity(g.cpu().numpy(), d, s, norm_kind, code_kind, seed=7, step=0, worker=0)


@pytest.mark.parametrize("bucket", [512, 128, 4096])
def test_wait_gives_up_under_policy(zero_polls, bucket):
    # one bucket per chunk, several per chunk (each lane starts its own copy), and the CTA-wide ring
    sizes = [30000, 700, 4096 * 6 + 8, 20000]
    s = 15
    plan = Q.Policy(sizes, bucket)
    g = torch.from_numpy(I.gaussian(sum(sizes), 0.01, seed=4)).cuda()
    cap = Q.qsgd_policy_message_capacity(plan, s, O.CODE_FIXED)
    big = torch.full((cap + 4096,), CANARY, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = Q.new_status()
    Q.qsgd_policy_encode(g, plan, s, O.NORM_L2, O.CODE_FIXED, 7, 0, 0, big[:cap], bits, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) & Q.binding.DEV_TIMEOUT
    assert bool((big[cap:] == CANARY).all())
