"""The library's calls only enqueue work on the caller's stream, so a whole step (K encodes, decode +
aggregate + SGD step) can be captured in a CUDA graph and replayed: results equal the eager ones."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_step_replays_from_a_cuda_graph(code_kind):
    n, d, s, K, eta = 2 ** 16 + 100, 512, 15, 4, 0.1
    B = O.n_buckets(n, d)
    g = [torch.from_numpy(I.gaussian(n, 0.01, seed=1 + w)).cuda() for w in range(K)]
    cap = Q.qsgd_message_capacity(n, d, s, code_kind)
    msgs = [torch.zeros(cap, dtype=torch.uint8, device="cuda") for _ in range(K)]
    bits = torch.zeros(K, 4, dtype=torch.int64, device="cuda")
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device="cuda")
    status = Q.new_status()
    x = torch.zeros(n, dtype=torch.float32, device="cuda")

    def encode_all(stream=None):
        for w in range(K):
            Q.qsgd_encode(g[w], d, s, O.NORM_L2, code_kind, 7, 0, w, msgs[w], bits[w], ws, status, stream=stream)

    def tables():
        if code_kind == O.CODE_FIXED:
            return None
        info = bits.cpu().numpy().view(np.uint64)
        return [msgs[w][int(info[w, 1]): int(info[w, 1]) + 8 * (B + 1)].view(torch.int64) for w in range(K)]

    # eager pass: also fixes the table positions (the inputs do not change between replays)
    encode_all()
    tabs = tables()
    Q.qsgd_decode_sgd_step(msgs, tabs, n, d, s, code_kind, x, eta, status)
    torch.cuda.synchronize()
    x_eager = x.clone()
    msgs_eager = [m.clone() for m in msgs]

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    for m in msgs:
        m.zero_()
    x.zero_()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        encode_all(stream=side)
        Q.qsgd_decode_sgd_step(msgs, tabs, n, d, s, code_kind, x, eta, status, stream=side)
    for _ in range(3):                                     # three replays: x moves three steps
        graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for a, b in zip(msgs, msgs_eager):
        assert torch.equal(a, b)
    x3 = x_eager.clone()
    acc = torch.zeros(n, dtype=torch.float32, device="cuda")
    Q.qsgd_decode_accumulate(msgs, tabs, n, d, s, code_kind, acc, status)
    Q.qsgd_sgd_step(x3, acc, eta, K)
    Q.qsgd_sgd_step(x3, acc, eta, K)
    torch.cuda.synchronize()
    assert torch.equal(x, x3)
