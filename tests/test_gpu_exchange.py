"""Algorithm 1's exchange step on the device: GPU encode into exchange slots -> all-gather over an
NCCL group (world size 1: this run has one GPU; slots, pitch, info gather and the packed decode are
the same code at any world size) -> GPU decode of the K gathered messages, against the oracle."""
import numpy as np
import pytest
import torch
import torch.distributed as dist

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import exchange as X, inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nccl_group(tmp_path_factory):
    store = dist.FileStore(str(tmp_path_factory.mktemp("pg") / "store"), 1)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", store=store, rank=0, world_size=1, device_id=torch.device("cuda", 0))
    yield
    dist.destroy_process_group()


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE])
@pytest.mark.parametrize("exact", [False, True])
def test_encode_exchange_decode_matches_oracle(nccl_group, code_kind, exact):
    n, d, s, W, eta = 9 * 4096 + 700, 512, 15, 3, 0.1
    dev = torch.device("cuda", 0)
    ex = X.Exchange(Q.qsgd_message_capacity(n, d, s, code_kind), W, dev)
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device=dev)
    status = Q.new_status(dev)
    gs = [I.gaussian_mixture(n, seed=20 + w) for w in range(W)]
    for w in range(W):
        out, info = ex.local_slot(w)
        Q.qsgd_encode(torch.from_numpy(gs[w]).to(dev), d, s, O.NORM_MAX, code_kind, 7, 4, w, out, info, ws, status)
    elias = code_kind != O.CODE_FIXED
    msgs, infos, nbytes = ex.run(exact=exact and elias, with_info=elias)
    x = torch.from_numpy(I.gaussian(n, 1.0, seed=5)).to(dev)
    x0 = x.cpu().numpy().copy()
    Q.qsgd_decode_sgd_step_packed(msgs, infos if elias else None, n, d, s, code_kind, x, eta, status, msg_bytes=nbytes)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the oracle, message by message (max-norm scales are exact on both sides)
    ref_msgs, ref_tabs = [], []
    for w in range(W):
        m, info = O.encode(gs[w], d, s, O.NORM_MAX, code_kind, 7, 4, w)
        got = msgs[w][: m.size].cpu().numpy()
        assert np.array_equal(got, m), "gathered slot %d differs from the oracle's message" % w
        if elias:
            assert [int(v) for v in infos[w].cpu()] == info
        ref_msgs.append(m)
        ref_tabs.append(O.message_table(m, info, n, d) if elias else None)
    st, acc = O.decode_accumulate(ref_msgs, ref_tabs if elias else None, n, d, s, code_kind)
    x_ref = O.sgd_step(x0, acc, eta, W)
    assert np.array_equal(x.cpu().numpy().view(np.uint32), x_ref.view(np.uint32))


def test_exchange_random_shapes(nccl_group):
    """Drawn shapes through slots, all-gather and the packed decode (capacity and exact slots in turn)."""
    rng = np.random.default_rng(77)
    dev = torch.device("cuda", 0)
    for case in range(14):
        d = int(rng.choice([32, 128, 512, 1024, 4096, 32 * int(rng.integers(1, 60))]))
        n = int(rng.integers(1, 40)) * d - int(rng.integers(0, d))
        n = max(n, 1)
        s = int(rng.choice([1, 3, 15, 64, 255]))
        W = int(rng.integers(1, 7))
        code_kind = int(rng.choice([O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE]))
        norm_kind = O.NORM_MAX
        elias = code_kind != O.CODE_FIXED
        exact = bool(case % 2) and elias
        ex = X.Exchange(Q.qsgd_message_capacity(n, d, s, code_kind), W, dev)
        ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device=dev)
        status = Q.new_status(dev)
        gs = [I.gaussian_mixture(n, seed=1000 + 10 * case + w) for w in range(W)]
        for w in range(W):
            out, info = ex.local_slot(w)
            Q.qsgd_encode(torch.from_numpy(gs[w]).to(dev), d, s, norm_kind, code_kind, 9, case, w, out, info, ws, status)
        msgs, infos, nbytes = ex.run(exact=exact, with_info=elias)
        x0 = I.gaussian(n, 1.0, seed=5 + case)
        x = torch.from_numpy(x0.copy()).to(dev)
        Q.qsgd_decode_sgd_step_packed(msgs, infos if elias else None, n, d, s, code_kind, x, 0.2, status, msg_bytes=nbytes)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (case, n, d, s, W, code_kind)
        ref_msgs, ref_tabs = [], []
        for w in range(W):
            m, info = O.encode(gs[w], d, s, norm_kind, code_kind, 9, case, w)
            assert np.array_equal(msgs[w][: m.size].cpu().numpy(), m), (case, w)
            ref_msgs.append(m)
            ref_tabs.append(O.message_table(m, info, n, d) if elias else None)
        st, acc = O.decode_accumulate(ref_msgs, ref_tabs if elias else None, n, d, s, code_kind)
        assert st == 0
        assert np.array_equal(x.cpu().numpy().view(np.uint32), O.sgd_step(x0, acc, 0.2, W).view(np.uint32)), (case, n, d, s, W)
