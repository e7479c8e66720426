"""World-size-2 test of the message exchange on CPU with the gloo backend: each rank encodes the
gradients of the workers it plays (with the oracle, as there is no GPU here), the ranks exchange
slots and info words through paper_1610_02132_b200.exchange, every rank decodes all K messages,
and all must end with the same parameters as a single process that holds every message."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, code_kind, n, d, s, W, exact, result_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle as O
    from paper_1610_02132_b200 import exchange as X, inputs as I
    elias = code_kind != O.CODE_FIXED
    ex = X.Exchange(O.message_capacity(n, d, s, code_kind), W, torch.device("cpu"))
    assert ex.K == world * W and ex.pitch % X.SLOT_ALIGN == 0
    mine = []
    for w in range(W):
        worker = rank * W + w
        m, info = O.encode(I.gaussian_mixture(n, seed=1 + worker), d, s, O.NORM_L2, code_kind, 7, 0, worker)
        buf, iw = ex.local_slot(w)
        buf[: m.size] = torch.from_numpy(m)
        iw.copy_(torch.tensor(info, dtype=torch.int64))
        mine.append(m)
    msgs, infos, nbytes = ex.run(exact=exact, with_info=elias)
    assert len(msgs) == ex.K and len(infos) == ex.K and len(nbytes) == ex.K
    if exact:
        assert nbytes[0] <= ex.pitch and nbytes[0] % X.SLOT_ALIGN == 0
    for w in range(W):                                                   # own slots hold own messages
        k = rank * W + w
        assert torch.equal(msgs[k][: mine[w].size], torch.from_numpy(mine[w]))
    msgs_np, tabs_np = [], []
    for k in range(ex.K):
        total = int(infos[k][2]) if elias else O.message_capacity(n, d, s, code_kind)
        assert total <= nbytes[k]
        m = msgs[k][:total].numpy()
        msgs_np.append(m)
        if elias:
            info = [int(v) for v in infos[k]]
            tabs_np.append(O.message_table(m, info, n, d))
    st, acc = O.decode_accumulate(msgs_np, tabs_np if elias else None, n, d, s, code_kind)
    assert st == 0
    x = O.sgd_step(np.zeros(n, np.float32), acc, 0.1, ex.K)
    np.save(os.path.join(result_dir, "x%d.npy" % rank), x)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("code_kind,W,exact", [(0, 1, False), (1, 1, False), (1, 2, True), (2, 1, True), (0, 2, False)])
def test_two_rank_exchange_matches_single_process(tmp_path, code_kind, W, exact):
    sys.path.insert(0, ROOT)
    from oracle import oracle as O
    from paper_1610_02132_b200 import inputs as I
    n, d, s, world = 5000, 512, 15, 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, code_kind, n, d, s, W, exact, str(tmp_path)), nprocs=world, join=True)
    msgs, tabs = [], []
    for w in range(world * W):
        m, info = O.encode(I.gaussian_mixture(n, seed=1 + w), d, s, O.NORM_L2, code_kind, 7, 0, w)
        msgs.append(m)
        tabs.append(None if code_kind == 0 else O.message_table(m, info, n, d))
    st, acc = O.decode_accumulate(msgs, None if code_kind == 0 else tabs, n, d, s, code_kind)
    ref = O.sgd_step(np.zeros(n, np.float32), acc, 0.1, world * W)
    for r in range(world):
        x = np.load(os.path.join(str(tmp_path), "x%d.npy" % r))
        assert np.array_equal(x.view(np.uint32), ref.view(np.uint32))


def test_slot_arithmetic():
    from paper_1610_02132_b200 import exchange as X
    assert X.slot_bytes(1) == 256 and X.slot_bytes(256) == 256 and X.slot_bytes(257) == 512
