"""World-size-2 test of the message exchange (rank = worker) on CPU with the gloo backend: each
rank encodes its own gradient (with the oracle, as there is no GPU here), the ranks exchange
messages through paper_1610_02132_b200.exchange, every rank decodes all of them, and both must
end with the same parameters as a single process that holds both messages."""
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


def _worker(rank, world, port, code_kind, n, d, s, result_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle as O
    from paper_1610_02132_b200 import exchange as X, inputs as I
    g = I.gaussian_mixture(n, seed=1 + rank)
    m, info = O.encode(g, d, s, O.NORM_L2, code_kind, 7, 0, rank)
    elias = code_kind != O.CODE_FIXED
    cap = O.message_capacity(n, d, s, code_kind) + X.SLOT_ALIGN
    buf = torch.zeros(cap, dtype=torch.uint8)
    buf[: m.size] = torch.from_numpy(m)
    info_t = torch.tensor(info, dtype=torch.int64)
    msgs, tables, infos = X.exchange(buf, info_t, n, d, elias, fixed_bytes=info[2])
    assert len(msgs) == world and infos.shape == (world, 4)
    assert torch.equal(msgs[rank], torch.from_numpy(m))                 # own slot holds own message
    msgs_np = [x.numpy() for x in msgs]
    tabs_np = None if tables is None else [t.numpy().view(np.uint64) for t in tables]
    st, acc = O.decode_accumulate(msgs_np, tabs_np, n, d, s, code_kind)
    assert st == 0
    x = O.sgd_step(np.zeros(n, np.float32), acc, 0.1, world)
    np.save(os.path.join(result_dir, "x%d.npy" % rank), x)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("code_kind", [0, 1])
def test_two_rank_exchange_matches_single_process(tmp_path, code_kind):
    sys.path.insert(0, ROOT)
    from oracle import oracle as O
    from paper_1610_02132_b200 import inputs as I
    n, d, s, world = 5000, 512, 15, 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, code_kind, n, d, s, str(tmp_path)), nprocs=world, join=True)
    msgs, tabs = [], []
    for w in range(world):
        m, info = O.encode(I.gaussian_mixture(n, seed=1 + w), d, s, O.NORM_L2, code_kind, 7, 0, w)
        msgs.append(m)
        tabs.append(None if code_kind == 0 else O.message_table(m, info, n, d))
    st, acc = O.decode_accumulate(msgs, None if code_kind == 0 else tabs, n, d, s, code_kind)
    ref = O.sgd_step(np.zeros(n, np.float32), acc, 0.1, world)
    for w in range(world):
        x = np.load(os.path.join(str(tmp_path), "x%d.npy" % w))
        assert np.array_equal(x.view(np.uint32), ref.view(np.uint32))


def test_slot_arithmetic():
    from paper_1610_02132_b200 import exchange as X
    assert X.slot_bytes(1) == 256 and X.slot_bytes(256) == 256 and X.slot_bytes(257) == 512
    infos = torch.tensor([[100, 16, 16 + 8 * 3, 0], [70, 16, 16 + 8 * 3, 0]], dtype=torch.int64)
    pitch = X.slot_bytes(40)
    buf = torch.arange(2 * pitch, dtype=torch.int64).to(torch.uint8)
    msgs, tables = X.slots(buf, pitch, infos, n=64, bucket=32, elias=True)
    assert msgs[1].data_ptr() - buf.data_ptr() == pitch and msgs[0].numel() == 40
    assert tables[1].data_ptr() - buf.data_ptr() == pitch + 16 and tables[0].numel() == 3
