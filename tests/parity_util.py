"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding and the CPU
oracle on the same bytes and compare bit for bit."""
import numpy as np
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O

CANARY = 0xAB


def gpu_encode(g_dev, d, s, norm_kind, code_kind, seed, step, worker, capacity=None):
    """Encode on the GPU into a canary-guarded buffer. Returns (message bytes as numpy, info
    list, status int, raw capacity)."""
    n = g_dev.numel()
    cap = Q.qsgd_message_capacity(n, d, s, code_kind) if capacity is None else capacity
    big = torch.full((cap + 256,), CANARY, dtype=torch.uint8, device=g_dev.device)
    out = big[:cap]
    bits = torch.zeros(4, dtype=torch.int64, device=g_dev.device)
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8,
                     device=g_dev.device)
    status = Q.new_status(g_dev.device)
    Q.qsgd_encode(g_dev, d, s, norm_kind, code_kind, seed, step, worker, out, bits, ws, status)
    torch.cuda.synchronize()
    info = [int(v) for v in bits.cpu().numpy().view(np.uint64)]
    assert bool((big[cap:] == CANARY).all()), "write past the message capacity"
    st = int(status.item())
    if st == 0:
        assert info[2] <= cap
        assert bool((big[info[2]:cap] == CANARY).all()), "write past the message length"
    return big, info, st, cap


def scales_from_message(msg, info, n, d, s, code_kind):
    B = O.n_buckets(n, d)
    if code_kind == O.CODE_FIXED:
        return msg[: 4 * B].view(np.float32).copy()
    table = O.message_table(msg, info, n, d)
    st, A, _, _ = O.elias_unpack(msg[: info[1]], table, n, d, s, dense=(code_kind == O.CODE_ELIAS_DENSE))
    assert st == 0, "oracle cannot parse the GPU stream (status %d)" % st
    return A


def check_scales(A_gpu, g, d, norm_kind):
    A_ref = O.bucket_scales(g, d, norm_kind)
    if norm_kind == O.NORM_MAX:
        assert np.array_equal(A_gpu.view(np.uint32), A_ref.view(np.uint32))
    else:
        assert np.all(np.abs(A_gpu.astype(np.float64) - A_ref) <= 1e-6 * A_ref)
        assert np.array_equal(A_gpu == 0, A_ref == 0)


def encode_parity(g, d, s, norm_kind, code_kind, seed, step, worker):
    """GPU message == oracle message given the GPU's scales. Returns (GPU message tensor view
    trimmed to its length, info)."""
    n = g.size
    g_dev = torch.from_numpy(g).cuda()
    big, info, st, cap = gpu_encode(g_dev, d, s, norm_kind, code_kind, seed, step, worker)
    assert st == 0
    msg = big[: info[2]].cpu().numpy()
    A_gpu = scales_from_message(msg, info, n, d, s, code_kind)
    check_scales(A_gpu, g, d, norm_kind)
    ref, ref_info = O.encode(g, d, s, norm_kind, code_kind, seed, step, worker, A_ext=A_gpu)
    assert info == ref_info, (info, ref_info)
    assert np.array_equal(msg, ref), "encoded stream differs from the oracle's"
    # determinism: a second run gives the same bytes
    big2, info2, st2, _ = gpu_encode(g_dev, d, s, norm_kind, code_kind, seed, step, worker)
    assert st2 == 0 and info2 == info and torch.equal(big2[: info[2]], big[: info[2]])
    return big[: info[2]], info


def table_view(msg_dev, info, n, d):
    B = O.n_buckets(n, d)
    return msg_dev[info[1]: info[1] + 8 * (B + 1)].view(torch.int64)


def decode_parity(msgs_dev, infos, n, d, s, code_kind, eta=0.1, x0=None, tables_first=False):
    """GPU decode+aggregate and SGD step (fused and unfused) == oracle, bit for bit. With
    tables_first each offset table is handed over in front of its payload instead of behind it, so
    the library cannot read the payload size off the two pointers."""
    K = len(msgs_dev)
    dev = msgs_dev[0].device
    tables = None if code_kind == O.CODE_FIXED else [table_view(m, i, n, d) for m, i in zip(msgs_dev, infos)]
    if tables_first and tables is not None:
        moved_msgs, moved_tables = [], []
        for m, t, i in zip(msgs_dev, tables, infos):
            tb = t.numel() * 8
            front = (tb + 15) // 16 * 16
            buf = torch.zeros(front + i[1] + 16, dtype=torch.uint8, device=dev)
            buf[:tb] = t.view(torch.uint8)
            buf[front: front + i[1]] = m[: i[1]]
            moved_tables.append(buf[:tb].view(torch.int64))
            moved_msgs.append(buf[front:])
        msgs_dev, tables = moved_msgs, moved_tables
    status = Q.new_status(dev)
    acc = torch.full((n + 64,), 7.0, dtype=torch.float32, device=dev)
    Q.qsgd_decode_accumulate(msgs_dev, tables, n, d, s, code_kind, acc[:n], status)
    x0 = np.zeros(n, np.float32) if x0 is None else x0
    x_unf = torch.from_numpy(x0.copy()).cuda()
    Q.qsgd_sgd_step(x_unf, acc[:n], eta, K)
    xf = torch.full((n + 64,), 3.0, dtype=torch.float32, device=dev)
    xf[:n] = torch.from_numpy(x0).cuda()
    Q.qsgd_decode_sgd_step(msgs_dev, tables, n, d, s, code_kind, xf[:n], eta, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((acc[n:] == 7.0).all()) and bool((xf[n:] == 3.0).all())
    if not tables_first:
        # the packed form (tables found on the device from the info words) gives the same bits
        info_dev = [torch.tensor([int(v) for v in i], dtype=torch.int64, device=dev) for i in infos]
        acc_p = torch.full((n + 64,), 7.0, dtype=torch.float32, device=dev)
        xp = torch.full((n + 64,), 3.0, dtype=torch.float32, device=dev)
        xp[:n] = torch.from_numpy(x0).cuda()
        Q.qsgd_decode_accumulate_packed(msgs_dev, info_dev, n, d, s, code_kind, acc_p[:n], status)
        Q.qsgd_decode_sgd_step_packed(msgs_dev, info_dev, n, d, s, code_kind, xp[:n], eta, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(acc_p.view(torch.int32), acc.view(torch.int32))
        assert torch.equal(xp.view(torch.int32), xf.view(torch.int32))
    msgs = [m.cpu().numpy() for m in msgs_dev]
    tabs = None if tables is None else [t.cpu().numpy().view(np.uint64) for t in tables]
    st, acc_ref = O.decode_accumulate(msgs, tabs, n, d, s, code_kind)
    assert st == 0
    assert np.array_equal(acc[:n].cpu().numpy().view(np.uint32), acc_ref.view(np.uint32))
    x_ref = O.sgd_step(x0, acc_ref, eta, K)
    assert np.array_equal(x_unf.cpu().numpy().view(np.uint32), x_ref.view(np.uint32))
    assert np.array_equal(xf[:n].cpu().numpy().view(np.uint32), x_ref.view(np.uint32))
    return acc_ref, x_ref
