"""Negative GPU tests: invalid arguments never launch; malformed Elias streams built on the host
(truncated, gap past the bucket, level above s, offsets not ascending) and undersized message
buffers raise the device status word, write nothing out of bounds, and the kernels return."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu

N, D, S = 4096 + 300, 512, 3


def good_message(code_kind=O.CODE_ELIAS, seed=5):
    g = I.gaussian(N, 1.0, seed=seed)
    m, info = O.encode(g, D, S, O.NORM_L2, code_kind, 7, 0, 0)
    return m, info


def run_decode(msg_np, info, code_kind=O.CODE_ELIAS, table_np=None, s=S, n=N):
    """Decode one (possibly corrupted) message on the GPU; returns (status, acc, guard ok)."""
    B = O.n_buckets(n, D)
    buf = torch.from_numpy(np.concatenate([msg_np, np.zeros(64, np.uint8)])).cuda()
    if table_np is None:
        table = buf[info[1]: info[1] + 8 * (B + 1)].view(torch.int64)
    else:
        table = torch.from_numpy(table_np.view(np.int64)).cuda()
    acc = torch.full((n + 256,), 7.0, dtype=torch.float32, device="cuda")
    status = Q.new_status()
    Q.qsgd_decode_accumulate([buf], [table], n, D, s, code_kind, acc[:n], status)
    torch.cuda.synchronize()
    return int(status.item()), acc[:n].cpu().numpy(), bool((acc[n:] == 7.0).all())


def test_well_formed_stream_has_clean_status():
    m, info = good_message()
    st, acc, guard = run_decode(m, info)
    ref = O.decode(m, O.message_table(m, info, N, D), N, D, S, O.CODE_ELIAS)[1]
    assert st == 0 and guard and np.array_equal(acc.view(np.uint32), ref.view(np.uint32))


def test_truncated_bucket_is_flagged():
    m, info = good_message()
    t = O.message_table(m, info, N, D).copy()
    t[3] -= 5                                    # bucket 2 loses its last 5 bits (bucket 3 starts early)
    st, _, guard = run_decode(m, info, table_np=t)
    assert st != 0 and guard
    assert O.elias_unpack(m[: info[1]], t, N, D, S)[0] != 0        # the oracle rejects it too


def test_offsets_not_ascending_and_short_bucket():
    m, info = good_message()
    t = O.message_table(m, info, N, D).copy()
    t[2], t[3] = t[3], t[2]
    st, _, guard = run_decode(m, info, table_np=t)
    assert st & Q.binding.DEV_TABLE and guard
    t = O.message_table(m, info, N, D).copy()
    t[1] = t[0] + 8                              # shorter than the 32-bit scale
    st, _, guard = run_decode(m, info, table_np=t)
    assert st != 0 and guard


def test_level_above_s_is_flagged():
    g = I.gaussian(N, 1.0, seed=6)
    m, info = O.encode(g, D, 15, O.NORM_MAX, O.CODE_ELIAS, 7, 0, 0)      # levels up to 15
    st, _, guard = run_decode(m, info, s=3)                                # decoder told s = 3
    assert st & Q.binding.DEV_LEVEL and guard


def test_gap_past_the_bucket_is_flagged():
    # a stream encoded for n coordinates decoded as if the vector ended earlier: the last
    # bucket's positions overshoot the (shorter) tail bucket
    n_short = 4096 + 40
    g = I.gaussian(N, 1.0, seed=7)
    g[4096 + 250] = 50.0                          # certainly a nonzero beyond position 40
    m, info = O.encode(g, D, S, O.NORM_L2, O.CODE_ELIAS, 7, 0, 0)
    st, _, guard = run_decode(m, info, n=n_short)
    assert st & (Q.binding.DEV_POSITION | Q.binding.DEV_OVERRUN) and guard


def test_random_garbage_payload_terminates():
    m, info = good_message()
    r = np.random.default_rng(1)
    bad = m.copy()
    bad[: info[1]] = r.integers(0, 256, info[1], dtype=np.uint8)          # table intact, payload noise
    st, _, guard = run_decode(bad, info)
    assert st != 0 and guard
    for kind in (O.CODE_ELIAS_DENSE,):
        m2, info2 = good_message(kind)
        bad = m2.copy()
        bad[: info2[1]] = r.integers(0, 256, info2[1], dtype=np.uint8)
        st, _, guard = run_decode(bad, info2, code_kind=kind)
        assert st != 0 and guard


def test_undersized_message_buffer_sets_capacity_flag():
    n, d, s = 50000, 128, 255
    g = torch.from_numpy(I.gaussian(n, 1.0, seed=2)).cuda()
    B = O.n_buckets(n, d)
    small = 16 * ((4 * B + 15) // 16) + 8 * (B + 1) + 64                   # passes the host check only
    big = torch.full((small + 4096,), 0xAB, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    ws = torch.empty(Q.qsgd_workspace_bytes(n, d, s, O.CODE_ELIAS), dtype=torch.uint8, device="cuda")
    status = Q.new_status()
    Q.qsgd_encode(g, d, s, O.NORM_MAX, O.CODE_ELIAS, 1, 0, 0, big[:small], bits, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) & Q.binding.DEV_CAPACITY
    assert bool((big == 0xAB).all())                                       # nothing was written
    need = int(bits.cpu().numpy().view(np.uint64)[2])
    assert need > small                                                    # the info words say how much is needed


def test_invalid_arguments_launch_nothing():
    g = torch.zeros(1024, dtype=torch.float32, device="cuda")
    out = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = Q.new_status()
    before = Q.qsgd_launch_count()
    for kwargs, code in ((dict(bucket=100), -3), (dict(s=0), -4), (dict(s=256), -4), (dict(code_kind=9), -8),
                         (dict(norm_kind=3), -8)):
        a = dict(bucket=512, s=15, norm_kind=0, code_kind=0)
        a.update(kwargs)
        with pytest.raises(Q.QsgdError) as e:
            Q.qsgd_encode(g, a["bucket"], a["s"], a["norm_kind"], a["code_kind"], 1, 0, 0, out, bits, None, status)
        assert "status %d" % code in str(e.value)
    with pytest.raises(Q.QsgdError):                                       # fixed-width capacity is checked on the host
        Q.qsgd_encode(g, 512, 15, 0, 0, 1, 0, 0, out[:64], bits, None, status)
    with pytest.raises(Q.QsgdError):                                       # misaligned gradient pointer
        Q.qsgd_encode(g[1:], 512, 15, 0, 0, 1, 0, 0, out, bits, None, status, n=1023)
    with pytest.raises(Q.QsgdError):                                       # K out of range
        Q.qsgd_decode_accumulate([out] * 65, None, 1024, 512, 15, 0, g, status)
    assert Q.qsgd_launch_count() == before


def test_sixty_four_peers_and_rerun_determinism():
    n, d, s, K = 30000, 512, 15, 64
    g = torch.from_numpy(I.gaussian_mixture(n, seed=4)).cuda()
    msgs, msgs_np = [], []
    for w in range(K):
        out, bits, status = Q.encode_alloc(g, d, s, O.NORM_L2, O.CODE_FIXED, 3, 1, w)
        msgs.append(out)
    torch.cuda.synchronize()
    status = Q.new_status()
    a1 = torch.empty(n, dtype=torch.float32, device="cuda")
    a2 = torch.empty(n, dtype=torch.float32, device="cuda")
    Q.qsgd_decode_accumulate(msgs, None, n, d, s, O.CODE_FIXED, a1, status)
    Q.qsgd_decode_accumulate(msgs, None, n, d, s, O.CODE_FIXED, a2, status)
    torch.cuda.synchronize()
    assert torch.equal(a1.view(torch.int32), a2.view(torch.int32))
    st, ref = O.decode_accumulate([m.cpu().numpy() for m in msgs], None, n, d, s, O.CODE_FIXED)
    assert np.array_equal(a1.cpu().numpy().view(np.uint32), ref.view(np.uint32))
