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

# (n, d, s, input): one shape per Elias decoder -- whole-bucket fields (d < 1024), fields by ranges
# (d >= 1024), and the entry-list decoder of the sparse regime (short strings)
SHAPES = [(4096 + 300, 512, 3, "gauss"), (2 * 4096 + 300, 4096, 3, "gauss"), (3 * 4096 + 300, 4096, 1, "sparse")]


@pytest.fixture(params=SHAPES, ids=["fields", "ranged", "sparse"])
def shape(request):
    return request.param


def gradient(shape, seed):
    n, _, _, kind = shape
    return I.gaussian(n, 1.0, seed=seed) if kind == "gauss" else I.sparse_laplace(n, 1e-3, 0.3, seed=seed)


def good_message(shape, code_kind=O.CODE_ELIAS, seed=5):
    _, d, s, _ = shape
    m, info = O.encode(gradient(shape, seed), d, s, O.NORM_L2, code_kind, 7, 0, 0)
    return m, info


def run_decode(shape, msg_np, info, code_kind=O.CODE_ELIAS, table_np=None, s=None, n=None, payload_bytes=None):
    """Decode one (possibly corrupted) message on the GPU; returns (status, acc, guard ok)."""
    d = shape[1]
    s = shape[2] if s is None else s
    n = shape[0] if n is None else n
    B = O.n_buckets(n, d)
    buf = torch.from_numpy(np.concatenate([msg_np, np.zeros(64, np.uint8)])).cuda()
    if table_np is None:
        table = buf[info[1]: info[1] + 8 * (B + 1)].view(torch.int64)
    else:
        table = torch.from_numpy(table_np.view(np.int64)).cuda()
    acc = torch.full((n + 256,), 7.0, dtype=torch.float32, device="cuda")
    status = Q.new_status()
    pb = None if payload_bytes is None else [payload_bytes]
    Q.qsgd_decode_accumulate([buf], [table], n, d, s, code_kind, acc[:n], status, payload_bytes=pb)
    x = torch.full((n + 256,), 3.0, dtype=torch.float32, device="cuda")
    status2 = Q.new_status()
    Q.qsgd_decode_sgd_step([buf], [table], n, d, s, code_kind, x[:n], 0.5, status2, payload_bytes=pb)
    torch.cuda.synchronize()
    guard = bool((acc[n:] == 7.0).all()) and bool((x[n:] == 3.0).all())
    assert (int(status.item()) != 0) == (int(status2.item()) != 0)
    return int(status.item()) | int(status2.item()), acc[:n].cpu().numpy(), guard


def test_well_formed_stream_has_clean_status(shape):
    n, d, s, _ = shape
    m, info = good_message(shape)
    st, acc, guard = run_decode(shape, m, info)
    ref = O.decode(m, O.message_table(m, info, n, d), n, d, s, O.CODE_ELIAS)[1]
    assert st == 0 and guard and np.array_equal(acc.view(np.uint32), ref.view(np.uint32))


def test_truncated_bucket_is_flagged(shape):
    n, d, s, _ = shape
    m, info = good_message(shape)
    t = O.message_table(m, info, n, d).copy()
    t[2] -= 5                                    # bucket 1 loses its last 5 bits (bucket 2 starts early)
    st, _, guard = run_decode(shape, m, info, table_np=t)
    assert st != 0 and guard
    assert O.elias_unpack(m[: info[1]], t, n, d, s)[0] != 0        # the oracle rejects it too


def test_offsets_not_ascending_and_short_bucket(shape):
    n, d, s, _ = shape
    m, info = good_message(shape)
    t = O.message_table(m, info, n, d).copy()
    t[1], t[2] = t[2], t[1]
    st, _, guard = run_decode(shape, m, info, table_np=t)
    assert st & Q.binding.DEV_TABLE and guard
    t = O.message_table(m, info, n, d).copy()
    t[1] = t[0] + 8                              # shorter than the 32-bit scale
    st, _, guard = run_decode(shape, m, info, table_np=t)
    assert st != 0 and guard


def test_table_claiming_more_payload_than_there_is(shape):
    """A table kept apart from its message whose last entry overstates the payload: with the payload
    length given, every string of that message is refused before a single payload bit is read."""
    n, d, s, _ = shape
    m, info = good_message(shape)
    t = O.message_table(m, info, n, d).copy()
    t[-1] += 1 << 33                              # the last bucket now "ends" a gigabyte past the buffer
    st, acc, guard = run_decode(shape, m, info, table_np=t, payload_bytes=info[1])
    assert st & Q.binding.DEV_TABLE and guard
    # the honest table with the same bound decodes cleanly
    st, acc, guard = run_decode(shape, m, info, table_np=O.message_table(m, info, n, d).copy(), payload_bytes=info[1])
    ref = O.decode(m, O.message_table(m, info, n, d), n, d, s, O.CODE_ELIAS)[1]
    assert st == 0 and guard and np.array_equal(acc.view(np.uint32), ref.view(np.uint32))


def test_packed_form_rejects_bad_table_places(shape):
    """Packed decode reads the table's place from the info words on the device: a place that is
    misaligned, or whose table would not fit in the bytes declared readable, is refused."""
    n, d, s, _ = shape
    m, info = good_message(shape)
    buf = torch.from_numpy(np.concatenate([m, np.zeros(64, np.uint8)])).cuda()
    for bad_info, nbytes in (([info[0], info[1] + 8, info[2], 0], buf.numel()),       # not 16-byte aligned
                             ([info[0], info[1], info[2], 0], info[2] - 16),            # table cut off
                             ([info[0], 1 << 40, info[2], 0], buf.numel())):           # far outside
        iw = torch.tensor(bad_info, dtype=torch.int64, device="cuda")
        acc = torch.full((n + 256,), 7.0, dtype=torch.float32, device="cuda")
        status = Q.new_status()
        Q.qsgd_decode_accumulate_packed([buf], [iw], n, d, s, O.CODE_ELIAS, acc[:n], status, msg_bytes=[nbytes])
        torch.cuda.synchronize()
        assert int(status.item()) & Q.binding.DEV_TABLE
        assert bool((acc[n:] == 7.0).all())


def test_level_above_s_is_flagged(shape):
    n, d, s, _ = shape
    s_sent = 15 if s == 3 else 3
    g = gradient(shape, 6)
    norm = O.NORM_MAX
    if shape[3] == "sparse":                      # keep the strings short: one dominant coordinate gets level 3
        g[100] = 1.0
        norm = O.NORM_L2
    m, info = O.encode(g, d, s_sent, norm, O.CODE_ELIAS, 7, 0, 0)         # levels above s occur
    assert O.elias_unpack(m[: info[1]], O.message_table(m, info, n, d), n, d, s)[0] != 0
    st, _, guard = run_decode(shape, m, info)                              # decoder told the smaller s
    assert st & Q.binding.DEV_LEVEL and guard


def test_gap_past_the_bucket_is_flagged(shape):
    # a stream encoded for n coordinates decoded as if the vector ended earlier: the last
    # bucket's positions overshoot the (shorter) tail bucket
    n, d, s, _ = shape
    base = n // d * d
    g = gradient(shape, 7)
    g[base + 250] = 50.0                          # certainly a nonzero beyond position 40
    m, info = O.encode(g, d, s, O.NORM_L2, O.CODE_ELIAS, 7, 0, 0)
    st, _, guard = run_decode(shape, m, info, n=base + 40)
    assert st & (Q.binding.DEV_POSITION | Q.binding.DEV_OVERRUN) and guard


def test_random_garbage_payload_terminates(shape):
    m, info = good_message(shape)
    r = np.random.default_rng(1)
    bad = m.copy()
    bad[: info[1]] = r.integers(0, 256, info[1], dtype=np.uint8)          # table intact, payload noise
    st, _, guard = run_decode(shape, bad, info)
    assert st != 0 and guard
    for kind in (O.CODE_ELIAS_DENSE,):
        m2, info2 = good_message(shape, kind)
        bad = m2.copy()
        bad[: info2[1]] = r.integers(0, 256, info2[1], dtype=np.uint8)
        st, _, guard = run_decode(shape, bad, info2, code_kind=kind)
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
