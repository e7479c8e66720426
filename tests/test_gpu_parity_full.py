"""GPU parity at the full sizes of the five workloads, in the launch configuration bench.py times.
The small configs are compared whole. The two 60M-coordinate model-shaped configs are compared
whole as well -- the complete messages of the first and the last worker against the oracle's
encoder, and the complete stepped x against the oracle's decoder over all K messages -- and, like
the 2^28-coordinate sweep points, on sampled buckets (first, last / tail, and random ones) that
the oracle recomputes one by one from the same gradient bytes, plus properties that hold at any
size (fused == unfused, table arithmetic, code-length bound)."""
import math

import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

from parity_util import check_scales, decode_parity, encode_parity, gpu_encode, scales_from_message, table_view

pytestmark = pytest.mark.gpu

SEED = 7


def sample_buckets(B, count, seed):
    r = np.random.default_rng(seed)
    pick = set(int(x) for x in r.integers(0, B, size=count))
    pick |= {0, B - 1, B // 2, max(B - 2, 0)}
    return sorted(pick)


def bits_of(words_u32, lo, hi):
    """Stream bits [lo, hi) of an MSB-first u32 word stream as a '0'/'1' string."""
    w0, w1 = lo // 32, (hi + 31) // 32
    s = "".join(format(int(x), "032b") for x in words_u32[w0:w1])
    return s[lo - 32 * w0: hi - 32 * w0]


def fixed_fields(msg, n, d, s, b):
    """Scale, levels and signs of bucket b from a fixed-width message (numpy uint8)."""
    lay = O.fixed_layout(n, d, s)
    lb = lay[3]
    lo, hi = b * d, min((b + 1) * d, n)
    A = msg[4 * b: 4 * b + 4].view(np.float32)[0]
    sw = msg[lay[0]:lay[1]].view(np.uint32)
    lw = msg[lay[1]:lay[2]].view(np.uint32)
    idx = np.arange(lo, hi, dtype=np.int64)
    sg = ((sw[idx // 32] >> (idx % 32).astype(np.uint32)) & 1).astype(np.uint8)
    bit = idx * lb
    lv = ((lw[bit // 32] >> (bit % 32).astype(np.uint32)) & ((1 << lb) - 1)).astype(np.uint8)
    return A, lv, sg


def check_sampled(g_dev, msg_dev, info, n, d, s, norm_kind, code_kind, step, worker, buckets):
    """Per sampled bucket: GPU scale close to / equal to the oracle's, and the bucket's fields or
    string equal to what the oracle produces from the GPU's scale. Returns {b: (A, lv, sg)}."""
    msg = msg_dev[: info[2]].cpu().numpy()
    B = O.n_buckets(n, d)
    out = {}
    if code_kind != O.CODE_FIXED:
        table = O.message_table(msg, info, n, d)
        assert table[0] == 0 and int(table[B]) == info[0]
        assert np.all(np.diff(table.astype(np.int64)) >= 32)
        assert info[1] == (info[0] + 7) // 8 + (-((info[0] + 7) // 8)) % 16
        assert info[2] == info[1] + 8 * (B + 1)
        words = msg[: info[1]].view(np.uint32)
    for b in buckets:
        lo, hi = b * d, min((b + 1) * d, n)
        gb = g_dev[lo:hi].cpu().numpy()
        if code_kind == O.CODE_FIXED:
            A, lv, sg = fixed_fields(msg, n, d, s, b)
        else:
            got = bits_of(words, int(table[b]), int(table[b + 1]))
            A = np.array([int(got[:32], 2)], dtype=np.uint32).view(np.float32)[0]
        A_ref = O.bucket_scales(gb, d, norm_kind)[0]
        if norm_kind == O.NORM_MAX:
            assert np.float32(A).view(np.uint32) == A_ref.view(np.uint32), b
        else:
            assert abs(float(A) - float(A_ref)) <= 1e-6 * float(A_ref), (b, A, A_ref)
        lv_ref, sg_ref = O.quantize(gb, d, s, np.array([A], np.float32), SEED, step, worker, i0=lo)
        if code_kind == O.CODE_FIXED:
            assert np.array_equal(lv, lv_ref) and np.array_equal(sg, sg_ref), b
        else:
            bits, payload, off = O.elias_pack(np.array([A], np.float32), lv_ref, sg_ref, d,
                                              dense=(code_kind == O.CODE_ELIAS_DENSE), s=s)
            want = bits_of(payload.view(np.uint32), 0, bits)
            assert got == want, b
        out[b] = (np.float32(A), lv_ref, sg_ref)
    return out


def run_sampled_config(gs, n, d, s, norm_kind, code_kind, step, nsample, eta=0.1):
    """Encode every worker on the GPU, check sampled buckets of every message, then check the
    decode / SGD kernels on the same buckets and fused == unfused on the whole vector."""
    K = len(gs)
    B = O.n_buckets(n, d)
    buckets = sample_buckets(B, nsample, seed=n % 1000 + d + s)
    cap = min(Q.qsgd_message_capacity(n, d, s, code_kind),
              2 * Q.qsgd_message_capacity(n, d, s, O.CODE_FIXED) + 8 * (B + 1))
    msgs, infos, fields = [], [], []
    for w in range(K):
        big, info, st, _ = gpu_encode(gs[w], d, s, norm_kind, code_kind, SEED, step, w, capacity=cap)
        assert st == 0
        fields.append(check_sampled(gs[w], big, info, n, d, s, norm_kind, code_kind, step, w, buckets))
        msgs.append(big[: info[2]])
        infos.append(info)
    tables = None if code_kind == O.CODE_FIXED else [table_view(m, i, n, d) for m, i in zip(msgs, infos)]
    status = Q.new_status()
    acc = torch.empty(n, dtype=torch.float32, device="cuda")
    Q.qsgd_decode_accumulate(msgs, tables, n, d, s, code_kind, acc, status)
    x0 = I.gaussian_device(n, 1.0, seed=99)
    x_unf = x0.clone()
    Q.qsgd_sgd_step(x_unf, acc, eta, K)
    x_fus = x0.clone()
    Q.qsgd_decode_sgd_step(msgs, tables, n, d, s, code_kind, x_fus, eta, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(x_unf.view(torch.int32), x_fus.view(torch.int32)), "fused != unfused"
    for b in buckets:
        lo, hi = b * d, min((b + 1) * d, n)
        ref = np.zeros(hi - lo, dtype=np.float32)
        for w in range(K):
            A, lv, sg = fields[w][b]
            ref = (ref + O.dequantize(np.array([A], np.float32), lv, sg, d, s)).astype(np.float32)
        assert np.array_equal(acc[lo:hi].cpu().numpy().view(np.uint32), ref.view(np.uint32)), b
        xr = O.sgd_step(x0[lo:hi].cpu().numpy(), ref, eta, K)
        assert np.array_equal(x_fus[lo:hi].cpu().numpy().view(np.uint32), xr.view(np.uint32)), b
    return infos


def run_whole_config(gs, n, d, s, norm_kind, code_kind, step, eta=0.1):
    """Whole-message, whole-vector compare at full size: every byte of the first and the last
    worker's message equals the oracle's encoding (given the GPU's scales, which are checked
    against the oracle's fp64 norms), and every coordinate of the fused step over all K messages
    equals the oracle's decode + aggregate + step of those messages."""
    K = len(gs)
    B = O.n_buckets(n, d)
    cap = min(Q.qsgd_message_capacity(n, d, s, code_kind),
              2 * Q.qsgd_message_capacity(n, d, s, O.CODE_FIXED) + 8 * (B + 1))
    msgs, infos = [], []
    for w in range(K):
        big, info, st, _ = gpu_encode(gs[w], d, s, norm_kind, code_kind, SEED, step, w, capacity=cap)
        assert st == 0
        msgs.append(big[: info[2]])
        infos.append(info)
    for w in (0, K - 1):
        g = gs[w].cpu().numpy()
        msg = msgs[w].cpu().numpy()
        A_gpu = scales_from_message(msg, infos[w], n, d, s, code_kind)
        check_scales(A_gpu, g, d, norm_kind)
        ref, ref_info = O.encode(g, d, s, norm_kind, code_kind, SEED, step, w, A_ext=A_gpu)
        assert infos[w] == ref_info
        assert np.array_equal(msg, ref), "message of worker %d differs from the oracle's" % w
        del g, ref
    x0 = I.gaussian_device(n, 1.0, seed=99)
    x = x0.clone()
    status = Q.new_status()
    info_dev = [torch.tensor(i, dtype=torch.int64, device="cuda") for i in infos]
    Q.qsgd_decode_sgd_step_packed(msgs, None if code_kind == O.CODE_FIXED else info_dev, n, d, s, code_kind, x, eta,
                                  status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    msgs_np = [m.cpu().numpy() for m in msgs]
    tabs = None if code_kind == O.CODE_FIXED else [O.message_table(m, i, n, d) for m, i in zip(msgs_np, infos)]
    st, acc = O.decode_accumulate(msgs_np, tabs, n, d, s, code_kind)
    assert st == 0
    x_ref = O.sgd_step(x0.cpu().numpy(), acc, eta, K)
    assert np.array_equal(x.cpu().numpy().view(np.uint32), x_ref.view(np.uint32)), "stepped x differs from the oracle's"


def test_config3_alexnet_whole():
    shapes = I.alexnet_shapes()
    n = I.numel(shapes)
    gs = [I.layered_gaussian_device(shapes, seed=1 + w) for w in range(16)]
    run_whole_config(gs, n, 512, 255, O.NORM_MAX, O.CODE_FIXED, step=0)


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_config4_resnet152_whole(code_kind):
    n = I.numel(I.resnet152_shapes())
    gs = [I.gaussian_mixture_device(n, seed=1 + w) for w in range(16)]
    run_whole_config(gs, n, 512, 15, O.NORM_L2, code_kind, step=0)


def test_config1_tiny_whole():
    n, d, s, K = 2 ** 20, 512, 15, 4
    msgs, infos = [], []
    for w in range(K):
        g = I.gaussian(n, 0.01, seed=1 + w)
        m, info = encode_parity(g, d, s, O.NORM_L2, O.CODE_FIXED, SEED, 0, w)
        assert info[2] == 663552
        msgs.append(m)
        infos.append(info)
    acc, x = decode_parity(msgs, infos, n, d, s, O.CODE_FIXED, eta=0.1, x0=np.zeros(n, np.float32))
    assert np.array_equal(x, -(np.float32(0.025) * acc))           # x0 = 0: x = -(eta / K) * acc


def test_config2_sparse_elias_whole():
    n, d, s, K = 2 ** 24, 4096, 1, 8
    bound = (3 + 1.5 * math.log2(2 * (1 + d) / (1 + math.sqrt(d)))) * (1 + math.sqrt(d)) + 32
    msgs, infos = [], []
    for w in range(K):
        g = I.sparse_laplace(n, 1e-3, 0.3, seed=1 + w)
        m, info = encode_parity(g, d, s, O.NORM_L2, O.CODE_ELIAS, SEED, 0, w)
        assert info[0] / n <= bound / d                             # Theorem 3.2 at s = 1
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=0.1, x0=I.gaussian(n, 1.0, seed=3))


def test_config3_alexnet_sampled():
    shapes = I.alexnet_shapes()
    n = I.numel(shapes)
    assert n == 61100840 and n % 512 == 296
    gs = [I.layered_gaussian_device(shapes, seed=1 + w) for w in range(16)]
    run_sampled_config(gs, n, 512, 255, O.NORM_MAX, O.CODE_FIXED, step=0, nsample=64)


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_config4_resnet152_sampled(code_kind):
    n = I.numel(I.resnet152_shapes())
    assert n == 60192808 and n % 512 == 40
    gs = [I.gaussian_mixture_device(n, seed=1 + w) for w in range(16)]
    run_sampled_config(gs, n, 512, 15, O.NORM_L2, code_kind, step=0, nsample=64)


@pytest.mark.parametrize("d,s,norm,code", [(512, 15, O.NORM_L2, O.CODE_FIXED),
                                           (4096, 255, O.NORM_MAX, O.CODE_FIXED),
                                           (128, 1, O.NORM_L2, O.CODE_ELIAS),
                                           (4096, 3, O.NORM_MAX, O.CODE_ELIAS_DENSE)])
def test_config5_sweep_point_full_size_sampled(d, s, norm, code):
    n = 2 ** 28
    g = I.gaussian_device(n, 1.0, seed=1)
    gs = [g, g, g]                       # one 1 GiB buffer encoded under three worker ids
    run_sampled_config(gs, n, d, s, norm, code, step=0, nsample=32)


@pytest.mark.parametrize("d", [128, 512, 4096])
@pytest.mark.parametrize("s", [1, 3, 15, 255])
@pytest.mark.parametrize("norm", [O.NORM_L2, O.NORM_MAX])
@pytest.mark.parametrize("code", [O.CODE_FIXED, O.CODE_ELIAS])
def test_config5_sweep_quick_whole(d, s, norm, code):
    n, K = 2 ** 20, 2
    msgs, infos = [], []
    for w in range(K):
        g = I.gaussian(n, 1.0, seed=1 + w)
        m, info = encode_parity(g, d, s, norm, code, SEED, 0, w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, code)


# Maximum sizes: index arithmetic past 2^31 coordinates on the whole path, and the largest n the ABI
# takes (QSGD_MAX_COORDS = 2^32) on Encode. Sampled buckets; about 55 GB on the device at the peak.
@pytest.mark.parametrize("d,s,norm,code", [(512, 15, O.NORM_L2, O.CODE_FIXED), (512, 15, O.NORM_L2, O.CODE_ELIAS),
                                           (4096, 1, O.NORM_MAX, O.CODE_ELIAS)])
def test_beyond_2_31_coordinates_sampled(d, s, norm, code):
    n = 2 ** 31 + 777
    gs = [I.gaussian_mixture_device(n, 31 + w, device="cuda") for w in range(2)]
    run_sampled_config(gs, n, d, s, norm, code, step=2, nsample=40)
    del gs
    torch.cuda.empty_cache()


def test_largest_n_encode_sampled():
    n = 2 ** 32 - 4096 * 3 - 5
    g = I.gaussian_mixture_device(n, 5, device="cuda")
    for d, s, norm, code in [(512, 15, O.NORM_L2, O.CODE_FIXED), (512, 3, O.NORM_L2, O.CODE_ELIAS)]:
        B = O.n_buckets(n, d)
        cap = min(Q.qsgd_message_capacity(n, d, s, code),
                  2 * Q.qsgd_message_capacity(n, d, s, O.CODE_FIXED) + 8 * (B + 1))
        big, info, st, _ = gpu_encode(g, d, s, norm, code, SEED, 1, 0, capacity=cap)
        assert st == 0
        check_sampled(g, big, info, n, d, s, norm, code, 1, 0, sample_buckets(B, 40, seed=7))
        del big
        torch.cuda.empty_cache()
    del g
    torch.cuda.empty_cache()
