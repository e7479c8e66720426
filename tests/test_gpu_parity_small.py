"""GPU parity, whole-message compare at sizes the oracle finishes in seconds: several tiles, a
ragged tail, every code kind, both norms, all field widths."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

from parity_util import decode_parity, encode_parity

pytestmark = pytest.mark.gpu

CODES = [O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE]


def make(n, kind, seed):
    if kind == "gauss":
        return I.gaussian(n, 0.01, seed=seed)
    if kind == "sparse":
        return I.sparse_laplace(n, 1e-3, 0.3, seed=seed)
    return I.gaussian_mixture(n, seed=seed)


@pytest.mark.parametrize("n,d", [(3 * 4096 + 1234 + 5, 512), (2 * 4096 + 1, 4096), (5000, 128),
                                 (40000, 96), (777, 32), (1, 32), (33, 32), (4096, 4096)])
@pytest.mark.parametrize("s", [1, 3, 15, 255])
@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
@pytest.mark.parametrize("code_kind", CODES)
def test_encode_decode_parity(n, d, s, norm_kind, code_kind):
    K = 3
    kinds = ["gauss", "sparse", "mix"]
    msgs, infos = [], []
    for w in range(K):
        g = make(n, kinds[w], seed=10 * n + w)
        m, info = encode_parity(g, d, s, norm_kind, code_kind, seed=7, step=2, worker=w)
        msgs.append(m)
        infos.append(info)
    x0 = I.gaussian(n, 1.0, seed=99)
    decode_parity(msgs, infos, n, d, s, code_kind, eta=0.1, x0=x0)


@pytest.mark.parametrize("s", [2, 5, 7, 100, 127, 128, 200])
@pytest.mark.parametrize("code_kind", CODES)
def test_levels_not_power_of_two(s, code_kind):
    n, d = 10000, 256
    msgs, infos = [], []
    for w in range(2):
        g = make(n, "gauss", seed=w + 3)
        m, info = encode_parity(g, d, s, O.NORM_MAX, code_kind, seed=11, step=0, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, code_kind)


@pytest.mark.parametrize("code_kind", CODES)
def test_degenerate_buckets(code_kind):
    n, d, s = 4 * 512, 512, 15
    g = np.zeros(n, dtype=np.float32)
    g[512:1024] = 1e-41                       # subnormal bucket -> zero bucket
    g[1024 + 7] = -2.5                        # single nonzero
    g[1536:] = 3.0                            # all at the maximum
    g[5] = -0.0
    for norm_kind in (O.NORM_L2, O.NORM_MAX):
        m, info = encode_parity(g, d, s, norm_kind, code_kind, seed=1, step=0, worker=0)
        acc, _ = decode_parity([m], [info], n, d, s, code_kind, eta=1.0)
        assert not acc[:1024].any() and not np.signbit(acc[:1024]).any()
        assert acc[1024 + 7] == -2.5
        if norm_kind == O.NORM_MAX:
            assert np.all(acc[1536:] == 3.0)


@pytest.mark.parametrize("d", [64, 512, 1024, 4096, 96])
@pytest.mark.parametrize("scale", [1e-22, 3e19])
@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_two_norm_outside_fp32_range(d, scale, code_kind):
    """Buckets whose fp32 sum of squares underflows (values around 1e-22) or overflows (3e19) take the
    fp64 path of every encoder (per-warp, CTA-wide for d >= 1024, generic), inside the streamed tiles
    and in the tail, next to ordinary buckets; the encode must finish with status 0 and match."""
    n = 5 * 4096 + 3 * d + 17
    g = I.gaussian(n, 1.0, seed=3)
    g[: 2 * 4096] *= np.float32(scale)                 # whole tiles out of range
    g[3 * 4096 + d: 3 * 4096 + 2 * d] *= np.float32(scale)   # one bucket among ordinary ones
    g[5 * 4096:] *= np.float32(scale)                  # the tail
    msgs, infos = [], []
    for w in range(2):
        m, info = encode_parity(np.roll(g, 5 * w), d, 15, O.NORM_L2, code_kind, seed=2, step=1, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, 15, code_kind)


@pytest.mark.parametrize("d", [64, 512, 1024, 96])
def test_two_norm_of_vanishing_squares(d):
    """Values whose squares are below fp32's smallest subnormal (|v| < 3.7e-23) give an fp32 sum of
    squares of exactly zero, yet their norm is far above FLT_MIN: such buckets are not zero buckets.
    One among the streamed tiles, one in the tail, and a last bucket of a single coordinate."""
    B = (3 * 4096) // d + 3                           # buckets, the last of one coordinate
    n = (B - 1) * d + 1
    g = I.gaussian(n, 1.0, seed=8)
    sign = np.where(np.arange(d) % 3 == 0, -1.0, 1.0).astype(np.float32)
    early, late = 4096 // d + 1, B - 2                # a bucket inside the streamed tiles, one in the tail
    g[early * d: (early + 1) * d] = np.float32(2e-23) * sign
    g[late * d: (late + 1) * d] = np.float32(3e-23) * sign
    g[-1] = np.float32(1.5e-23)
    for code_kind in (O.CODE_FIXED, O.CODE_ELIAS):
        m, info = encode_parity(g, d, 15, O.NORM_L2, code_kind, seed=2, step=1, worker=0)
        acc, _ = decode_parity([m], [info], n, d, 15, code_kind, eta=1.0)
        assert acc[-1] != 0.0                         # a bucket of one value: level s, decoded to the value itself
        assert np.any(acc[early * d: (early + 1) * d] != 0.0) and np.any(acc[late * d: (late + 1) * d] != 0.0)


@pytest.mark.parametrize("d", [128, 512, 4096])
@pytest.mark.parametrize("shape", ["equal", "ascending", "descending", "one_large"])
def test_two_norm_tolerance_on_adversarial_inputs(d, shape):
    """fp32 accumulation of the sum of squares must stay within 1e-6 of the exact norm also when the
    rounding errors cannot cancel: all magnitudes equal (every partial sum rounds the same way),
    magnitudes sorted (small terms meet a large running sum, or the reverse), one dominant value."""
    n = 6 * 4096 + 2 * d + 40
    rng = np.random.default_rng(d)
    if shape == "equal":
        g = np.full(n, 0.3337, dtype=np.float32) * rng.choice([-1.0, 1.0], n).astype(np.float32)
    elif shape == "one_large":
        g = np.full(n, 1e-3, dtype=np.float32)
        g[::d] = 0.777
    else:
        g = (1.0 + 1e-3 * np.arange(n, dtype=np.float64) % d).astype(np.float32)
        g = np.sort(g.reshape(-1)[: n]) if shape == "ascending" else np.sort(g)[::-1].copy()
        g = (g * (1.0 + (np.arange(n) % d) / d)).astype(np.float32)
        if shape == "descending":
            g = g[::-1].copy()
    for s in (1, 15):
        m, info = encode_parity(np.ascontiguousarray(g, dtype=np.float32), d, s, O.NORM_L2, O.CODE_FIXED,
                                seed=3, step=1, worker=0)
        decode_parity([m], [info], n, d, s, O.CODE_FIXED)


def test_many_peers_and_philox_keying():
    n, d, s = 20000, 512, 15
    g = make(n, "gauss", 5)
    msgs, infos = [], []
    for w in range(20):                       # same gradient, different worker ids
        m, info = encode_parity(g, d, s, O.NORM_L2, O.CODE_FIXED, seed=2 ** 40 + 3, step=9, worker=w)
        msgs.append(m)
        infos.append(info)
    assert not torch.equal(msgs[0], msgs[1])
    acc, _ = decode_parity(msgs, infos, n, d, s, O.CODE_FIXED)
    # the mean of 20 independent quantizations is close to g (unbiasedness, Lemma 3.1)
    A = O.bucket_scales(g, d, O.NORM_L2)
    err = np.abs(acc / 20 - g)
    assert err.max() < 5 * np.repeat(A, d)[:n].max() / 15 / np.sqrt(20) * 0.5 + 1e-3


@pytest.mark.parametrize("K", [1, 5, 16, 33, 40])
@pytest.mark.parametrize("code_kind", [O.CODE_ELIAS, O.CODE_ELIAS_DENSE])
def test_elias_peer_counts(K, code_kind):
    n, d, s = 3 * 512 + 77, 512, 7
    msgs, infos = [], []
    for w in range(K):
        g = make(n, "mix", seed=100 + w)
        m, info = encode_parity(g, d, s, O.NORM_L2, code_kind, seed=5, step=1, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, code_kind, eta=0.05, x0=I.gaussian(n, 1.0, seed=9))
    decode_parity(msgs, infos, n, d, s, code_kind, eta=0.05, x0=I.gaussian(n, 1.0, seed=9), tables_first=True)


@pytest.mark.parametrize("K", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("d,tail", [(512, 188), (512, 300), (256, 100), (96, 40), (992, 500)])
def test_elias_few_peers_high_levels_ragged_tail(K, d, tail):
    """Few peers (a warp then owns many buckets), max-norm scaling at s = 15 (negative levels of 8 and
    more occur, the codes whose value sits in the upper lanes of the decoder's shuffle table) and a
    last bucket that is shorter than a decoding range."""
    n, s = 9 * d + tail, 15
    msgs, infos = [], []
    for w in range(K):
        g = make(n, "mix", seed=500 + w)
        m, info = encode_parity(g, d, s, O.NORM_MAX, O.CODE_ELIAS, seed=9, step=2, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=0.3, x0=I.gaussian(n, 1.0, seed=2))


@pytest.mark.parametrize("d", [32, 64, 160, 256, 288, 480, 512, 736, 1000 // 32 * 32])
@pytest.mark.parametrize("K,s,norm_kind", [(1, 15, O.NORM_MAX), (2, 3, O.NORM_L2), (4, 7, O.NORM_MAX), (7, 1, O.NORM_L2),
                                           (16, 15, O.NORM_L2), (17, 2, O.NORM_MAX), (32, 15, O.NORM_MAX)])
def test_elias_decoder_shapes_below_1024(d, K, s, norm_kind):
    """Bucket sizes around the decoder's range length (256), peer counts around the powers of two that
    set how many buckets a warp owns, every field width up to 4 bits, a ragged tail."""
    n = 11 * d + d // 2 + 3
    msgs, infos = [], []
    for w in range(K):
        g = make(n, ["gauss", "sparse", "mix"][w % 3], seed=700 + w)
        m, info = encode_parity(g, d, s, norm_kind, O.CODE_ELIAS, seed=3, step=5, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=0.2, x0=I.gaussian(n, 1.0, seed=4))


@pytest.mark.parametrize("d,s", [(4096, 255), (4096, 1), (2048, 15), (1024, 3), (64, 15), (32, 1)])
def test_elias_bucket_shapes(d, s):
    n, K = 5 * d + 123, 4
    for code_kind in (O.CODE_ELIAS, O.CODE_ELIAS_DENSE):
        msgs, infos = [], []
        for w in range(K):
            g = make(n, "gauss", seed=200 + w)
            m, info = encode_parity(g, d, s, O.NORM_MAX, code_kind, seed=5, step=1, worker=w)
            msgs.append(m)
            infos.append(info)
        decode_parity(msgs, infos, n, d, s, code_kind)


def sparse_regime_bits(K, d):
    """Average bits per string below which the decoder takes its entry-list path."""
    return 32 + d // 4


# Short strings (Section 3.1, sparse regime) take the entry-list decoder; these cases sit on
# that side of its switch, which is decided on the device from the payload lengths.
@pytest.mark.parametrize("n,d,s,K,zeros", [(5 * 4096 + 123, 4096, 1, 8, 0.3), (9 * 1024 + 77, 1024, 1, 5, 0.3),
                                           (11 * 3008 + 5, 3008, 1, 3, 0.3), (4 * 2048, 2048, 1, 32, 0.3),
                                           (3 * 4096 + 1, 4096, 1, 1, 0.3), (70 * 64 + 9, 64, 3, 16, 0.98),
                                           # enough buckets that a warp takes its full share of them
                                           (7200 * 64 + 5, 64, 1, 8, 0.98), (14300 * 128 + 3, 128, 1, 3, 0.95),
                                           (57000 * 32 + 31, 32, 1, 1, 0.98),
                                           # few buckets of a size that is no power of two, one or two peers:
                                           # one bucket per warp, lists of 928 / 32 = 29 and 608 / 32 = 19 entries
                                           (46 * 928, 928, 1, 1, 0.3), (30 * 608 - 3, 608, 1, 2, 0.7)])
@pytest.mark.parametrize("eta", [0.1, -0.25])
def test_elias_sparse_regime(n, d, s, K, zeros, eta):
    msgs, infos = [], []
    for w in range(K):
        g = I.sparse_laplace(n, 1e-3, zeros, seed=300 + w)
        m, info = encode_parity(g, d, s, O.NORM_L2, O.CODE_ELIAS, seed=5, step=3, worker=w)
        msgs.append(m)
        infos.append(info)
    B = O.n_buckets(n, d)
    assert sum(i[0] for i in infos) < K * B * sparse_regime_bits(K, d), "case is not in the sparse regime"
    x0 = I.gaussian(n, 1.0, seed=9)
    x0[::7] = -0.0                                  # x - c * (+0) must keep the sign of zero
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=eta, x0=x0)
    if eta > 0:
        decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=eta, x0=x0, tables_first=True)


@pytest.mark.parametrize("d,s,Bn", [(512, 15, 80), (4096, 255, 200), (128, 3, 48)])
def test_elias_sparse_regime_long_lists(d, s, Bn):
    """Mostly empty buckets keep the payload short while a few buckets hold far more nonzeros
    than one list has room for."""
    K = 6
    n = Bn * d - 17
    msgs, infos = [], []
    for w in range(K):
        g = np.zeros(n, dtype=np.float32)
        for b in (3 + w % 2, 20, Bn - 1):
            lo, hi = b * d, min((b + 1) * d, n)
            g[lo:hi] = make(hi - lo, "gauss", seed=400 + 7 * w + b)
        m, info = encode_parity(g, d, s, O.NORM_MAX, O.CODE_ELIAS, seed=6, step=0, worker=w)
        msgs.append(m)
        infos.append(info)
    assert sum(i[0] for i in infos) < K * Bn * sparse_regime_bits(K, d), "case is not in the sparse regime"
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS, eta=0.5, x0=I.gaussian(n, 1.0, seed=1))


@pytest.mark.parametrize("d,s,code_kind", [(512, 15, O.CODE_FIXED), (512, 15, O.CODE_ELIAS), (4096, 1, O.CODE_ELIAS),
                                           (128, 255, O.CODE_ELIAS_DENSE), (96, 3, O.CODE_FIXED)])
def test_pointers_with_the_minimum_alignment(d, s, code_kind):
    """Every pointer the ABI takes needs 16-byte alignment and no more: gradient, message, workspace,
    accumulator and parameters all sit 16 (or 48) bytes into their allocations here."""
    n, K = 6 * 4096 + 2 * d + 13, 3
    dev = "cuda"
    status = Q.new_status(dev)
    cap = Q.qsgd_message_capacity(n, d, s, code_kind)
    wsb = max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16)
    ws = torch.empty(wsb + 64, dtype=torch.uint8, device=dev)[48: 48 + wsb]
    msgs, infos, ref_msgs, ref_tabs = [], [], [], []
    for w in range(K):
        g = I.gaussian_mixture(n, seed=60 + w)
        g_dev = torch.empty(n + 8, dtype=torch.float32, device=dev)[4: 4 + n]
        g_dev.copy_(torch.from_numpy(g))
        out = torch.zeros(cap + 64, dtype=torch.uint8, device=dev)[16: 16 + cap]
        bits = torch.zeros(4, dtype=torch.int64, device=dev)
        Q.qsgd_encode(g_dev, d, s, O.NORM_MAX, code_kind, 3, 1, w, out, bits, ws, status)
        torch.cuda.synchronize()
        info = [int(v) for v in bits.cpu()]
        m, ref_info = O.encode(g, d, s, O.NORM_MAX, code_kind, 3, 1, w)
        assert info == ref_info
        assert np.array_equal(out[: m.size].cpu().numpy(), m)
        msgs.append(out)
        infos.append(bits)
        ref_msgs.append(m)
        ref_tabs.append(O.message_table(m, ref_info, n, d) if code_kind != O.CODE_FIXED else None)
    x0 = I.gaussian(n, 1.0, seed=4)
    x = torch.empty(n + 24, dtype=torch.float32, device=dev)[12: 12 + n]
    x.copy_(torch.from_numpy(x0))
    acc = torch.empty(n + 8, dtype=torch.float32, device=dev)[4: 4 + n]
    elias = code_kind != O.CODE_FIXED
    Q.qsgd_decode_accumulate_packed(msgs, infos if elias else None, n, d, s, code_kind, acc, status)
    Q.qsgd_decode_sgd_step_packed(msgs, infos if elias else None, n, d, s, code_kind, x, 0.1, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    st, acc_ref = O.decode_accumulate(ref_msgs, ref_tabs if elias else None, n, d, s, code_kind)
    assert st == 0
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), acc_ref.view(np.uint32))
    assert np.array_equal(x.cpu().numpy().view(np.uint32), O.sgd_step(x0, acc_ref, 0.1, K).view(np.uint32))


@pytest.mark.parametrize("d", [1024, 4096])
@pytest.mark.parametrize("s,norm_kind", [(3, O.NORM_L2), (64, O.NORM_L2), (255, O.NORM_MAX), (7, O.NORM_MAX), (8, O.NORM_MAX)])
def test_dense_code_long_buckets(d, s, norm_kind):
    """Code'_s with d >= 1024: the decoder takes up to three symbols per table lookup when their levels
    are at most min(s, 7) and a range has room for them, one symbol by the definition's decoder
    otherwise (max-norm: every bucket holds level s; ragged last bucket; ranges of 512 positions)."""
    n, K = 5 * d + d // 2 + 3, 3
    msgs, infos = [], []
    for w in range(K):
        g = I.gaussian(n, 1.0, seed=500 + w)
        m, info = encode_parity(g, d, s, norm_kind, O.CODE_ELIAS_DENSE, seed=8, step=2, worker=w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, O.CODE_ELIAS_DENSE, eta=0.3, x0=I.gaussian(n, 1.0, seed=2))
