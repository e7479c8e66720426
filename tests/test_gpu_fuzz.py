"""Seeded random shapes through the whole path on the GPU against the oracle: the parametrised
parity tests pick their shapes by hand; these draw them (n, bucket size, s, norm, code kind, number
of peers, input family) from a fixed seed, so that a shape nobody thought of gets its turn. Every
case is small enough for the oracle to finish in well under a second."""
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I
from parity_util import decode_parity, encode_parity

pytestmark = pytest.mark.gpu


def draw_case(rng):
    # bucket sizes: the streaming kernels' powers of two, the generic kernel's other multiples of 32
    d = int(rng.choice([32, 64, 128, 256, 512, 512, 1024, 2048, 4096, 4096,
                        32 * int(rng.integers(1, 80))]))
    buckets = int(rng.integers(1, 1 + max(1, 200000 // d)))
    n = max(1, buckets * d - int(rng.integers(0, d)))            # ragged last bucket more often than not
    s = int(rng.choice([1, 2, 3, 4, 7, 15, 15, 16, 31, 64, 200, 255]))
    norm_kind = int(rng.choice([O.NORM_L2, O.NORM_MAX]))
    code_kind = int(rng.choice([O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS, O.CODE_ELIAS_DENSE]))
    K = int(rng.choice([1, 2, 3, 4, 5, 8, 16, 17, 33, 64]))
    family = str(rng.choice(["mixture", "gauss", "sparse", "tiny_values", "huge_values", "zeros_inside"]))
    return n, d, s, norm_kind, code_kind, K, family


def make_input(family, n, seed):
    if family == "mixture":
        return I.gaussian_mixture(n, seed=seed)
    if family == "gauss":
        return I.gaussian(n, 1.0, seed=seed)
    if family == "sparse":
        return I.sparse_laplace(n, 1e-3, 0.3, seed=seed)
    if family == "tiny_values":                       # sums of squares far below fp32's normal range
        return (I.gaussian(n, 1.0, seed=seed) * np.float32(1e-22)).astype(np.float32)
    if family == "huge_values":                       # sums of squares beyond fp32's range
        return (I.gaussian(n, 1.0, seed=seed) * np.float32(3e19)).astype(np.float32)
    g = I.gaussian(n, 1.0, seed=seed)                 # whole stretches of exact zeros (zero buckets)
    z = np.random.default_rng(seed).integers(0, n, size=4)
    for a in z:
        g[a: a + 3000] = 0.0
    return g


# QSGD_FUZZ_CASES / QSGD_FUZZ_POLICY_CASES draw more cases from the same seeds (the defaults are a prefix)
SEED0 = int(os.environ.get("QSGD_FUZZ_SEED", "0"))          # shifts every case's seed: a different campaign
N_CASES = int(os.environ.get("QSGD_FUZZ_CASES", "72"))
N_POLICY_CASES = int(os.environ.get("QSGD_FUZZ_POLICY_CASES", "40"))
CASES = [draw_case(np.random.default_rng(1000 + SEED0 + i)) for i in range(N_CASES)]


@pytest.mark.parametrize("case", CASES, ids=["n%d_d%d_s%d_norm%d_code%d_K%d_%s" % c for c in CASES])
def test_random_shape_matches_oracle(case):
    n, d, s, norm_kind, code_kind, K, family = case
    msgs, infos = [], []
    for w in range(K):
        g = make_input(family, n, seed=300 + 7 * w)
        m, info = encode_parity(g, d, s, norm_kind, code_kind, 11, 5, w)
        msgs.append(m)
        infos.append(info)
    # step sizes of either sign and zero, and parameters that hold both zeros: x - c * (+0) is x bit for
    # bit only for some of these, which the decoders that skip untouched coordinates must get right
    eta = [0.05, -0.05, 0.0, 1.0, 3e-39][(n + d + s) % 5]
    x0 = I.gaussian(n, 1.0, seed=77)
    x0[::7] = -0.0
    x0[3::11] = 0.0
    decode_parity(msgs, infos, n, d, s, code_kind, eta=eta, x0=x0)
    if code_kind != O.CODE_FIXED and (n + K) % 2 == 0:
        # offset tables kept in front of the payloads: the library cannot read sizes off the pointers
        decode_parity(msgs, infos, n, d, s, code_kind, eta=eta, x0=x0, tables_first=True)
    torch.cuda.synchronize()


def draw_policy_case(rng):
    d = int(rng.choice([32, 128, 256, 512, 512, 1024, 4096, 32 * int(rng.integers(1, 40))]))
    aligned = bool(rng.integers(0, 2))                 # every size a multiple of 4: the bulk-copy paths
    T = int(rng.integers(1, 12))
    sizes = []
    for _ in range(T):
        kind = int(rng.integers(0, 4))
        if kind == 0:
            m = int(rng.integers(1, 300))                                  # stays raw
        elif kind == 1:
            m = int(rng.integers(1, 40)) * d                               # whole buckets
        elif kind == 2:
            m = int(rng.integers(4096, 60000))                             # ends in a short bucket
        else:
            m = 4096 * int(rng.integers(1, 12)) + int(rng.integers(0, 9))  # several tiles, tiny remainder
        if aligned:
            m = max(4, m // 4 * 4)
        sizes.append(m)
    s = int(rng.choice([1, 3, 7, 15, 64, 255]))
    norm_kind = int(rng.choice([O.NORM_L2, O.NORM_MAX]))
    code_kind = int(rng.choice([O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE]))
    K = int(rng.choice([1, 2, 3, 5, 16]))
    tau = int(rng.choice([1, 1000, 4096, 10000, 50000]))
    return tuple(sizes), d, s, norm_kind, code_kind, K, tau


POLICY_CASES = [draw_policy_case(np.random.default_rng(5000 + SEED0 + i)) for i in range(N_POLICY_CASES)]


@pytest.mark.parametrize("case", POLICY_CASES,
                         ids=["T%d_n%d_d%d_s%d_norm%d_code%d_K%d_tau%d" % (len(c[0]), sum(c[0]), *c[1:]) for c in POLICY_CASES])
def test_random_policy_matches_oracle(case):
    from test_gpu_policy import run_case
    sizes, d, s, norm_kind, code_kind, K, tau = case
    run_case(list(sizes), d, s, norm_kind, code_kind, K=K, tau=tau)


def draw_mid_case(rng):
    # enough tiles for every persistent warp / CTA of the streaming encoders to go round its ring
    # of stages several times (2.4 M coordinates fill the grid once)
    d = int(rng.choice([32, 128, 512, 1024, 4096]))
    n = int(rng.integers(1_500_000, 14_000_000))      # from less than one tile per CTA of the grid to several
    s = int(rng.choice([1, 3, 15, 255]))
    norm_kind = int(rng.choice([O.NORM_L2, O.NORM_MAX]))
    code_kind = int(rng.choice([O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE]))
    family = str(rng.choice(["mixture", "sparse", "zeros_inside"]))
    return n, d, s, norm_kind, code_kind, family


MID_CASES = [draw_mid_case(np.random.default_rng(9000 + SEED0 + i)) for i in range(int(os.environ.get("QSGD_FUZZ_MID_CASES", "10")))]


@pytest.mark.parametrize("case", MID_CASES, ids=["n%d_d%d_s%d_norm%d_code%d_%s" % c for c in MID_CASES])
def test_random_mid_size_matches_oracle(case):
    n, d, s, norm_kind, code_kind, family = case
    msgs, infos = [], []
    for w in range(2):
        m, info = encode_parity(make_input(family, n, seed=40 + w), d, s, norm_kind, code_kind, 3, 9, w)
        msgs.append(m)
        infos.append(info)
    decode_parity(msgs, infos, n, d, s, code_kind, eta=0.05, x0=I.gaussian(n, 1.0, seed=78))


CAP_CASES = [(draw_case(np.random.default_rng(13000 + SEED0 + i)), float(np.random.default_rng(13000 + SEED0 + i).uniform(0.0, 1.15)))
             for i in range(int(os.environ.get("QSGD_FUZZ_CAPACITY_CASES", "30")))]


@pytest.mark.parametrize("case,frac", CAP_CASES, ids=["n%d_d%d_s%d_norm%d_code%d_K%d_%s" % c + "_f%.2f" % f for c, f in CAP_CASES])
def test_random_message_capacity(case, frac):
    """An Elias encode into a buffer between the smallest size the host accepts and a little more than
    the message needs: either the message is there, identical to the unconstrained one, or the
    capacity flag is up, the size needed is reported and not a byte of the buffer was written."""
    import paper_1610_02132_b200 as Q
    from parity_util import CANARY, gpu_encode
    n, d, s, norm_kind, code_kind, K, family = case
    if code_kind == O.CODE_FIXED:
        code_kind = O.CODE_ELIAS
    g_dev = torch.from_numpy(make_input(family, n, seed=21)).cuda()
    full, info, st, _ = gpu_encode(g_dev, d, s, norm_kind, code_kind, 4, 2, 1)
    assert st == 0
    need = info[2]
    B = O.n_buckets(n, d)
    floor = 16 * ((4 * B + 15) // 16) + 8 * (B + 1)             # scales and table: the host's minimum
    cap = (floor + int(frac * (need - floor))) // 16 * 16
    cap = max(cap, floor)
    big, info2, st2, _ = gpu_encode(g_dev, d, s, norm_kind, code_kind, 4, 2, 1, capacity=cap) if cap >= need else (None, None, None, None)
    if cap >= need:
        assert st2 == 0 and info2 == info and torch.equal(big[:need], full[:need])
        return
    buf = torch.full((cap + 256,), CANARY, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code_kind), 16), dtype=torch.uint8, device="cuda")
    status = Q.new_status("cuda")
    Q.qsgd_encode(g_dev, d, s, norm_kind, code_kind, 4, 2, 1, buf[:cap], bits, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == Q.binding.DEV_CAPACITY
    assert bool((buf == CANARY).all()), "bytes written into a buffer that is too small"
    assert int(bits.cpu().numpy().view(np.uint64)[2]) == need
