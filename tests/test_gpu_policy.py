"""GPU parity of the per-tensor policy (Section 5, "Protocol"): messages, sums and the stepped x
equal the oracle's bit for bit, given the GPU's bucket scales."""
import numpy as np
import pytest
import torch

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

from parity_util import CANARY, check_scales, scales_from_message

pytestmark = pytest.mark.gpu


def numel(shape):
    n = 1
    for v in shape:
        n *= v
    return n


def gpu_policy_encode(g_dev, pl, s, norm_kind, code_kind, seed, step, worker):
    cap = Q.qsgd_policy_message_capacity(pl, s, code_kind)
    big = torch.full((cap + 256,), CANARY, dtype=torch.uint8, device="cuda")
    bits = torch.zeros(4, dtype=torch.int64, device="cuda")
    ws = torch.empty(max(Q.qsgd_policy_workspace_bytes(pl, s, code_kind), 16), dtype=torch.uint8, device="cuda")
    status = Q.new_status("cuda")
    Q.qsgd_policy_encode(g_dev, pl, s, norm_kind, code_kind, seed, step, worker, big[:cap], bits, ws, status)
    torch.cuda.synchronize()
    info = [int(v) for v in bits.cpu().numpy().view(np.uint64)]
    assert int(status.item()) == 0
    assert info[2] <= cap and bool((big[info[2]:] == CANARY).all()), "write past the message"
    return big[:info[2]], info


def policy_encode_parity(g, sizes, pl, oplan, d, s, norm_kind, code_kind, seed, step, worker):
    g_dev = torch.from_numpy(g).cuda()
    msg_dev, info = gpu_policy_encode(g_dev, pl, s, norm_kind, code_kind, seed, step, worker)
    msg = msg_dev.cpu().numpy()
    A_gpu = None
    if oplan["n_compact"]:
        prefix = oplan["raw_prefix"]
        body_info = [info[0], info[1] - prefix if info[1] else 0, info[2] - prefix, 0]
        A_gpu = scales_from_message(msg[prefix:], body_info, oplan["n_compact"], d, s, code_kind)
        compact, _ = O.policy_gather(g, oplan)
        check_scales(A_gpu, compact, d, norm_kind)
    ref, ref_info = O.policy_encode(g, oplan, s, norm_kind, code_kind, seed, step, worker, A_ext=A_gpu)
    assert info == ref_info, (info, ref_info)
    assert np.array_equal(msg, ref), "policy message differs from the oracle's"
    return msg_dev, info


def policy_decode_parity(msgs_dev, infos, pl, oplan, s, code_kind, eta, x0):
    n, K = oplan["n"], len(msgs_dev)
    tables = None
    if code_kind != O.CODE_FIXED:
        B = oplan["n_compact"] // oplan["d"]
        tables = [m[i[1]: i[1] + 8 * (B + 1)].view(torch.int64) if B else m[:0].view(torch.int64)
                  for m, i in zip(msgs_dev, infos)]
        if B == 0:
            tables = [torch.zeros(2, dtype=torch.int64, device="cuda") for _ in msgs_dev]
    status = Q.new_status("cuda")
    acc = torch.full((n + 64,), 7.0, dtype=torch.float32, device="cuda")
    Q.qsgd_policy_decode_accumulate(msgs_dev, tables, pl, s, code_kind, acc[:n], status)
    x_unf = torch.from_numpy(x0.copy()).cuda()
    Q.qsgd_sgd_step(x_unf, acc[:n], eta, K)
    xf = torch.full((n + 64,), 3.0, dtype=torch.float32, device="cuda")
    xf[:n] = torch.from_numpy(x0).cuda()
    Q.qsgd_policy_decode_sgd_step(msgs_dev, tables, pl, s, code_kind, xf[:n], eta, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((acc[n:] == 7.0).all()) and bool((xf[n:] == 3.0).all())
    st, acc_ref = O.policy_decode_accumulate([m.cpu().numpy() for m in msgs_dev], infos, oplan, s, code_kind)
    assert st == 0
    assert np.array_equal(acc[:n].cpu().numpy().view(np.uint32), acc_ref.view(np.uint32))
    x_ref = O.sgd_step(x0, acc_ref, eta, K)
    assert np.array_equal(x_unf.cpu().numpy().view(np.uint32), x_ref.view(np.uint32))
    assert np.array_equal(xf[:n].cpu().numpy().view(np.uint32), x_ref.view(np.uint32))


def run_case(sizes, d, s, norm_kind, code_kind, K, tau=10000, kind="mix", eta=0.1):
    n = sum(sizes)
    pl = Q.Policy(sizes, d, min_quantized=tau)
    oplan = O.policy_plan(sizes, d, tau)
    msgs, infos = [], []
    for w in range(K):
        if kind == "sparse":
            g = I.sparse_laplace(n, 1e-3, 0.3, seed=50 + w)
        else:
            g = I.gaussian_mixture(n, seed=50 + w)
        m, info = policy_encode_parity(g, sizes, pl, oplan, d, s, norm_kind, code_kind, 7, 3, w)
        msgs.append(m)
        infos.append(info)
    policy_decode_parity(msgs, infos, pl, oplan, s, code_kind, eta, I.gaussian(n, 1.0, seed=99))


ALIGNED = [64, 20480, 12, 4096 * 3 + 512, 1000, 8192 + 256, 4]            # every place and length a multiple of 4
RAGGED = [50, 10000 + 37, 3, 12800, 9999, 10000 + 128 * 3 + 1, 1]          # odd places and lengths


@pytest.mark.parametrize("sizes", [ALIGNED, RAGGED])
@pytest.mark.parametrize("d,s", [(512, 15), (128, 3), (4096, 1), (96, 255), (1024, 15)])
@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE])
def test_policy_parity(sizes, d, s, norm_kind, code_kind):
    run_case(sizes, d, s, norm_kind, code_kind, K=3, tau=4096)


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_policy_many_tiles_and_sparse_regime(code_kind):
    # enough buckets for several tiles per CTA of the streaming encoder; s = 1 puts the Elias decode
    # on its entry-list path
    sizes = [300000, 17, 4096 * 40 + 4, 999, 65536, 12288, 8]
    run_case(sizes, 512, 15, O.NORM_L2, code_kind, K=4)
    run_case(sizes, 4096, 1, O.NORM_L2, code_kind, K=8, kind="sparse")


@pytest.mark.parametrize("d", [32, 128, 256, 512])
@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
def test_policy_short_buckets_inside_the_stream(d, norm_kind):
    # every place and length a multiple of 4 (bulk copies), most tensors ending in a short bucket that
    # lies among the complete tiles of the streaming encoder: of 4, of d - 4 and of d / 2 coordinates
    sizes = [4096 * 5 + 4, 8192 + d - 4, 20, 20480 + d // 2, 4096 * 9, 12288 + 36, 65536 + 8]
    run_case(sizes, d, 15, norm_kind, O.CODE_FIXED, K=2, tau=4096)
    run_case(sizes, d, 3, norm_kind, O.CODE_ELIAS, K=2, tau=4096)


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_policy_long_raw_tensors(code_kind):
    # a large threshold leaves long tensors raw
    run_case([20000, 9001, 4096 * 12, 30, 17000], 512, 15, O.NORM_L2, code_kind, K=3, tau=30000)


def test_policy_many_peers():
    run_case(RAGGED, 256, 7, O.NORM_L2, O.CODE_ELIAS, K=33, tau=4096)


@pytest.mark.parametrize("sizes", [[10, 20, 5], [40960]])
@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_policy_only_raw_or_only_quantized(sizes, code_kind):
    run_case(sizes, 512, 15, O.NORM_MAX, code_kind, K=2)


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_policy_resnet152_shapes(code_kind):
    sizes = [numel(sh) for sh in I.resnet152_shapes()]
    run_case(sizes, 512, 15, O.NORM_L2, code_kind, K=2)
