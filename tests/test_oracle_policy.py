"""Pins for the per-tensor policy of the oracle (Section 5, "Protocol": small tensors travel in
full precision, buckets are cut to fit the tensors). Every check compares the policy functions with
something computed without them: the ordinary oracle applied tensor by tensor, plain numpy, or counts
that follow from the public layer shapes and the 10K threshold."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I


def numel(shape):
    n = 1
    for v in shape:
        n *= v
    return n


def test_small_tensor_counts_of_the_model_shapes():
    # AlexNet: the eight bias vectors are the only tensors under 10K elements.
    sizes = [numel(s) for s in I.alexnet_shapes()]
    plan = O.policy_plan(sizes, 512)
    assert len(plan["small"]) == 8
    assert plan["n_raw"] == 64 + 192 + 384 + 256 + 256 + 4096 + 4096 + 1000 == 10344
    assert plan["n"] == 61100840
    # ResNet-152: all batch-norm vectors, the fc bias, the stem and the first 1x1 convolution
    sizes = [numel(s) for s in I.resnet152_shapes()]
    plan = O.policy_plan(sizes, 512)
    small = [m for m in sizes if m < 10000]
    assert len(plan["small"]) == len(small) == 313
    assert plan["n_raw"] == sum(small) == 165928
    assert plan["n"] == 60192808
    # every quantized tensor starts on a bucket boundary of the compact vector
    assert all(c0 % 512 == 0 for _, _, c0 in plan["large"])
    assert plan["n_compact"] == sum((m + 511) // 512 * 512 for m in sizes if m >= 10000)


def test_threshold_is_inclusive_at_the_limit():
    plan = O.policy_plan([9999, 10000, 0, 10001], 128)
    assert [m for _, m, _ in plan["small"]] == [9999]
    assert [m for _, m, _ in plan["large"]] == [10000, 10001]


@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE])
def test_one_large_tensor_of_whole_buckets_is_the_ordinary_message(code_kind):
    d, s = 256, 15
    g = I.gaussian(40 * d, 0.01, seed=3)
    plan = O.policy_plan([g.size], d)
    m, info = O.policy_encode(g, plan, s, O.NORM_L2, code_kind, 7, 1, 2)
    ref, ref_info = O.encode(g, d, s, O.NORM_L2, code_kind, 7, 1, 2)
    assert np.array_equal(m, ref) and info == [ref_info[0], ref_info[1], ref_info[2], 0]
    st, acc = O.policy_decode_accumulate([m], [info], plan, s, code_kind)
    tabs = None if code_kind == O.CODE_FIXED else [O.message_table(ref, ref_info, g.size, d)]
    st2, acc2 = O.decode_accumulate([ref], tabs, g.size, d, s, code_kind)
    assert st == 0 and st2 == 0 and np.array_equal(acc.view(np.uint32), acc2.view(np.uint32))


@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
@pytest.mark.parametrize("code_kind", [O.CODE_FIXED, O.CODE_ELIAS])
def test_buckets_restart_at_every_tensor(norm_kind, code_kind):
    """The decoded update of each quantized tensor equals what the ordinary quantizer gives for that
    tensor alone, with its uniforms taken at the tensor's place in the compact vector."""
    d, s = 128, 7
    sizes = [50, 10000 + 37, 3, 12800, 9999, 10000 + 128 * 3 + 1]
    g = I.gaussian_mixture(sum(sizes), seed=11)
    plan = O.policy_plan(sizes, d)
    m, info = O.policy_encode(g, plan, s, norm_kind, code_kind, 5, 2, 1)
    st, acc = O.policy_decode_accumulate([m], [info], plan, s, code_kind)
    assert st == 0
    off = 0
    c0 = 0
    for size in sizes:
        part = g[off:off + size]
        if size < 10000:
            assert np.array_equal(acc[off:off + size].view(np.uint32), part.view(np.uint32))
        else:
            A = O.bucket_scales(part, d, norm_kind)
            lv, sg = O.quantize(part, d, s, A, 5, 2, 1, i0=c0)
            q = O.dequantize(A, lv, sg, d, s)
            assert np.array_equal(acc[off:off + size].view(np.uint32), q.view(np.uint32))
            c0 += (size + d - 1) // d * d
        off += size


def test_raw_values_are_summed_in_worker_order():
    d, s, K = 64, 3, 5
    sizes = [700, 10048, 33]
    plan = O.policy_plan(sizes, d)
    gs = [I.gaussian(sum(sizes), 10.0 ** (w - 2), seed=20 + w) for w in range(K)]
    enc = [O.policy_encode(g, plan, s, O.NORM_MAX, O.CODE_FIXED, 9, 0, w) for w, g in enumerate(gs)]
    st, acc = O.policy_decode_accumulate([e[0] for e in enc], [e[1] for e in enc], plan, s, O.CODE_FIXED)
    assert st == 0
    for lo, hi in ((0, 700), (700 + 10048, 700 + 10048 + 33)):
        ref = np.zeros(hi - lo, dtype=np.float32)
        for g in gs:
            ref = (ref.astype(np.float32) + g[lo:hi]).astype(np.float32)
        assert np.array_equal(acc[lo:hi].view(np.uint32), ref.view(np.uint32))
    # K = 1 and eta = 1: the step subtracts a raw tensor exactly
    st, acc1 = O.policy_decode_accumulate([enc[0][0]], [enc[0][1]], plan, s, O.CODE_FIXED)
    x = O.sgd_step(np.zeros(sum(sizes), np.float32), acc1, 1.0, 1)
    assert np.array_equal(x[:700], -gs[0][:700])


def test_message_sizes_and_raw_region():
    d, s = 512, 15
    sizes = [5, 20000, 11]
    g = I.gaussian(sum(sizes), 0.01, seed=1)
    plan = O.policy_plan(sizes, d)
    m, info = O.policy_encode(g, plan, s, O.NORM_L2, O.CODE_FIXED, 7, 0, 0)
    assert plan["raw_prefix"] == 64 and info[3] == 64                     # 16 floats, already 16-byte aligned
    raw = m[:64].view(np.float32)
    assert np.array_equal(raw[:5], g[:5]) and np.array_equal(raw[5:16], g[20005:])
    n_c = 40 * 512                                                          # 20000 padded to whole buckets
    assert plan["n_compact"] == n_c
    fixed_bytes = 4 * 40 + 4 * (n_c // 32) + 4 * (n_c * 4 // 32)             # scales, signs, 4-bit levels
    assert fixed_bytes == 12960
    assert info[2] == 64 + fixed_bytes and info[1] == 0
    assert info[0] == 32 * 16 + 8 * fixed_bytes


def test_only_small_tensors():
    plan = O.policy_plan([10, 20], 512)
    g = I.gaussian(30, 1.0, seed=4)
    m, info = O.policy_encode(g, plan, 15, O.NORM_L2, O.CODE_ELIAS, 7, 0, 0)
    assert info == [32 * 30, 0, 128, 128]
    st, acc = O.policy_decode_accumulate([m, m], [info, info], plan, 15, O.CODE_ELIAS)
    assert st == 0 and np.array_equal(acc, g + g)
