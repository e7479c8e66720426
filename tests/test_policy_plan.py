"""The library's host-side plan of the per-tensor policy against the oracle's (no GPU needed)."""
import numpy as np
import pytest

import paper_1610_02132_b200 as Q
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I


def numel(shape):
    n = 1
    for v in shape:
        n *= v
    return n


def oracle_arrays(sizes, d, min_quantized):
    """Bucket places / lengths and raw segments written out from the oracle's plan."""
    plan = O.policy_plan(sizes, d, min_quantized)
    src, ln = [], []
    for off, m, _ in plan["large"]:
        for c in range(0, m, d):
            src.append(off + c)
            ln.append(min(d, m - c))
    rsrc = [off for off, _, _ in plan["small"]]
    rstart = [r0 for _, _, r0 in plan["small"]] + [plan["n_raw"]]
    return plan, src, ln, rsrc, rstart


@pytest.mark.parametrize("sizes,d,tau", [
    ([100, 12000, 5, 20000, 9999, 10000, 0, 10001], 512, 10000),
    ([64, 64, 4096], 32, 64),
    ([7], 128, 10000),
    ([40000], 4096, 10000),
    ([numel(s) for s in I.alexnet_shapes()], 512, 10000),
    ([numel(s) for s in I.resnet152_shapes()], 512, 10000),
])
def test_plan_matches_oracle(sizes, d, tau):
    plan, src, ln, rsrc, rstart = oracle_arrays(sizes, d, tau)
    pl = Q.Policy(sizes, d, min_quantized=tau, device="cpu")
    assert pl.n == plan["n"] and pl.n_raw == plan["n_raw"] and pl.raw_prefix == plan["raw_prefix"]
    assert pl.n_buckets * d == plan["n_compact"]
    assert pl.host["bucket_src"].tolist() == src and pl.host["bucket_len"].tolist() == ln
    assert pl.host["raw_src"].tolist() == rsrc and pl.host["raw_start"].tolist() == rstart
    assert pl.quads == int(all(v % 4 == 0 for v in src + ln))


def test_model_shapes_allow_16_byte_accesses():
    for shapes in (I.alexnet_shapes(), I.resnet152_shapes()):
        assert Q.Policy([numel(s) for s in shapes], 512, device="cpu").quads == 1


def test_plan_rejects_bad_arguments():
    with pytest.raises(Q.QsgdError):
        Q.Policy([0, 0], 512, device="cpu")
    with pytest.raises(Q.QsgdError):
        Q.Policy([100], 100, device="cpu")


def test_policy_entry_points_validate_before_launching():
    """Argument errors come back as negative status codes with no GPU work (none is available here)."""
    import ctypes as C
    from paper_1610_02132_b200 import binding as B
    L = B.lib()
    pl = Q.Policy([64, 20000], 512, device="cpu")
    st = B.PolicyStruct(0, 0, pl.n_buckets, 0, 0, pl.n_raw_segments, pl.n_raw, pl.n, 1)    # null plan arrays
    assert L.qsgd_policy_encode(None, C.byref(st), 512, 15, 0, 0, 7, 0, 0, None, 0, None, None, None, None) == -1
    assert L.qsgd_policy_message_capacity(C.byref(st), 512, 15, 0) == 0
    good = B.PolicyStruct(16, 16, pl.n_buckets, 16, 16, pl.n_raw_segments, pl.n_raw, pl.n, 1)    # non-null, never read
    assert L.qsgd_policy_message_capacity(C.byref(good), 512, 15, 0) == \
        pl.raw_prefix + Q.qsgd_message_capacity(pl.n_buckets * 512, 512, 15, 0)
    assert L.qsgd_policy_message_capacity(C.byref(good), 100, 15, 0) == 0                        # bad bucket
    assert L.qsgd_policy_workspace_bytes(C.byref(good), 512, 15, 0) == 0                         # fixed-width: none
    assert L.qsgd_policy_workspace_bytes(C.byref(good), 512, 15, 1) == Q.qsgd_workspace_bytes(pl.n_buckets * 512, 512, 15, 1)
    msgs = (C.c_void_p * 1)(16)
    assert L.qsgd_policy_decode_sgd_step(msgs, None, None, 0, C.byref(good), 512, 15, 0, 16, 0.1, 16, None) == -7   # K = 0
    assert L.qsgd_policy_decode_sgd_step(msgs, None, None, 1, C.byref(good), 512, 15, 0, 8, 0.1, 16, None) == -5    # x misaligned
    assert L.qsgd_policy_decode_sgd_step(msgs, None, None, 1, C.byref(good), 512, 15, 1, 16, 0.1, 16, None) == -1   # Elias needs tables
