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
