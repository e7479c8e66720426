"""The benchmark's step (K encodes, then the fused decode) gives the same bytes whether the K
independent encodes are issued on one stream or round-robin on several, and those are the oracle's."""
import numpy as np
import pytest
import torch

import bench
from oracle import oracle as O
from paper_1610_02132_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("codes", [["fixed", "elias"], ["elias_dense"]])
@pytest.mark.parametrize("policy", [None, "sizes"])
def test_step_on_one_and_on_three_streams(codes, policy, monkeypatch):
    sizes = [4096 * 5 + 8, 120, 20480, 9000, 4096 * 3]
    n = sum(sizes) if policy else 4096 * 11 + 300
    wl = dict(n=n, d=512, s=15, norm="max", codes=codes, K=5, gen="mixture", desc="test")
    if policy:
        wl["policy"] = "test"
        monkeypatch.setattr(bench, "policy_sizes", lambda name: sizes)
    dev = torch.device("cuda", 0)
    got = {}
    for streams in (1, 3):
        hp = bench.HotPath(wl, dev, streams=streams)
        hp.x.copy_(torch.from_numpy(I.gaussian(n, 1.0, seed=3)).to(dev))
        for step in range(2):
            hp.step(step)
        torch.cuda.synchronize()
        assert int(hp.status.item()) == 0
        got[streams] = (hp.x.cpu().numpy(), {c: [m.cpu().numpy() for m in hp.msgs[c]] for c in hp.codes},
                        {c: hp.bits[c].cpu().numpy() for c in hp.codes}, hp.g[0].cpu().numpy())
    assert np.array_equal(got[1][0].view(np.uint32), got[3][0].view(np.uint32))
    for c in got[1][1]:
        assert np.array_equal(got[1][2][c], got[3][2][c])
        for w, (a, b) in enumerate(zip(got[1][1][c], got[3][1][c])):
            nbytes = int(got[1][2][c][w][2])
            assert np.array_equal(a[:nbytes], b[:nbytes])
    if policy is None:
        # against the oracle: the last step's messages of worker 0 (max-norm: exact scales)
        for cname in codes:
            code = bench.CODE[cname]
            m, info = O.encode(got[3][3], 512, 15, O.NORM_MAX, code, bench.PHILOX_SEED, 1, 0)
            assert np.array_equal(got[3][1][code][0][: m.size], m)
