"""Pins for the oracle's Q_s (Eq. 2, Lemma 3.1, bucketing and max-norm of Section 4) -- CPU only.

Everything the oracle is compared with here is computed independently in fp64 numpy from the
paper's formulas: interval index l = floor(s a), p(a, s) = a s - l, the variance term
||v||^2 / s^2 * sum p (1 - p) of the lemma's proof, and exhaustive enumeration of outcomes.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import oracle as O

TRIALS = 10000


def fp64_model(v, s, norm_kind):
    v = v.astype(np.float64)
    A = math.sqrt(float(np.sum(v * v))) if norm_kind == O.NORM_L2 else float(np.max(np.abs(v)))
    a = np.abs(v) / A
    low = np.floor(s * a)
    low = np.minimum(low, s - 1) if s >= 1 else low      # a = 1 belongs to the top interval
    p = s * a - low
    return A, low, p


def draws(v, s, norm_kind, seed, trials=TRIALS):
    """`trials` independent quantizations of v: v repeated as `trials` buckets of size len(v)."""
    n = v.size
    g = np.tile(v, trials).astype(np.float32)
    A = O.bucket_scales(g, n, norm_kind)
    lv, sg = O.quantize(g, n, s, A, seed, 3, 1)
    q = O.dequantize(A, lv, sg, n, s)
    return A, lv.reshape(trials, n), sg.reshape(trials, n), q.reshape(trials, n).astype(np.float64)


VECS = {
    1: [2.5], 2: [3.0, -4.0], 5: [0.1, -0.7, 0.0, 2.0, -0.05],
    8: [1.0, -2.0, 0.5, 0.25, -0.125, 3.0, 0.0, -1.5],
    64: list(np.random.default_rng(11).standard_normal(64)),
}


@pytest.mark.parametrize("n", [1, 2, 5, 8, 64])
@pytest.mark.parametrize("s", [1, 3, 15, 255])
@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
def test_lemma_3_1_monte_carlo(n, s, norm_kind):
    v = np.array(VECS[n], dtype=np.float32)
    A64, low, p = fp64_model(v, s, norm_kind)
    A, lv, sg, q = draws(v, s, norm_kind, seed=1000 + n + s)
    assert np.allclose(A, A64, rtol=1e-6)
    # (i) unbiased: per-coordinate mean within 5 sigma of v
    sd = A64 / s * np.sqrt(p * (1 - p))
    err = np.abs(q.mean(axis=0) - v.astype(np.float64))
    assert np.all(err <= 5 * sd / math.sqrt(TRIALS) + 1e-6 * np.abs(v))
    # support: each level is floor or floor + 1, sign follows v, zero maps to zero
    assert np.all((lv == low) | (lv == low + 1))
    assert np.all(sg[:, v >= 0] == 0)
    assert np.all(sg[:, v < 0] == (lv[:, v < 0] > 0))
    # level-up frequency is p(a, s)
    up = (lv == low + 1).mean(axis=0)
    assert np.all(np.abs(up - p) <= 5 * np.sqrt(p * (1 - p) / TRIALS) + 2e-5)
    # (ii) variance: Monte-Carlo vs the proof's exact term, and vs the lemma's bound (2-norm)
    var_mc = np.mean(np.sum((q - v.astype(np.float64)) ** 2, axis=1))
    var_exact = A64 ** 2 / s ** 2 * float(np.sum(p * (1 - p)))
    assert abs(var_mc - var_exact) <= 0.08 * var_exact + 1e-12
    if norm_kind == O.NORM_L2:
        assert var_mc <= min(n / s ** 2, math.sqrt(n) / s) * A64 ** 2 * 1.02 + 1e-12
        # (iii) sparsity in the lemma's form s (s + sqrt n). (The appendix restates it as
        # s^2 + sqrt n; its proof takes P[nonzero] = u_i where Eq. 2 gives s u_i, and that
        # form is exceeded for s > 1 -- e.g. n = 64, s = 3 -- so only the lemma's form is
        # asserted.) s = 1: E nnz = ||v||_1 / ||v||_2 exactly, from p(a, 1) = a.
        nnz = (lv > 0).sum(axis=1).mean()
        assert nnz <= s * (s + math.sqrt(n)) + 0.05
        exact_nnz = float(np.sum(np.where(low > 0, 1.0, p)))
        assert abs(nnz - exact_nnz) <= 0.05 * math.sqrt(n)
        if s == 1:
            assert abs(nnz - np.abs(v).sum() / A64) <= 0.05 * math.sqrt(n)


@pytest.mark.parametrize("s", [1, 2, 3, 7, 15])
@pytest.mark.parametrize("norm_kind", [O.NORM_L2, O.NORM_MAX])
def test_exhaustive_enumeration_small_n(s, norm_kind):
    rng = np.random.default_rng(100 + s)
    for n in (1, 2, 3, 5, 8):
        v = rng.standard_normal(n).astype(np.float32)
        if n >= 3:
            v[1] = 0.0
        A64, low, p = fp64_model(v, s, norm_kind)
        A = O.bucket_scales(v, n, norm_kind)
        v64 = v.astype(np.float64)
        mean = np.zeros(n)
        second = 0.0
        total = 0.0
        for ups in itertools.product((0, 1), repeat=n):
            ups = np.array(ups)
            prob = float(np.prod(np.where(ups == 1, p, 1 - p)))
            if prob == 0.0:
                continue
            # uniforms that select exactly this outcome: up iff u >= 1 - p
            u = np.where(ups == 1, (1 - p) + p / 2, (1 - p) / 2).astype(np.float32)
            lv, sg = O.quantize_with_uniforms(v, n, s, A, u)
            assert np.array_equal(lv, (low + ups).astype(np.uint8)), (v, ups, lv)
            q = O.dequantize(A, lv, sg, n, s).astype(np.float64)
            q_model = A64 * np.sign(v64) * (low + ups) / s
            assert np.allclose(q, q_model, rtol=3e-7, atol=0)
            mean += prob * q_model
            second += prob * float(np.sum((q_model - v64) ** 2))
            total += prob
        assert abs(total - 1) < 1e-12
        assert np.allclose(mean, v64, rtol=1e-12, atol=1e-15)                 # E Q = v
        assert math.isclose(second, A64 ** 2 / s ** 2 * float(np.sum(p * (1 - p))),
                            rel_tol=1e-9, abs_tol=1e-15)
        if norm_kind == O.NORM_L2:
            assert second <= min(n / s ** 2, math.sqrt(n) / s) * A64 ** 2 + 1e-12


def test_philox_draw_selects_the_outcome():
    # With the keyed uniforms: level goes up iff u_i >= 1 - p_i (away from the threshold).
    rng = np.random.default_rng(3)
    g = rng.standard_normal(4096).astype(np.float32)
    d, s = 8, 5
    A = O.bucket_scales(g, d, O.NORM_L2)
    lv, sg = O.quantize(g, d, s, A, 99, 4, 2)
    u = np.array([O.uniform(99, 4, 2, i) for i in range(g.size)])
    a = np.abs(g.astype(np.float64)) / np.repeat(A.astype(np.float64), d)
    low = np.floor(s * a)
    p = s * a - low
    clear = np.abs(u - (1 - p)) > 1e-5
    assert clear.mean() > 0.99
    assert np.array_equal(lv[clear], (low + (u >= 1 - p))[clear].astype(np.uint8))


def test_global_index_offset():
    g = np.random.default_rng(4).standard_normal(1024).astype(np.float32)
    d, s = 64, 15
    A = O.bucket_scales(g, d, O.NORM_MAX)
    lv, sg = O.quantize(g, d, s, A, 5, 0, 0)
    lo = 5 * d
    lv2, sg2 = O.quantize(g[lo:lo + 3 * d], d, s, A[5:8], 5, 0, 0, i0=lo)
    assert np.array_equal(lv[lo:lo + 3 * d], lv2) and np.array_equal(sg[lo:lo + 3 * d], sg2)


def test_special_cases():
    # Q(0) = 0; subnormal scale counts as zero; -0.0 decodes to +0.0
    z = np.zeros(16, dtype=np.float32)
    z[3] = -0.0
    for kind in (O.NORM_L2, O.NORM_MAX):
        A = O.bucket_scales(z, 16, kind)
        assert A[0] == 0 and not np.signbit(A[0])
        lv, sg = O.quantize(z, 16, 15, A, 1, 0, 0)
        assert not lv.any() and not sg.any()
        q = O.dequantize(A, lv, sg, 16, 15)
        assert not q.any() and not np.signbit(q).any()
        tiny = np.full(16, 1e-41, dtype=np.float32)
        assert O.bucket_scales(tiny, 16, kind)[0] == 0
    # d = 1 with power-of-two values: no quantization at all (Section 4: d = 1 is vanilla SGD)
    v = np.array([0.5, -2.0, 8.0, -0.125], dtype=np.float32)
    for kind in (O.NORM_L2, O.NORM_MAX):
        A = O.bucket_scales(v, 1, kind)
        lv, sg = O.quantize(v, 1, 7, A, 1, 0, 0)
        assert np.array_equal(O.dequantize(A, lv, sg, 1, 7), v)
    # s = 1 is ternary {-A, 0, +A}; with max-norm the max element is always kept at level 1
    g = np.random.default_rng(8).standard_normal(512).astype(np.float32)
    g[17] = 9.0
    A = O.bucket_scales(g, 512, O.NORM_MAX)
    assert A[0] == 9.0
    lv, sg = O.quantize(g, 512, 1, A, 3, 0, 0)
    q = O.dequantize(A, lv, sg, 512, 1)
    assert set(np.unique(q)) <= {-9.0, 0.0, 9.0} and q[17] == 9.0
    # a single nonzero element under the 2-norm: level s, decoded exactly
    e = np.zeros(64, dtype=np.float32)
    e[5] = -3.25
    A = O.bucket_scales(e, 64, O.NORM_L2)
    lv, sg = O.quantize(e, 64, 15, A, 3, 0, 0)
    assert lv[5] == 15 and sg[5] == 1 and O.dequantize(A, lv, sg, 64, 15)[5] == -3.25
    # tail bucket gets its own scale
    t = np.arange(1, 11, dtype=np.float32)
    A = O.bucket_scales(t, 4, O.NORM_MAX)
    assert list(A) == [4.0, 8.0, 10.0]
    # bucketed variance example printed in Section 4: d = 512, "4 bits" -> sqrt(512)/2^4 ~ 1.41
    assert abs(math.sqrt(512) / 2 ** 4 - 1.41) < 0.005
