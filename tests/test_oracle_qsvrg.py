"""Pins for the oracle's QSVRG (Section 3.3; appendix "Quantized SVRG") on a synthetic ridge
least-squares problem whose minimiser is known in closed form (normal equations, fp64)."""
import numpy as np
import pytest

from oracle import oracle as O
from oracle import qsvrg as QV
from paper_1610_02132_b200 import inputs as I

M, N, K, LAM = 1024, 256, 4, 0.1


def problem(seed=1):
    A, b = I.least_squares_problem(M, N, seed=seed)
    A64, b64 = A.astype(np.float64), b.astype(np.float64)
    share = M // K

    def f(x):
        r = A64 @ x - b64
        return 0.5 * np.mean(r * r) + 0.5 * LAM * np.dot(x, x)

    def grad_share(i, y):
        Ai, bi = A64[i * share:(i + 1) * share], b64[i * share:(i + 1) * share]
        y = np.asarray(y, dtype=np.float64)
        return ((Ai.T @ (Ai @ y - bi)) / M + LAM * y / K).astype(np.float32)

    def grad_sample(j, x):
        x = np.asarray(x, dtype=np.float64)
        return (A64[j] * (A64[j] @ x - b64[j]) + LAM * x).astype(np.float32)

    x_star = np.linalg.solve(A64.T @ A64 / M + LAM * np.eye(N), A64.T @ b64 / M)
    return f, grad_share, grad_sample, x_star


L_SMOOTH, ELL = 1.0 + LAM, LAM                    # unit rows: each f_j is (1 + lam)-smooth, f is lam-strongly convex
T_ITERS, ETA = int(20 * L_SMOOTH / ELL), 0.1 / L_SMOOTH


@pytest.mark.parametrize("quantize_full", [True, False])
def test_rate_of_theorem_3_6(quantize_full):
    """f(y^(p+1)) - f* <= 0.9^p (f(y^(1)) - f*) with eta = O(1 / L), T = O(L / l)."""
    f, gs, gj, x_star = problem()
    P = 5
    idx = I.sample_indices(P, T_ITERS, K, M, seed=3)
    out = QV.qsvrg(gs, gj, N, K, P, T_ITERS, ETA, idx, np.zeros(N, np.float32), quantize_full=quantize_full)
    gap = [f(y.astype(np.float64)) - f(x_star) for y in out["y"]]
    assert all(g >= -1e-12 for g in gap)
    for p in range(1, P + 1):
        assert gap[p] <= 0.9 ** p * gap[0]
    assert gap[2] < 0.1 * gap[0]                  # and in fact far faster on this well-conditioned problem


def test_bits_per_processor_against_the_stated_bound():
    """P (F + 2.8 n)(T + 1) bits per processor with the dense code at s = sqrt(n) (F = 32). The 2.8 is
    asymptotic (the literal code spends 2 / 4 / 4 / 7 bits on levels 0 / 1 / 2 / 3), so within 20 %."""
    f, gs, gj, x_star = problem()
    P = 2
    idx = I.sample_indices(P, T_ITERS, K, M, seed=4)
    out = QV.qsvrg(gs, gj, N, K, P, T_ITERS, ETA, idx, np.zeros(N, np.float32), code_kind=O.CODE_ELIAS_DENSE)
    bound = P * (32 + 2.8 * N) * (T_ITERS + 1)
    assert np.all(out["bits"] <= 1.2 * bound)
    assert np.all(out["bits"] >= 0.5 * bound)      # not trivially small either: every coordinate is coded
    # the fixed-width message of the same quantizer costs 1 + 8 bits per coordinate (s = 16 needs 8 level bits)
    out_f = QV.qsvrg(gs, gj, N, K, P, T_ITERS, ETA, idx, np.zeros(N, np.float32), code_kind=O.CODE_FIXED)
    assert np.all(out_f["bits"] > 2 * out["bits"])


def test_code_kind_does_not_change_the_iterates():
    """The three codes are lossless encodings of the same Q_s(v): identical trajectories, bit for bit."""
    f, gs, gj, _ = problem(seed=2)
    idx = I.sample_indices(2, 40, K, M, seed=5)
    runs = [QV.qsvrg(gs, gj, N, K, 2, 40, ETA, idx, np.zeros(N, np.float32), code_kind=c)
            for c in (O.CODE_FIXED, O.CODE_ELIAS, O.CODE_ELIAS_DENSE)]
    for r in runs[1:]:
        assert np.array_equal(r["x"].view(np.uint32), runs[0]["x"].view(np.uint32))
        assert all(np.array_equal(a, b) for a, b in zip(r["y"], runs[0]["y"]))


def test_fine_quantization_tracks_plain_svrg():
    """With s = 255 levels on n = 64 coordinates the quantization error is small: the iterates stay
    close to SVRG computed here without any quantizer (same indices, same arithmetic order)."""
    n, m, k = 64, 256, 2
    A, b = I.least_squares_problem(m, n, seed=7)
    A64, b64 = A.astype(np.float64), b.astype(np.float64)
    share = m // k
    gs = lambda i, y: ((A64[i * share:(i + 1) * share].T @ (A64[i * share:(i + 1) * share] @ np.asarray(y, np.float64)
                        - b64[i * share:(i + 1) * share])) / m + LAM * np.asarray(y, np.float64) / k).astype(np.float32)
    gj = lambda j, x: (A64[j] * (A64[j] @ np.asarray(x, np.float64) - b64[j]) + LAM * np.asarray(x, np.float64)).astype(np.float32)
    P, T = 2, 60
    idx = I.sample_indices(P, T, k, m, seed=8)
    out = QV.qsvrg(gs, gj, n, k, P, T, ETA, idx, np.zeros(n, np.float32), code_kind=O.CODE_FIXED, s=255)
    x = np.zeros(n)
    y = x.copy()
    for p in range(P):
        x = y.copy()                          # SVRG as the appendix states it: x_1^(p) = y^(p)
        H = sum(gs(i, y).astype(np.float64) for i in range(k))
        xs = np.zeros(n)
        for t in range(T):
            xs += x
            u = np.mean([gj(int(idx[p, t, i]), x).astype(np.float64) - gj(int(idx[p, t, i]), y) + H for i in range(k)], axis=0)
            x = x - ETA * u
        y = xs / T
    assert np.linalg.norm(out["x"] - x) <= 0.05 * np.linalg.norm(x)
    assert np.linalg.norm(out["y"][-1] - y) <= 0.05 * np.linalg.norm(y)
