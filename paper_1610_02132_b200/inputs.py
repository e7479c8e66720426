"""Seeded synthetic gradients with the shapes and value distributions of the QSGD workloads.

This module only draws random inputs (numpy on the host, torch generators on a device). It holds
none of the method's arithmetic: no norm, no rounding, no code. The same bytes are handed to the
CUDA path and to the CPU checker, so parity never depends on the generator.

The paper's experiments quantize gradients of ImageNet / CIFAR-10 / AN4 networks; those need
datasets and training runs, so the vectors below stand in for their shapes and magnitudes only.
"""
import math

import numpy as np


def _rng(seed):
    return np.random.Generator(np.random.PCG64(int(seed)))


def gaussian(n, sigma=1.0, seed=0):
    """n i.i.d. N(0, sigma^2) fp32 values."""
    return (_rng(seed).standard_normal(n, dtype=np.float32) * np.float32(sigma)).astype(np.float32)


def sparse_laplace(n, scale=1e-3, zero_frac=0.3, seed=0):
    """Laplace(0, scale) values with a seeded Bernoulli(zero_frac) mask set exactly to zero."""
    r = _rng(seed)
    v = r.laplace(0.0, scale, n).astype(np.float32)
    v[r.random(n) < zero_frac] = 0.0
    return v


def gaussian_mixture(n, seed=0, w_small=0.9, sigma_small=1e-4, sigma_large=1e-2):
    """Every element from w_small * N(0, sigma_small^2) + (1 - w_small) * N(0, sigma_large^2)."""
    r = _rng(seed)
    v = r.standard_normal(n, dtype=np.float32)
    sig = np.where(r.random(n) < w_small, np.float32(sigma_small), np.float32(sigma_large))
    return (v * sig.astype(np.float32)).astype(np.float32)


def alexnet_shapes():
    """Parameter tensors of the 5-conv + 3-FC AlexNet, weight then bias per layer (61 100 840)."""
    conv = [(64, 3, 11, 11), (192, 64, 5, 5), (384, 192, 3, 3), (256, 384, 3, 3), (256, 256, 3, 3)]
    fc = [(4096, 9216), (4096, 4096), (1000, 4096)]
    shapes = []
    for w in conv + fc:
        shapes.append(w)
        shapes.append((w[0],))
    return shapes


def resnet152_shapes():
    """Parameter tensors of ResNet-152 (bottleneck stages [3, 8, 36, 3]); total 60 192 808."""
    shapes = [(64, 3, 7, 7), (64,), (64,)]
    inplanes = 64
    for planes, blocks in zip((64, 128, 256, 512), (3, 8, 36, 3)):
        for blk in range(blocks):
            shapes += [(planes, inplanes, 1, 1), (planes,), (planes,)]
            shapes += [(planes, planes, 3, 3), (planes,), (planes,)]
            shapes += [(planes * 4, planes, 1, 1), (planes * 4,), (planes * 4,)]
            if blk == 0:
                shapes += [(planes * 4, inplanes, 1, 1), (planes * 4,), (planes * 4,)]
            inplanes = planes * 4
    shapes += [(1000, 2048), (1000,)]
    return shapes


def numel(shapes):
    return int(sum(math.prod(s) for s in shapes))


def fan_in(shape, prev_fan_in):
    """in_channels * kh * kw or in_features; a bias shares the fan-in of its layer."""
    return math.prod(shape[1:]) if len(shape) > 1 else prev_fan_in


def layered_gaussian(shapes, seed=0, base_sigma=1e-2):
    """Flat concatenation; tensor L drawn N(0, (base_sigma / sqrt(fan_in_L))^2)."""
    r = _rng(seed)
    parts, fi = [], 1
    for s in shapes:
        fi = fan_in(s, fi)
        sigma = np.float32(base_sigma / math.sqrt(fi))
        parts.append(r.standard_normal(math.prod(s), dtype=np.float32) * sigma)
    return np.concatenate(parts).astype(np.float32)


def layer_sigmas(shapes, base_sigma=1e-2):
    """Per-element sigma of layered_gaussian as (start, stop, sigma) segments."""
    segs, fi, pos = [], 1, 0
    for s in shapes:
        fi = fan_in(s, fi)
        m = math.prod(s)
        segs.append((pos, pos + m, base_sigma / math.sqrt(fi)))
        pos += m
    return segs


# ------------------------------- device-side generators -------------------------------------
# For the large workloads the gradients are drawn directly in HBM with a seeded torch generator;
# a test that needs the values on the host copies them back, so both sides still see the same
# bytes.

def _gen(device, seed):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian_device(n, sigma=1.0, seed=0, device="cuda"):
    import torch
    out = torch.empty(n, dtype=torch.float32, device=device)
    out.normal_(0.0, float(sigma), generator=_gen(device, seed))
    return out


def sparse_laplace_device(n, scale=1e-3, zero_frac=0.3, seed=0, device="cuda"):
    import torch
    g = _gen(device, seed)
    u = torch.rand(n, dtype=torch.float32, device=device, generator=g) - 0.5
    v = -float(scale) * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.49999997))
    mask = torch.rand(n, dtype=torch.float32, device=device, generator=g) < zero_frac
    v[mask] = 0.0
    return v.contiguous()


def gaussian_mixture_device(n, seed=0, w_small=0.9, sigma_small=1e-4, sigma_large=1e-2,
                            device="cuda"):
    import torch
    g = _gen(device, seed)
    v = torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g)
    pick = torch.rand(n, dtype=torch.float32, device=device, generator=g) < w_small
    v.mul_(torch.where(pick, float(sigma_small), float(sigma_large)))
    return v


def layered_gaussian_device(shapes, seed=0, base_sigma=1e-2, device="cuda"):
    import torch
    g = _gen(device, seed)
    out = torch.empty(numel(shapes), dtype=torch.float32, device=device)
    out.normal_(0.0, 1.0, generator=g)
    for lo, hi, sig in layer_sigmas(shapes, base_sigma):
        out[lo:hi].mul_(float(sig))
    return out


# ---- finite-sum problem for the variance-reduced variant (Section 3.3) -------------------------------
def least_squares_problem(m, n, seed=0, noise=0.01):
    """m unit-norm random rows A[m, n] and targets b = A x_true + noise (fp32). With the ridge term
    the functions f_j(x) = (a_j . x - b_j)^2 / 2 + lam |x|^2 / 2 are (1 + lam)-smooth and their mean
    is at least lam-strongly convex, so the condition number is set by lam."""
    r = _rng(seed)
    A = r.standard_normal((m, n)).astype(np.float64)
    A /= np.linalg.norm(A, axis=1, keepdims=True)
    x_true = r.standard_normal(n)
    b = A @ x_true + noise * r.standard_normal(m)
    return A.astype(np.float32), b.astype(np.float32)


def sample_indices(P, T, K, m, seed=0):
    """The uniformly random function indices j[p, t, i] in [0, m) that the K processors draw."""
    return _rng(seed).integers(0, m, size=(P, T, K), dtype=np.int64)
