"""QSVRG (Section 3.3 and its appendix): the variance-reduced variant, orchestrated on the host around
the library's Encode / Decode. Every epoch starts its iterate at the epoch's own point, x_1 = y^(p)
(appendix, "Background on SVRG"). Every broadcast vector is encoded by `qsgd_encode` with one bucket
spanning the whole vector (bucket = n <= 4096), s = floor(sqrt(n)) levels and the 2-norm, and the K
messages of an iteration are decoded, averaged and applied by one `qsgd_decode_sgd_step`
(x <- x - (eta / K) * sum_i u_i is exactly the paper's x_(t+1) = x_t - eta * u_t). The per-epoch sum
H_p = sum_i Q~(grad h_i) is one `qsgd_decode_accumulate`.

The gradients are the caller's: grad_share(i, y) and grad_sample(j, x) return CUDA fp32 tensors (or
anything `torch.as_tensor` accepts, e.g. numpy arrays in a test). `least_squares_gradients` supplies
them for f_j(x) = (a_j . x - b_j)^2 / 2 + lam |x|^2 / 2 with torch operations on the device.
"""
import math

import numpy as np
import torch

from . import binding as Q


def default_levels(n):
    return min(int(math.floor(math.sqrt(n))), 255)


def least_squares_gradients(A, b, lam, K):
    """(grad_share, grad_sample) for rows A[m, n], targets b[m] (CUDA fp32), m divisible by K."""
    m = A.shape[0]
    share = m // K

    def grad_share(i, y):
        Ai, bi = A[i * share:(i + 1) * share], b[i * share:(i + 1) * share]
        return (Ai.t() @ (Ai @ y - bi)) / m + (lam / K) * y

    def grad_sample(j, x):
        """One function index, or a tensor of K indices: then a [K, n] tensor, one row per index."""
        if torch.is_tensor(j) and j.dim() == 1:
            a = A[j]                                              # [K, n]
            return a * (a @ x - b[j]).unsqueeze(1) + lam * x
        a = A[j]
        return a * (torch.dot(a, x) - b[j]) + lam * x

    grad_sample.batched = True
    return grad_share, grad_sample


def qsvrg(grad_share, grad_sample, n, K, P, T, eta, indices, x0, code_kind=Q.CODE_ELIAS_DENSE, s=None, seed=7,
          quantize_full=True, norm_kind=Q.NORM_L2, device="cuda"):
    """Runs P epochs of T iterations. indices[p, t, i] is the function index processor i draws.
    Returns dict(y=[y^(1) .. y^(P+1)] (CPU numpy), x (CUDA tensor), bits (per processor, numpy int64))."""
    if n % 32 or n > 4096:
        raise Q.QsgdError("QSVRG here quantizes the whole vector as one bucket: n must be a multiple of 32, at most 4096")
    s = default_levels(n) if s is None else s
    dev = torch.device(device)
    x = torch.as_tensor(x0, dtype=torch.float32).to(dev).clone()
    y = x.clone()
    ys = [y.cpu().numpy().copy()]
    cap = Q.qsgd_message_capacity(n, n, s, code_kind)
    msgs = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(K)]
    info = torch.zeros(K, 4, dtype=torch.int64, device=dev)
    total_bits = torch.zeros(K, dtype=torch.int64, device=dev)
    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, n, s, code_kind), 16), dtype=torch.uint8, device=dev)
    status = Q.new_status(dev)
    H = torch.zeros(n, dtype=torch.float32, device=dev)
    own_tables = torch.zeros(K, 2, dtype=torch.int64, device=dev)
    idx_dev = torch.as_tensor(np.asarray(indices), dtype=torch.int64).to(dev)

    def broadcast(vectors, step):
        for i, v in enumerate(vectors):
            v = torch.as_tensor(v, dtype=torch.float32).to(dev).contiguous()
            Q.qsgd_encode(v, n, s, norm_kind, code_kind, seed, step, i, msgs[i], info[i], ws, status)
        total_bits.add_(info[:, 0])
        if code_kind == Q.CODE_FIXED:
            return None
        # One bucket per message: its offset table is (0, payload bits). Building it on the device
        # from the size words avoids reading the table's place in the message back to the host.
        own_tables[:, 1] = info[:, 0]
        return [own_tables[i] for i in range(K)]

    for p in range(P):
        step0 = p * (T + 1)
        x.copy_(y)                                                # every epoch starts at x_1 = y^(p)
        shares = [grad_share(i, y) for i in range(K)]
        if quantize_full:
            tables = broadcast(shares, step0)
            Q.qsgd_decode_accumulate(msgs, tables, n, n, s, code_kind, H, status)
        else:
            H.zero_()
            for g in shares:
                H.add_(torch.as_tensor(g, dtype=torch.float32).to(dev))
            total_bits.add_(32 * n)
        x_sum = torch.zeros(n, dtype=torch.float64, device=dev)
        for t in range(T):
            x_sum.add_(x.double())
            if getattr(grad_sample, "batched", False):            # all K update vectors in a few tensor operations
                js = idx_dev[p, t]
                us = (grad_sample(js, x) - grad_sample(js, y)) + H
            else:
                us = []
                for i in range(K):
                    j = int(indices[p, t, i])
                    gx = torch.as_tensor(grad_sample(j, x), dtype=torch.float32).to(dev)
                    gy = torch.as_tensor(grad_sample(j, y), dtype=torch.float32).to(dev)
                    us.append((gx - gy) + H)
            tables = broadcast(us, step0 + 1 + t)
            Q.qsgd_decode_sgd_step(msgs, tables, n, n, s, code_kind, x, eta, status)
        # a true fp64 division (a tensor divisor: a Python scalar would be turned into a multiplication)
        y = torch.div(x_sum, torch.full((1,), float(T), dtype=torch.float64, device=dev)).float()
        ys.append(y.cpu().numpy().copy())
    if int(status.item()) != 0:
        raise Q.QsgdError("device status %d during QSVRG" % int(status.item()))
    return {"y": ys, "x": x, "bits": total_bits.cpu().numpy()}
