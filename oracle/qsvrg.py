"""CPU statement of QSVRG (Section 3.3 and its appendix, "Quantized SVRG") on top of the oracle codec.

TEST INFRASTRUCTURE ONLY, like oracle.py. Written step by step in the paper's order:

  epoch p:   x_1 = y^(p) (appendix, "Background on SVRG": every epoch starts from its own average);
             every processor i quantizes the gradient of its share h_i at y^(p) and broadcasts it,
             H_p = sum_i Q~(grad h_i(y^(p)))                                   (appendix form);
  t = 1..T:  processor i draws j, broadcasts u_i = Q~(grad f_j(x_t) - grad f_j(y^(p)) + H_p),
             x_(t+1) = x_t - eta * (1 / K) * sum_i u_i;
  end:       y^(p+1) = (1 / T) * sum_t x_t.

Q~(v) = Q(v, s) with s = floor(sqrt(n)) levels and the 2-norm of the whole vector (one bucket = n);
the max-norm of Section 4 can be chosen instead.
Every broadcast goes through Encode and Decode of the oracle, so message bits are the paper's
|Code'_s| (or |Code_s|, or the fixed-width size). The gradients come from caller-supplied functions so
that a test can hand the same arithmetic to this file and to the GPU path.
"""
import numpy as np

from . import oracle as O


def default_levels(n):
    return min(int(np.floor(np.sqrt(n))), 255)


def qsvrg(grad_share, grad_sample, n, K, P, T, eta, indices, x0, code_kind=O.CODE_ELIAS_DENSE, s=None,
          seed=7, quantize_full=True, norm_kind=O.NORM_L2):
    """grad_share(i, y) -> grad h_i(y); grad_sample(j, x) -> grad f_j(x); indices[p, t, i] = j.
    quantize_full: the appendix quantizes the per-epoch broadcast of grad h_i, the main text sends it
    in full precision (then H_p is the fp32 sum in processor order and costs 32 n bits each).
    Returns dict(y=[y^(1) .. y^(P+1)], x=x_final, bits=[per processor message bits, summed])."""
    s = default_levels(n) if s is None else s
    x = np.asarray(x0, dtype=np.float32).copy()
    y = x.copy()
    ys = [y.copy()]
    bits = np.zeros(K, dtype=np.int64)

    def broadcast(vectors, step):
        """Every processor encodes its vector; returns the messages as all processors decode them."""
        msgs, tabs = [], []
        for i, v in enumerate(vectors):
            m, info = O.encode(np.asarray(v, dtype=np.float32), n, s, norm_kind, code_kind, seed, step, i)
            bits[i] += info[0]
            msgs.append(m)
            tabs.append(None if code_kind == O.CODE_FIXED else O.message_table(m, info, n, n))
        return msgs, (None if code_kind == O.CODE_FIXED else tabs)

    for p in range(P):
        step0 = p * (T + 1)
        x = y.copy()                                                           # x_1^(p) = y^(p)
        shares = [np.asarray(grad_share(i, y), dtype=np.float32) for i in range(K)]
        if quantize_full:
            msgs, tabs = broadcast(shares, step0)
            st, H = O.decode_accumulate(msgs, tabs, n, n, s, code_kind)       # H_p = sum_i Q~(grad h_i)
            assert st == 0
        else:
            H = np.zeros(n, dtype=np.float32)
            for g in shares:
                H = (H + g).astype(np.float32)                                 # grad f(y) = sum_i grad h_i
            bits += 32 * n
        x_sum = np.zeros(n, dtype=np.float64)
        for t in range(T):
            x_sum += x                                                         # the average runs over x_1 .. x_T
            us = []
            for i in range(K):
                j = int(indices[p, t, i])
                us.append((grad_sample(j, x) - grad_sample(j, y)).astype(np.float32) + H)
            msgs, tabs = broadcast(us, step0 + 1 + t)
            st, acc = O.decode_accumulate(msgs, tabs, n, n, s, code_kind)
            assert st == 0
            x = O.sgd_step(x, acc, eta, K)                                     # x - eta * (1 / K) * sum_i u_i
        y = (x_sum / T).astype(np.float32)
        ys.append(y.copy())
    return {"y": ys, "x": x, "bits": bits}
