"""ctypes front end of the CPU oracle (oracle/qsgd_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of
bench.py. Nothing in the product package imports this module, and this module imports nothing
from the product package.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qsgd_oracle.cpp")
_LIB = os.path.join(_HERE, "libqsgd_oracle.so")

NORM_L2, NORM_MAX = 0, 1
CODE_FIXED, CODE_ELIAS, CODE_ELIAS_DENSE = 0, 1, 2

CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force=False):
    """Compile the oracle with g++ (no FMA contraction, no fast-math). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++"] + CXXFLAGS + [_SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u32p, u64p, f32p = (C.POINTER(t) for t in (C.c_uint8, C.c_uint32, C.c_uint64, C.c_float))
        L.oq_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.oq_philox4x32_10.restype = None
        L.oq_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
        L.oq_uniform.restype = C.c_float
        L.oq_level_bits.argtypes = [C.c_uint32]
        L.oq_level_bits.restype = C.c_int
        L.oq_bucket_scales.argtypes = [f32p, C.c_uint64, C.c_uint32, C.c_int, f32p]
        L.oq_bucket_scales.restype = None
        L.oq_quantize.argtypes = [f32p, C.c_uint64, C.c_uint32, C.c_uint32, f32p, C.c_uint64,
                                  C.c_uint32, C.c_uint32, C.c_uint64, u8p, u8p]
        L.oq_quantize.restype = None
        L.oq_quantize_with_uniforms.argtypes = [f32p, C.c_uint64, C.c_uint32, C.c_uint32, f32p,
                                                f32p, u8p, u8p]
        L.oq_quantize_with_uniforms.restype = None
        L.oq_dequantize.argtypes = [f32p, u8p, u8p, C.c_uint64, C.c_uint32, C.c_uint32, f32p]
        L.oq_dequantize.restype = None
        L.oq_fixed_layout.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, u64p]
        L.oq_fixed_layout.restype = None
        L.oq_fixed_pack.argtypes = [f32p, u8p, u8p, C.c_uint64, C.c_uint32, C.c_uint32, u8p]
        L.oq_fixed_pack.restype = None
        L.oq_fixed_unpack.argtypes = [u8p, C.c_uint64, C.c_uint32, C.c_uint32, f32p, u8p, u8p]
        L.oq_fixed_unpack.restype = None
        L.oq_elias_string.argtypes = [C.c_uint64, C.c_char_p]
        L.oq_elias_string.restype = C.c_int
        L.oq_elias_parse.argtypes = [C.c_char_p, C.c_int, u64p]
        L.oq_elias_parse.restype = C.c_int
        L.oq_elias_pack.argtypes = [f32p, u8p, u8p, C.c_uint64, C.c_uint32, C.c_int, u8p,
                                    C.c_uint64, u64p]
        L.oq_elias_pack.restype = C.c_uint64
        L.oq_elias_unpack.argtypes = [u8p, u64p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int,
                                      f32p, u8p, u8p]
        L.oq_elias_unpack.restype = C.c_int
        L.oq_message_capacity.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int]
        L.oq_message_capacity.restype = C.c_uint64
        L.oq_encode.argtypes = [f32p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, C.c_int,
                                C.c_uint64, C.c_uint32, C.c_uint32, f32p, u8p, C.c_uint64, u64p]
        L.oq_encode.restype = C.c_int
        L.oq_decode.argtypes = [u8p, u64p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, f32p]
        L.oq_decode.restype = C.c_int
        L.oq_decode_accumulate.argtypes = [C.POINTER(u8p), C.POINTER(u64p), C.c_uint32,
                                           C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, f32p]
        L.oq_decode_accumulate.restype = C.c_int
        L.oq_sgd_step.argtypes = [f32p, f32p, C.c_float, C.c_uint32, C.c_uint64]
        L.oq_sgd_step.restype = None
        _lib = L
    return _lib


def _p(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def n_buckets(n, d):
    return (n + d - 1) // d


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    lib().oq_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(o, C.c_uint32))
    return o


def uniform(seed, step, worker, i):
    return float(lib().oq_uniform(seed, step, worker, i))


def level_bits(s):
    return int(lib().oq_level_bits(s))


def bucket_scales(g, d, norm_kind):
    g = _f32(g)
    A = np.zeros(n_buckets(g.size, d), dtype=np.float32)
    lib().oq_bucket_scales(_p(g, C.c_float), g.size, d, norm_kind, _p(A, C.c_float))
    return A


def quantize(g, d, s, A, seed, step, worker, i0=0):
    g = _f32(g)
    A = _f32(A)
    lv = np.zeros(g.size, dtype=np.uint8)
    sg = np.zeros(g.size, dtype=np.uint8)
    lib().oq_quantize(_p(g, C.c_float), g.size, d, s, _p(A, C.c_float), seed, step, worker, i0,
                      _p(lv, C.c_uint8), _p(sg, C.c_uint8))
    return lv, sg


def quantize_with_uniforms(g, d, s, A, u):
    g = _f32(g)
    A = _f32(A)
    u = _f32(u)
    lv = np.zeros(g.size, dtype=np.uint8)
    sg = np.zeros(g.size, dtype=np.uint8)
    lib().oq_quantize_with_uniforms(_p(g, C.c_float), g.size, d, s, _p(A, C.c_float),
                                    _p(u, C.c_float), _p(lv, C.c_uint8), _p(sg, C.c_uint8))
    return lv, sg


def dequantize(A, levels, signs, d, s):
    A = _f32(A)
    out = np.zeros(levels.size, dtype=np.float32)
    lib().oq_dequantize(_p(A, C.c_float), _p(levels, C.c_uint8), _p(signs, C.c_uint8),
                        levels.size, d, s, _p(out, C.c_float))
    return out


def fixed_layout(n, d, s):
    lay = np.zeros(4, dtype=np.uint64)
    lib().oq_fixed_layout(n, d, s, _p(lay, C.c_uint64))
    return [int(v) for v in lay]


def fixed_pack(A, levels, signs, d, s):
    A = _f32(A)
    n = levels.size
    out = np.zeros(fixed_layout(n, d, s)[2], dtype=np.uint8)
    lib().oq_fixed_pack(_p(A, C.c_float), _p(levels, C.c_uint8), _p(signs, C.c_uint8), n, d, s,
                        _p(out, C.c_uint8))
    return out


def fixed_unpack(msg, n, d, s):
    msg = np.ascontiguousarray(msg, dtype=np.uint8)
    A = np.zeros(n_buckets(n, d), dtype=np.float32)
    lv = np.zeros(n, dtype=np.uint8)
    sg = np.zeros(n, dtype=np.uint8)
    lib().oq_fixed_unpack(_p(msg, C.c_uint8), n, d, s, _p(A, C.c_float), _p(lv, C.c_uint8),
                          _p(sg, C.c_uint8))
    return A, lv, sg


def elias_string(k):
    buf = C.create_string_buffer(96)
    ln = lib().oq_elias_string(int(k), buf)
    return buf.value.decode()[:ln]


def elias_parse(bits):
    """Decode one integer from a '0'/'1' string. Returns (value, bits consumed) or None."""
    v = C.c_uint64(0)
    used = lib().oq_elias_parse(bits.encode(), len(bits), C.byref(v))
    return None if used < 0 else (int(v.value), used)


def message_capacity(n, d, s, code_kind):
    return int(lib().oq_message_capacity(n, d, s, code_kind))


def elias_pack(A, levels, signs, d, dense=False, cap_bytes=None, s=255):
    A = _f32(A)
    n = levels.size
    if cap_bytes is None:
        cap_bytes = message_capacity(n, d, s, CODE_ELIAS_DENSE if dense else CODE_ELIAS)
    payload = np.zeros(cap_bytes, dtype=np.uint8)
    off = np.zeros(n_buckets(n, d) + 1, dtype=np.uint64)
    bits = lib().oq_elias_pack(_p(A, C.c_float), _p(levels, C.c_uint8), _p(signs, C.c_uint8), n,
                               d, int(dense), _p(payload, C.c_uint8), cap_bytes,
                               _p(off, C.c_uint64))
    if bits == 2 ** 64 - 1:
        return None, payload, off
    return int(bits), payload, off


def elias_unpack(payload, offsets, n, d, s, dense=False):
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint64)
    A = np.zeros(n_buckets(n, d), dtype=np.float32)
    lv = np.zeros(n, dtype=np.uint8)
    sg = np.zeros(n, dtype=np.uint8)
    st = lib().oq_elias_unpack(_p(payload, C.c_uint8), _p(offsets, C.c_uint64), n, d, s,
                               int(dense), _p(A, C.c_float), _p(lv, C.c_uint8), _p(sg, C.c_uint8))
    return int(st), A, lv, sg


def encode(g, d, s, norm_kind, code_kind, seed, step, worker, A_ext=None, cap_bytes=None):
    """Whole-message Encode. Returns (message bytes trimmed to its length, info[4])."""
    g = _f32(g)
    n = g.size
    if cap_bytes is None:
        cap_bytes = message_capacity(n, d, s, code_kind)
    out = np.zeros(cap_bytes, dtype=np.uint8)
    info = np.zeros(4, dtype=np.uint64)
    a_ptr = None
    if A_ext is not None:
        A_ext = _f32(A_ext)
        a_ptr = _p(A_ext, C.c_float)
    st = lib().oq_encode(_p(g, C.c_float), n, d, s, norm_kind, code_kind, seed, step, worker,
                         a_ptr, _p(out, C.c_uint8), cap_bytes, _p(info, C.c_uint64))
    if st != 0:
        raise RuntimeError("oracle encode: capacity too small")
    info = [int(v) for v in info]
    return out[:info[2]].copy(), info


def message_table(msg, info, n, d):
    """View of the offset table inside an Elias message."""
    B = n_buckets(n, d)
    return np.frombuffer(msg.tobytes()[info[1]:info[1] + 8 * (B + 1)], dtype=np.uint64).copy()


def decode(msg, table, n, d, s, code_kind):
    msg = np.ascontiguousarray(msg, dtype=np.uint8)
    out = np.zeros(n, dtype=np.float32)
    tp = None
    if table is not None:
        table = np.ascontiguousarray(table, dtype=np.uint64)
        tp = _p(table, C.c_uint64)
    st = lib().oq_decode(_p(msg, C.c_uint8), tp, n, d, s, code_kind, _p(out, C.c_float))
    return int(st), out


def decode_accumulate(msgs, tables, n, d, s, code_kind):
    K = len(msgs)
    msgs = [np.ascontiguousarray(m, dtype=np.uint8) for m in msgs]
    mp = (C.POINTER(C.c_uint8) * K)(*[_p(m, C.c_uint8) for m in msgs])
    tp = None
    if tables is not None:
        tables = [np.ascontiguousarray(t, dtype=np.uint64) for t in tables]
        tp = (C.POINTER(C.c_uint64) * K)(*[_p(t, C.c_uint64) for t in tables])
    acc = np.zeros(n, dtype=np.float32)
    st = lib().oq_decode_accumulate(mp, tp, K, n, d, s, code_kind, _p(acc, C.c_float))
    return int(st), acc


def sgd_step(x, acc, eta, K):
    x = _f32(x).copy()
    acc = _f32(acc)
    lib().oq_sgd_step(_p(x, C.c_float), _p(acc, C.c_float), eta, K, x.size)
    return x


# --------------------------------------------------------------------------------------------------
# Per-tensor policy (Section 5, "Protocol": tensors below a size threshold are sent in full
# precision, and buckets are cut so that they fit the tensors). Written on top of the functions
# above, in numpy, tensor by tensor:
#   * the flat gradient is a concatenation of T tensors of the given sizes;
#   * a tensor with fewer than `min_quantized` elements is "raw": its fp32 values travel as they are;
#   * every other tensor is cut into buckets of d starting at its own first element, the last one
#     shorter. Its values are laid out in a "compact" vector in which each tensor is padded with
#     zeros up to a multiple of d, so that the compact vector has uniform buckets and the ordinary
#     Encode applies to it unchanged (zeros do not change a norm and quantize to level 0). The
#     uniform of a coordinate is keyed by its compact index.
# Policy message = raw values (fp32, padded to 16 bytes) followed by the ordinary message of the
# compact vector. Decode: ordinary decode of the compact part; the raw values of the K messages are
# summed in ascending k from +0; both are put back at the tensors' positions.
# --------------------------------------------------------------------------------------------------
def policy_plan(sizes, d, min_quantized=10000):
    """Layout of the compact vector and of the raw region for tensors of the given sizes."""
    sizes = [int(m) for m in sizes]
    plan = {"d": d, "n": sum(sizes), "large": [], "small": [], "n_compact": 0, "n_raw": 0}
    off = 0
    for m in sizes:
        if m >= min_quantized:
            padded = (m + d - 1) // d * d
            plan["large"].append((off, m, plan["n_compact"]))     # flat offset, size, compact offset
            plan["n_compact"] += padded
        elif m > 0:
            plan["small"].append((off, m, plan["n_raw"]))         # flat offset, size, raw offset
            plan["n_raw"] += m
        off += m
    plan["raw_prefix"] = (4 * plan["n_raw"] + 15) // 16 * 16
    return plan


def policy_gather(g, plan):
    g = _f32(g)
    assert g.size == plan["n"]
    compact = np.zeros(plan["n_compact"], dtype=np.float32)
    raw = np.zeros(plan["n_raw"], dtype=np.float32)
    for off, m, c0 in plan["large"]:
        compact[c0:c0 + m] = g[off:off + m]
    for off, m, r0 in plan["small"]:
        raw[r0:r0 + m] = g[off:off + m]
    return compact, raw


def policy_scatter(compact, raw, plan):
    out = np.zeros(plan["n"], dtype=np.float32)
    for off, m, c0 in plan["large"]:
        out[off:off + m] = compact[c0:c0 + m]
    for off, m, r0 in plan["small"]:
        out[off:off + m] = raw[r0:r0 + m]
    return out


def policy_encode(g, plan, s, norm_kind, code_kind, seed, step, worker, A_ext=None):
    """Returns (policy message bytes, info[4]): info[0] = information bits (32 per raw value plus
    the ordinary message's), info[1] = byte offset of the offset table (0 if none), info[2] =
    message bytes, info[3] = bytes of the raw region in front."""
    compact, raw = policy_gather(g, plan)
    prefix = plan["raw_prefix"]
    head = np.zeros(prefix, dtype=np.uint8)
    head[:4 * raw.size] = raw.view(np.uint8)
    if plan["n_compact"] == 0:
        return head, [32 * raw.size, 0, prefix, prefix]
    msg, info = encode(compact, plan["d"], s, norm_kind, code_kind, seed, step, worker, A_ext=A_ext)
    return (np.concatenate([head, msg]),
            [info[0] + 32 * raw.size, info[1] + prefix if info[1] else 0, info[2] + prefix, prefix])


def policy_decode_accumulate(msgs, infos, plan, s, code_kind):
    """Sum of the K decoded policy messages, ascending k from +0, at the tensors' positions."""
    d, prefix, nc, nr = plan["d"], plan["raw_prefix"], plan["n_compact"], plan["n_raw"]
    st, acc_c = 0, np.zeros(0, dtype=np.float32)
    if nc:
        parts = [np.ascontiguousarray(m[prefix:]) for m in msgs]
        tabs = None
        if code_kind != CODE_FIXED:
            tabs = [message_table(p, [i[0], i[1] - prefix, i[2] - prefix, 0], nc, d) for p, i in zip(parts, infos)]
        st, acc_c = decode_accumulate(parts, tabs, nc, d, s, code_kind)
    acc_r = np.zeros(nr, dtype=np.float32)
    for m in msgs:
        acc_r = acc_r + np.ascontiguousarray(m[:4 * nr]).view(np.float32)     # fp32 adds, ascending k
    return st, policy_scatter(acc_c, acc_r, plan)
