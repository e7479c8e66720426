"""ctypes binding of libqsgd.so: the same entry points as include/qsgd.h, argument marshalling
only. PyTorch supplies device memory and the CUDA stream; every step of the path runs in the
library's kernels. There is no CPU fallback: a missing library or a missing device raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libqsgd.so")

NORM_L2, NORM_MAX = 0, 1
CODE_FIXED, CODE_ELIAS, CODE_ELIAS_DENSE = 0, 1, 2

DEV_CAPACITY, DEV_OVERRUN, DEV_POSITION, DEV_LEVEL, DEV_TABLE, DEV_TIMEOUT = 1, 2, 4, 8, 16, 32

EXPORTS = ["qsgd_message_capacity", "qsgd_workspace_bytes", "qsgd_fixed_layout", "qsgd_encode",
           "qsgd_decode_accumulate", "qsgd_sgd_step", "qsgd_decode_sgd_step",
           "qsgd_decode_accumulate_packed", "qsgd_decode_sgd_step_packed",
           "qsgd_status_string", "qsgd_launch_count", "qsgd_profile_enable",
           "qsgd_profile_kernel_count", "qsgd_profile_kernel_name", "qsgd_profile_collect",
           "qsgd_static_scratch_bytes", "qsgd_encode_elias_static",
           "qsgd_policy_plan_sizes", "qsgd_policy_plan", "qsgd_policy_message_capacity",
           "qsgd_policy_workspace_bytes", "qsgd_policy_encode", "qsgd_policy_decode_accumulate",
           "qsgd_policy_decode_sgd_step", "qsgd_test_set_wait_polls", "qsgd_test_default_wait_polls",
           "qsgd_set_launch_chaining"]

_lib = None


class QsgdError(RuntimeError):
    pass


class PolicyStruct(C.Structure):
    """qsgd_policy of include/qsgd.h."""
    _fields_ = [("bucket_src", C.c_void_p), ("bucket_len", C.c_void_p), ("n_buckets", C.c_uint64),
                ("raw_src", C.c_void_p), ("raw_start", C.c_void_p), ("n_raw_segments", C.c_uint64),
                ("n_raw", C.c_uint64), ("n", C.c_uint64), ("quads", C.c_uint32)]


def lib():
    """Loads libqsgd.so (must have been built: `python -m paper_1610_02132_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise QsgdError("libqsgd.so is not built; run paper_1610_02132_b200.build.build()")
        L = C.CDLL(_LIB_PATH)
        vp, u64, u32, sz = C.c_void_p, C.c_uint64, C.c_uint32, C.c_size_t
        L.qsgd_message_capacity.argtypes = [u64, u32, u32, C.c_int]
        L.qsgd_message_capacity.restype = sz
        L.qsgd_workspace_bytes.argtypes = [u64, u32, u32, C.c_int]
        L.qsgd_workspace_bytes.restype = sz
        L.qsgd_fixed_layout.argtypes = [u64, u32, u32, C.POINTER(u64)]
        L.qsgd_fixed_layout.restype = C.c_int
        L.qsgd_encode.argtypes = [vp, u64, u32, u32, C.c_int, C.c_int, u64, u32, u32, vp, sz, vp,
                                  vp, vp, vp]
        L.qsgd_encode.restype = C.c_int
        L.qsgd_decode_accumulate.argtypes = [C.POINTER(vp), C.POINTER(vp), C.POINTER(u64), u32, u64, u32, u32,
                                             C.c_int, vp, vp, vp]
        L.qsgd_decode_accumulate.restype = C.c_int
        L.qsgd_decode_accumulate_packed.argtypes = L.qsgd_decode_accumulate.argtypes
        L.qsgd_decode_accumulate_packed.restype = C.c_int
        L.qsgd_sgd_step.argtypes = [vp, vp, C.c_float, u32, u64, vp]
        L.qsgd_sgd_step.restype = C.c_int
        L.qsgd_decode_sgd_step.argtypes = [C.POINTER(vp), C.POINTER(vp), C.POINTER(u64), u32, u64, u32, u32,
                                           C.c_int, vp, C.c_float, vp, vp]
        L.qsgd_decode_sgd_step.restype = C.c_int
        L.qsgd_decode_sgd_step_packed.argtypes = L.qsgd_decode_sgd_step.argtypes
        L.qsgd_decode_sgd_step_packed.restype = C.c_int
        L.qsgd_status_string.argtypes = [C.c_int]
        L.qsgd_status_string.restype = C.c_char_p
        L.qsgd_static_scratch_bytes.argtypes = []
        L.qsgd_static_scratch_bytes.restype = sz
        L.qsgd_encode_elias_static.argtypes = [vp, u64, u32, u32, C.c_int, C.c_int, u64, u32, u32, vp,
                                               sz, vp, vp, vp]
        L.qsgd_encode_elias_static.restype = C.c_int
        L.qsgd_launch_count.argtypes = []
        L.qsgd_launch_count.restype = u64
        pu64, pu32, pp = C.POINTER(u64), C.POINTER(u32), C.POINTER(PolicyStruct)
        L.qsgd_policy_plan_sizes.argtypes = [pu64, u32, u32, u64, pu64, pu64, pu64]
        L.qsgd_policy_plan_sizes.restype = C.c_int
        L.qsgd_policy_plan.argtypes = [pu64, u32, u32, u64, pu64, pu32, pu64, pu64, pu32]
        L.qsgd_policy_plan.restype = C.c_int
        L.qsgd_policy_message_capacity.argtypes = [pp, u32, u32, C.c_int]
        L.qsgd_policy_message_capacity.restype = sz
        L.qsgd_policy_workspace_bytes.argtypes = [pp, u32, u32, C.c_int]
        L.qsgd_policy_workspace_bytes.restype = sz
        L.qsgd_policy_encode.argtypes = [vp, pp, u32, u32, C.c_int, C.c_int, u64, u32, u32, vp, sz, vp,
                                         vp, vp, vp]
        L.qsgd_policy_encode.restype = C.c_int
        L.qsgd_policy_decode_accumulate.argtypes = [C.POINTER(vp), C.POINTER(vp), pu64, u32, pp, u32, u32,
                                                    C.c_int, vp, vp, vp]
        L.qsgd_policy_decode_accumulate.restype = C.c_int
        L.qsgd_policy_decode_sgd_step.argtypes = [C.POINTER(vp), C.POINTER(vp), pu64, u32, pp, u32, u32,
                                                  C.c_int, vp, C.c_float, vp, vp]
        L.qsgd_policy_decode_sgd_step.restype = C.c_int
        L.qsgd_set_launch_chaining.argtypes = [C.c_int]
        L.qsgd_set_launch_chaining.restype = C.c_int
        L.qsgd_test_set_wait_polls.argtypes = [u32]
        L.qsgd_test_set_wait_polls.restype = None
        L.qsgd_test_default_wait_polls.argtypes = []
        L.qsgd_test_default_wait_polls.restype = u32
        L.qsgd_profile_enable.argtypes = [C.c_int]
        L.qsgd_profile_enable.restype = None
        L.qsgd_profile_kernel_count.argtypes = []
        L.qsgd_profile_kernel_count.restype = C.c_int
        L.qsgd_profile_kernel_name.argtypes = [C.c_int]
        L.qsgd_profile_kernel_name.restype = C.c_char_p
        L.qsgd_profile_collect.argtypes = [C.POINTER(C.c_double), C.POINTER(u64)]
        L.qsgd_profile_collect.restype = C.c_int
        _lib = L
    return _lib


def _check(st):
    if st != 0:
        raise QsgdError("qsgd status %d: %s" % (st, lib().qsgd_status_string(st).decode()))


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _require_cuda(t, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise QsgdError("%s must be a contiguous CUDA tensor" % name)


def qsgd_message_capacity(n, bucket, s, code_kind):
    return int(lib().qsgd_message_capacity(n, bucket, s, code_kind))


def qsgd_workspace_bytes(n, bucket, s, code_kind):
    return int(lib().qsgd_workspace_bytes(n, bucket, s, code_kind))


def qsgd_fixed_layout(n, bucket, s):
    lay = (C.c_uint64 * 4)()
    _check(lib().qsgd_fixed_layout(n, bucket, s, lay))
    return [int(v) for v in lay]


def qsgd_launch_count():
    return int(lib().qsgd_launch_count())


def qsgd_set_launch_chaining(on):
    """Turns programmatic dependent launch of the library's kernels on or off; returns the previous setting."""
    return bool(lib().qsgd_set_launch_chaining(1 if on else 0))


def qsgd_test_set_wait_polls(polls):
    """Test hook: bound of the streaming encoder's main-loop waits (0 = give up at once)."""
    lib().qsgd_test_set_wait_polls(int(polls))


def qsgd_test_default_wait_polls():
    return int(lib().qsgd_test_default_wait_polls())


def qsgd_profile_enable(on):
    lib().qsgd_profile_enable(1 if on else 0)


def qsgd_profile_collect():
    """Returns {kernel name: (total ms, launches)} for the launches recorded since the last call."""
    L = lib()
    k = L.qsgd_profile_kernel_count()
    ms = (C.c_double * k)()
    cnt = (C.c_uint64 * k)()
    st = L.qsgd_profile_collect(ms, cnt)
    if st != 0:
        raise QsgdError("qsgd_profile_collect: cuda error %d" % st)
    return {L.qsgd_profile_kernel_name(i).decode(): (float(ms[i]), int(cnt[i]))
            for i in range(k) if cnt[i]}


def qsgd_encode(g, bucket, s, norm_kind, code_kind, seed, step, worker, out, out_bits,
                workspace=None, status_dev=None, stream=None, n=None):
    """Encode g (fp32 CUDA tensor) into `out` (uint8 CUDA tensor); see include/qsgd.h."""
    _require_cuda(g, "g")
    _require_cuda(out, "out")
    _require_cuda(out_bits, "out_bits")
    _require_cuda(status_dev, "status_dev")
    n = g.numel() if n is None else n
    ws = None if workspace is None else C.c_void_p(workspace.data_ptr())
    _check(lib().qsgd_encode(g.data_ptr(), n, bucket, s, norm_kind, code_kind, seed, step, worker,
                             out.data_ptr(), out.numel() * out.element_size(),
                             out_bits.data_ptr(), ws, status_dev.data_ptr(), _stream(stream)))


def qsgd_static_scratch_bytes():
    return int(lib().qsgd_static_scratch_bytes())


def qsgd_encode_elias_static(g, bucket, s, norm_kind, code_kind, seed, step, worker, out, out_bits,
                             status_dev, stream=None):
    """Elias Encode without a workspace argument: the scratch is a 32 MiB array built into the
    library, so this call allocates nothing (for callers that may not allocate device memory when
    they encode). Same results as qsgd_encode; sizes beyond the built-in scratch raise. Calls
    that overlap on the GPU share the scratch and must be serialised by the caller."""
    _require_cuda(g, "g")
    _require_cuda(out, "out")
    _require_cuda(out_bits, "out_bits")
    _require_cuda(status_dev, "status_dev")
    _check(lib().qsgd_encode_elias_static(g.data_ptr(), g.numel(), bucket, s, norm_kind, code_kind,
                                          seed, step, worker, out.data_ptr(),
                                          out.numel() * out.element_size(), out_bits.data_ptr(),
                                          status_dev.data_ptr(), _stream(stream)))


def _ptr_array(tensors):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t if isinstance(t, int) else t.data_ptr()
    return arr


def _u64_array(values):
    if values is None:
        return None
    return (C.c_uint64 * len(values))(*[int(v) for v in values])


def qsgd_decode_accumulate(msgs, tables, n, bucket, s, code_kind, acc, status_dev, stream=None,
                           payload_bytes=None):
    """acc <- ascending-k sum of the decoded messages; msgs / tables: lists of CUDA tensors
    (or raw device addresses); payload_bytes: optional list of payload lengths (read bound)."""
    _require_cuda(acc, "acc")
    mp = _ptr_array(msgs)
    tp = None if tables is None else _ptr_array(tables)
    _check(lib().qsgd_decode_accumulate(mp, tp, _u64_array(payload_bytes), len(msgs), n, bucket, s, code_kind,
                                        acc.data_ptr(), status_dev.data_ptr(), _stream(stream)))


def _msg_bytes(msgs, msg_bytes):
    if msg_bytes is not None:
        return _u64_array(msg_bytes)
    return _u64_array([m.numel() * m.element_size() for m in msgs])


def qsgd_decode_accumulate_packed(msgs, infos, n, bucket, s, code_kind, acc, status_dev, stream=None,
                                  msg_bytes=None):
    """As qsgd_decode_accumulate, for messages as Encode left them: infos[k] is the CUDA tensor (or
    device address) of message k's four info words; the tables are found on the device. msg_bytes
    defaults to the sizes of the message tensors."""
    _require_cuda(acc, "acc")
    ip = None if infos is None else _ptr_array(infos)
    _check(lib().qsgd_decode_accumulate_packed(_ptr_array(msgs), ip, _msg_bytes(msgs, msg_bytes), len(msgs), n,
                                               bucket, s, code_kind, acc.data_ptr(), status_dev.data_ptr(),
                                               _stream(stream)))


def qsgd_decode_sgd_step_packed(msgs, infos, n, bucket, s, code_kind, x, eta, status_dev, stream=None,
                                msg_bytes=None):
    _require_cuda(x, "x")
    ip = None if infos is None else _ptr_array(infos)
    _check(lib().qsgd_decode_sgd_step_packed(_ptr_array(msgs), ip, _msg_bytes(msgs, msg_bytes), len(msgs), n,
                                             bucket, s, code_kind, x.data_ptr(), eta, status_dev.data_ptr(),
                                             _stream(stream)))


def qsgd_sgd_step(x, acc, eta, K, stream=None):
    _require_cuda(x, "x")
    _require_cuda(acc, "acc")
    _check(lib().qsgd_sgd_step(x.data_ptr(), acc.data_ptr(), eta, K, x.numel(), _stream(stream)))


def qsgd_decode_sgd_step(msgs, tables, n, bucket, s, code_kind, x, eta, status_dev, stream=None,
                         payload_bytes=None):
    _require_cuda(x, "x")
    mp = _ptr_array(msgs)
    tp = None if tables is None else _ptr_array(tables)
    _check(lib().qsgd_decode_sgd_step(mp, tp, _u64_array(payload_bytes), len(msgs), n, bucket, s, code_kind,
                                      x.data_ptr(), eta, status_dev.data_ptr(), _stream(stream)))


# ------------------------------- per-tensor policy -------------------------------------------
class Policy:
    """A plan made by qsgd_policy_plan for tensors of the given sizes, with its arrays copied to
    the device (the copies are the only thing this class adds to the C calls)."""

    def __init__(self, tensor_sizes, bucket, min_quantized=10000, device="cuda"):
        T = len(tensor_sizes)
        sizes = (C.c_uint64 * max(T, 1))(*[int(m) for m in tensor_sizes])
        nb, ns, nr = C.c_uint64(), C.c_uint64(), C.c_uint64()
        _check(lib().qsgd_policy_plan_sizes(sizes, T, bucket, min_quantized, C.byref(nb), C.byref(ns), C.byref(nr)))
        nb, ns, nr = nb.value, ns.value, nr.value
        src = torch.zeros(max(nb, 1), dtype=torch.int64)
        ln = torch.zeros(max(nb, 1), dtype=torch.int32)
        rsrc = torch.zeros(max(ns, 1), dtype=torch.int64)
        rstart = torch.zeros(ns + 1, dtype=torch.int64)
        quads = C.c_uint32()
        as_p = lambda t, ct: C.cast(t.data_ptr(), C.POINTER(ct))
        _check(lib().qsgd_policy_plan(sizes, T, bucket, min_quantized, as_p(src, C.c_uint64), as_p(ln, C.c_uint32),
                                      as_p(rsrc, C.c_uint64), as_p(rstart, C.c_uint64), C.byref(quads)))
        self.bucket = bucket
        self.host = {"bucket_src": src[:nb], "bucket_len": ln[:nb], "raw_src": rsrc[:ns], "raw_start": rstart}
        self.dev = {k: v.to(device) for k, v in (("bucket_src", src), ("bucket_len", ln), ("raw_src", rsrc),
                                                ("raw_start", rstart))}
        self.n = int(sum(int(m) for m in tensor_sizes))
        self.n_buckets, self.n_raw_segments, self.n_raw, self.quads = nb, ns, nr, quads.value
        self.raw_prefix = (4 * nr + 15) // 16 * 16
        self.struct = PolicyStruct(self.dev["bucket_src"].data_ptr(), self.dev["bucket_len"].data_ptr(), nb,
                                   self.dev["raw_src"].data_ptr(), self.dev["raw_start"].data_ptr(), ns, nr,
                                   self.n, quads.value)


def qsgd_policy_message_capacity(plan, s, code_kind):
    return int(lib().qsgd_policy_message_capacity(C.byref(plan.struct), plan.bucket, s, code_kind))


def qsgd_policy_workspace_bytes(plan, s, code_kind):
    return int(lib().qsgd_policy_workspace_bytes(C.byref(plan.struct), plan.bucket, s, code_kind))


def qsgd_policy_encode(g, plan, s, norm_kind, code_kind, seed, step, worker, out, out_bits, workspace=None,
                       status_dev=None, stream=None):
    _require_cuda(g, "g")
    _require_cuda(out, "out")
    _require_cuda(out_bits, "out_bits")
    _require_cuda(status_dev, "status_dev")
    if g.numel() != plan.n:
        raise QsgdError("g has %d elements, the plan covers %d" % (g.numel(), plan.n))
    ws = None if workspace is None else C.c_void_p(workspace.data_ptr())
    _check(lib().qsgd_policy_encode(g.data_ptr(), C.byref(plan.struct), plan.bucket, s, norm_kind, code_kind, seed,
                                    step, worker, out.data_ptr(), out.numel() * out.element_size(),
                                    out_bits.data_ptr(), ws, status_dev.data_ptr(), _stream(stream)))


def qsgd_policy_decode_accumulate(msgs, tables, plan, s, code_kind, acc, status_dev, stream=None,
                                  payload_bytes=None):
    _require_cuda(acc, "acc")
    if acc.numel() != plan.n:
        raise QsgdError("acc has %d elements, the plan covers %d" % (acc.numel(), plan.n))
    mp = _ptr_array(msgs)
    tp = None if tables is None else _ptr_array(tables)
    _check(lib().qsgd_policy_decode_accumulate(mp, tp, _u64_array(payload_bytes), len(msgs), C.byref(plan.struct), plan.bucket, s, code_kind,
                                               acc.data_ptr(), status_dev.data_ptr(), _stream(stream)))


def qsgd_policy_decode_sgd_step(msgs, tables, plan, s, code_kind, x, eta, status_dev, stream=None,
                                payload_bytes=None):
    _require_cuda(x, "x")
    if x.numel() != plan.n:
        raise QsgdError("x has %d elements, the plan covers %d" % (x.numel(), plan.n))
    mp = _ptr_array(msgs)
    tp = None if tables is None else _ptr_array(tables)
    _check(lib().qsgd_policy_decode_sgd_step(mp, tp, _u64_array(payload_bytes), len(msgs), C.byref(plan.struct), plan.bucket, s, code_kind,
                                             x.data_ptr(), eta, status_dev.data_ptr(), _stream(stream)))


# ------------------------------- conveniences (allocation only) -----------------------------
def new_status(device="cuda"):
    return torch.zeros(1, dtype=torch.int32, device=device)


def encode_alloc(g, bucket, s, norm_kind, code_kind, seed, step, worker, capacity=None,
                 stream=None):
    """Allocates the message, info words, workspace and status, then calls qsgd_encode.
    Returns (out, out_bits, status_dev); synchronise before reading them on the host."""
    n = g.numel()
    cap = qsgd_message_capacity(n, bucket, s, code_kind) if capacity is None else capacity
    out = torch.empty(cap, dtype=torch.uint8, device=g.device)
    out_bits = torch.zeros(4, dtype=torch.int64, device=g.device)
    wsb = qsgd_workspace_bytes(n, bucket, s, code_kind)
    ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device=g.device)
    status = new_status(g.device)
    qsgd_encode(g, bucket, s, norm_kind, code_kind, seed, step, worker, out, out_bits, ws, status,
                stream)
    return out, out_bits, status
