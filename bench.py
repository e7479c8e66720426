#!/usr/bin/env python
"""Benchmark of the QSGD hot path on B200: Encode -> (K messages in HBM) -> Decode + aggregate +
SGD step, through the C ABI (include/qsgd.h).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole hot path over one batch of synthetic gradients: for every code
kind of the workload, K worker encodes followed by one fused decode + aggregate + SGD step. The K
encodes are independent of one another and are issued round-robin on --streams streams (default 2);
`ms_per_step_one_stream` is the same step with everything on one stream, and the per-kernel figures
come from a third pass with CUDA events around every launch.
Prints ONE JSON line (rank 0). Timing is on the device with CUDA events; inputs are resident in
HBM before the timed region for `value`, and copied from pinned host memory inside it for `e2e`.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

NORM = {"l2": 0, "max": 1}
CODE = {"fixed": 0, "elias": 1, "elias_dense": 2}

WORKLOADS = {
    # the five workloads the metric is defined on: name -> (n, d, s, norm, codes, K, generator)
    "tiny": dict(n=2 ** 20, d=512, s=15, norm="l2", codes=["fixed"], K=4, gen="gauss0.01",
                 desc="tiny ref: N(0,0.01^2), n=2^20"),
    "sparse_elias": dict(n=2 ** 24, d=4096, s=1, norm="l2", codes=["elias"], K=8, gen="sparse_laplace",
                         desc="sparse Elias regime: Laplace(0,1e-3) with 30% exact zeros, n=2^24"),
    "alexnet": dict(n=61100840, d=512, s=255, norm="max", codes=["fixed"], K=16, gen="alexnet",
                    desc="AlexNet-shaped flat gradient, layer sigma 1e-2/sqrt(fan_in)"),
    "resnet152": dict(n=60192808, d=512, s=15, norm="l2", codes=["fixed", "elias"], K=16, gen="mixture",
                      desc="ResNet-152-shaped flat gradient, 0.9 N(0,1e-4^2) + 0.1 N(0,1e-2^2)"),
    # Per-tensor policy (tensors under 10K elements raw, buckets cut to the tensors) on the two model shapes
    "alexnet_policy": dict(n=61100840, d=512, s=255, norm="max", codes=["fixed"], K=16, gen="alexnet",
                           policy="alexnet",
                           desc="AlexNet-shaped gradient under the per-tensor policy (8 bias tensors raw)"),
    "resnet152_policy": dict(n=60192808, d=512, s=15, norm="l2", codes=["fixed", "elias"], K=16, gen="mixture",
                             policy="resnet152",
                             desc="ResNet-152-shaped gradient under the per-tensor policy (313 small tensors raw)"),
    # Corollary 3.3's regime: the dense code Code'_s at s = sqrt(d)
    "dense_elias": dict(n=2 ** 24, d=4096, s=64, norm="l2", codes=["elias_dense"], K=8, gen="gauss1",
                        desc="dense Elias regime: N(0,1), n=2^24, s = sqrt(d), every coordinate coded"),
    "sweep_point": dict(n=2 ** 28, d=512, s=15, norm="l2", codes=["fixed"], K=16, gen="gauss1",
                        desc="bandwidth sweep point: N(0,1), n=2^28"),
}
DEFAULT_WORKLOAD = "resnet152"
ETA = 0.1
PHILOX_SEED = 7


# The one JSON line goes to the process's real standard output; whatever libraries print on file
# descriptor 1 meanwhile (NCCL announces its version there) is sent to standard error.
_REAL_STDOUT = None


def claim_stdout():
    global _REAL_STDOUT
    if _REAL_STDOUT is None:
        sys.stdout.flush()
        _REAL_STDOUT = os.fdopen(os.dup(1), "w")
        os.dup2(2, 1)


def emit(text):
    out = _REAL_STDOUT if _REAL_STDOUT is not None else sys.stdout
    out.write(text + "\n")
    out.flush()


def elen(k):
    return 1 if k == 1 else k.bit_length() + elen(k.bit_length() - 1)


def policy_sizes(name):
    from paper_1610_02132_b200 import inputs as I
    shapes = I.alexnet_shapes() if name == "alexnet" else I.resnet152_shapes()
    return [int(np.prod(sh)) for sh in shapes]


def fixed_bytes(n, d, s):
    lb = 1 if s <= 1 else 2 if s <= 3 else 4 if s <= 15 else 8
    a16 = lambda x: (x + 15) // 16 * 16  # noqa: E731
    B = (n + d - 1) // d
    return a16(4 * B) + a16(4 * ((n + 31) // 32)) + a16(4 * ((n * lb + 31) // 32))


# ------------------------------------------------------------------------------------------------
# inputs
# ------------------------------------------------------------------------------------------------
def host_gradient(wl, worker, n=None):
    from paper_1610_02132_b200 import inputs as I
    n = wl["n"] if n is None else n
    seed = 1 + worker
    gen = wl["gen"]
    if gen == "gauss0.01":
        return I.gaussian(n, 0.01, seed)
    if gen == "gauss1":
        return I.gaussian(n, 1.0, seed)
    if gen == "sparse_laplace":
        return I.sparse_laplace(n, 1e-3, 0.3, seed)
    if gen == "alexnet":
        return I.layered_gaussian(I.alexnet_shapes(), seed)[:n]
    return I.gaussian_mixture(n, seed)


def device_gradient(wl, worker, device):
    from paper_1610_02132_b200 import inputs as I
    n, seed, gen = wl["n"], 1 + worker, wl["gen"]
    if gen == "gauss0.01":
        return I.gaussian_device(n, 0.01, seed, device)
    if gen == "gauss1":
        return I.gaussian_device(n, 1.0, seed, device)
    if gen == "sparse_laplace":
        return I.sparse_laplace_device(n, 1e-3, 0.3, seed, device)
    if gen == "alexnet":
        return I.layered_gaussian_device(I.alexnet_shapes(), seed, device=device)
    return I.gaussian_mixture_device(n, seed, device=device)


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile(prefix="clocks", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); mx.append(float(p[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), p[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            busy = [c for c in sm if c > 0.5 * max(sm)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
class HotPath:
    """Buffers and one step of the hot path for a workload on one GPU."""

    def __init__(self, wl, device, rank=0, streams=1):
        import torch
        import paper_1610_02132_b200 as Q
        self.torch, self.Q, self.wl, self.dev = torch, Q, wl, device
        # The K workers' encodes are independent of one another; issued round-robin on `streams`
        # streams (a workspace each) the tail of one encode runs beside the head of the next. The
        # decode waits for all of them on the caller's stream.
        self.n_streams = max(1, streams)
        self.side = [torch.cuda.Stream(device=device) for _ in range(self.n_streams)] if self.n_streams > 1 else []
        self.use_streams = self.n_streams > 1
        n, d, s, K = wl["n"], wl["d"], wl["s"], wl["K"]
        self.n, self.d, self.s, self.K = n, d, s, K
        self.B = (n + d - 1) // d
        # per-tensor policy: nq coordinates are quantized (whole buckets), the rest travel raw in
        # `prefix` bytes in front of each message
        self.plan, self.nq, self.n_raw, self.prefix = None, n, 0, 0
        if wl.get("policy"):
            sizes = policy_sizes(wl["policy"])
            assert sum(sizes) == n, "policy workloads run at the model's own size"
            self.plan = Q.Policy(sizes, d, device=device)
            self.B, self.n_raw, self.prefix = self.plan.n_buckets, self.plan.n_raw, self.plan.raw_prefix
            self.nq = self.B * d
        self.norm = NORM[wl["norm"]]
        self.codes = [CODE[c] for c in wl["codes"]]
        # the K workers' gradients (rank shifts the seeds so replicas differ)
        self.g = [device_gradient(wl, rank * K + w, device) for w in range(K)]
        self.x = torch.zeros(n, dtype=torch.float32, device=device)
        self.status = Q.new_status(device)
        self.msgs, self.bits, self.ws, self.tables = {}, {}, {}, {}
        for code in self.codes:
            cap = self.message_capacity(code)
            self.msgs[code] = [torch.empty(cap, dtype=torch.uint8, device=device) for _ in range(K)]
            self.bits[code] = torch.zeros(K, 4, dtype=torch.int64, device=device)
            wsb = max(Q.qsgd_workspace_bytes(self.nq, d, s, code), 16)
            self.ws[code] = [torch.empty(wsb, dtype=torch.uint8, device=device) for _ in range(self.n_streams)]
        self.info = {}

    def message_capacity(self, code):
        """Fixed-width: exact. Elias: the fixed-width size is used as capacity (an Elias message
        longer than that is not worth sending); a first encode verifies it fits."""
        Q = self.Q
        if code == 0:
            return self.prefix + Q.qsgd_message_capacity(self.nq, self.d, self.s, code)
        worst = Q.qsgd_message_capacity(self.nq, self.d, self.s, code)
        return self.prefix + min(worst, 2 * fixed_bytes(self.nq, self.d, self.s) + 8 * (self.B + 1))

    def encode_one(self, code, step, w, g, ws, stream=None):
        Q = self.Q
        if self.plan is not None:
            Q.qsgd_policy_encode(g, self.plan, self.s, self.norm, code, PHILOX_SEED, step, w,
                                 self.msgs[code][w], self.bits[code][w], ws, self.status, stream=stream)
        else:
            Q.qsgd_encode(g, self.d, self.s, self.norm, code, PHILOX_SEED, step, w,
                          self.msgs[code][w], self.bits[code][w], ws, self.status, stream=stream)

    def encode_all(self, code, step, src=None):
        torch = self.torch
        g = self.g if src is None else src
        if not self.use_streams:
            for w in range(self.K):
                self.encode_one(code, step, w, g[w], self.ws[code][0])
            return
        main = torch.cuda.current_stream(self.dev)
        fork = torch.cuda.Event()
        fork.record(main)
        for st in self.side:
            st.wait_event(fork)                    # whatever wrote g, x or the messages before is done
        for w in range(self.K):
            i = w % self.n_streams
            self.encode_one(code, step, w, g[w], self.ws[code][i], stream=self.side[i])
        for st in self.side:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def read_info(self, code):
        """Message sizes of the last encode (a host read-back; outside the timed step except under
        the per-tensor policy, whose decode takes host-resolved table pointers)."""
        if code != 0:
            self.info[code] = self.bits[code].cpu().numpy().view(np.uint64)        # synchronises the stream

    def resolve_tables(self, code):
        """Elias under the per-tensor policy: the offset table sits at byte out_bits[1] of each message."""
        if code == 0:
            return None
        self.read_info(code)
        info = self.info[code]
        nb = 8 * (self.B + 1)
        return [self.msgs[code][w][int(info[w, 1]): int(info[w, 1]) + nb].view(self.torch.int64)
                for w in range(self.K)]

    def decode(self, code):
        """Fused decode + aggregate + SGD step of the K messages of `code`. Ordinary workloads use
        the packed form: the kernels find each offset table from the message's info words on the
        device, so nothing is read back between Encode and Decode."""
        if self.plan is not None:
            self.Q.qsgd_policy_decode_sgd_step(self.msgs[code], self.resolve_tables(code), self.plan, self.s, code,
                                               self.x, ETA, self.status)
        else:
            infos = None if code == 0 else [self.bits[code][w] for w in range(self.K)]
            self.Q.qsgd_decode_sgd_step_packed(self.msgs[code], infos, self.n, self.d, self.s, code, self.x, ETA,
                                               self.status)

    def step(self, step_idx, src=None):
        for code in self.codes:
            self.encode_all(code, step_idx, src)
            self.decode(code)

    def message_bytes(self, code):
        if code == 0:
            return float(self.prefix + fixed_bytes(self.nq, self.d, self.s))
        info = self.info[code]
        return float(np.mean(info[:, 2].astype(np.float64)))

    def payload_bits_per_coord(self, code):
        if code == 0:
            return 8.0 * (self.prefix + fixed_bytes(self.nq, self.d, self.s)) / self.n
        return float(np.mean(self.info[code][:, 0].astype(np.float64))) / self.n


def kernel_algorithmic_bytes(hp, code_name):
    """Bytes each kernel must move per launch (the method's own inputs and outputs)."""
    d, s, K, B = hp.d, hp.s, hp.K, hp.B
    n = hp.n - hp.n_raw                       # coordinates that are quantized (all of them without a policy)
    MF = fixed_bytes(hp.nq, d, s)
    out = {"quantize_fixed": 4 * n + MF, "decode_fixed": K * MF + 8 * n, "sgd_step": 12 * n,
           "raw_gather": 8 * hp.n_raw, "raw_decode": (4 * K + 8) * hp.n_raw}
    for elias_code in (1, 2):                  # sparse code, else the dense code (a workload has one of them)
        if elias_code not in hp.info:
            continue
        info = hp.info[elias_code]
        msg = float(np.mean(info[:, 2].astype(np.float64))) - hp.prefix
        pay = float(np.mean(info[:, 1].astype(np.float64))) - hp.prefix
        out.update({"decode_elias": K * msg + 8 * n, "decode_elias_sparse": K * msg + 8 * n,
                    "elias_scatter": MF + pay + 8 * (B + 1),
                    "elias_length": MF - 4 * ((n + 31) // 32) + 4 * B})
        break
    return out


def load_traffic():
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        return json.load(open(p))
    except Exception:
        return {}


def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_1610_02132_b200 as Q
    if getattr(args, 'no_chaining', False):
        Q.qsgd_set_launch_chaining(False)

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    wl = dict(WORKLOADS[args.workload])
    for k in ("n", "d", "s", "K"):
        if getattr(args, k) is not None:
            wl[k] = getattr(args, k)
    if args.norm:
        wl["norm"] = args.norm
    if args.codes:
        wl["codes"] = args.codes.split(",")

    hp = HotPath(wl, device, rank, streams=args.streams)
    n, K = hp.n, hp.K

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ---------------------------------------------------------------
    for i in range(args.warmup):
        hp.step(i)
    barrier()
    assert int(hp.status.item()) == 0, "device status %d after warm-up" % int(hp.status.item())
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    # The K timed steps run three times. First as a caller with K independent workers' gradients on
    # one GPU runs them: the encodes issued round-robin on --streams streams (default 2, a workspace
    # each), the decode after all of them, nothing between the kernels; this pass gives `value`.
    # Then on one stream (`one_stream`: every kernel strictly after the one before). Then on one
    # stream with a pair of CUDA events around every kernel launch on the launching stream, which
    # gives the per-kernel durations of the roofline and the kernel table (and, the events
    # serialising the launches, a step a few per cent longer: ms_per_step_with_events).
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_steps(first):
        barrier()
        ev0.record()
        for i in range(args.steps):
            hp.step(first + i)
        ev1.record()
        barrier()
        return ev0.elapsed_time(ev1)

    launches0 = Q.qsgd_launch_count()
    ms = timed_steps(args.warmup)
    launches = Q.qsgd_launch_count() - launches0
    ms_one_stream = ms / args.steps
    if hp.use_streams:
        hp.use_streams = False
        hp.step(args.warmup)
        ms_one_stream = timed_steps(args.warmup + args.steps) / args.steps
    Q.qsgd_profile_enable(True)
    Q.qsgd_profile_collect()
    ms_events = timed_steps(args.warmup + 2 * args.steps) / args.steps
    Q.qsgd_profile_enable(False)
    kern = Q.qsgd_profile_collect()
    hp.use_streams = hp.n_streams > 1
    clocks = sampler.stop() if rank == 0 else None
    assert int(hp.status.item()) == 0
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t.item()) / args.steps

    # fp32 gradient bytes that went through Encode plus through Decode, per step, all ranks
    grad_bytes = world * len(hp.codes) * 2 * K * 4 * n
    value = grad_bytes / (ms_step * 1e-3) / 1e9

    # ---- per-phase figures (one extra pass, per-call events) ----------------------------------
    phases = {}
    for code_name, code in zip(wl["codes"], hp.codes):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        torch.cuda.synchronize()
        e[0].record()
        hp.encode_all(code, 1000)
        e[1].record()
        hp.read_info(code)
        torch.cuda.synchronize()
        e[1].record()
        hp.decode(code)
        e[2].record()
        torch.cuda.synchronize()
        t_dec = e[1].elapsed_time(e[2]) * 1e-3
        torch.cuda.synchronize(); e[0].record(); hp.encode_all(code, 1001); e[1].record()
        torch.cuda.synchronize()
        t_enc = e[0].elapsed_time(e[1]) * 1e-3 / K
        M = hp.message_bytes(code)
        phases[code_name] = {
            "encode_GBps_fp32": 4 * n / t_enc / 1e9,
            "decode_sgd_GBps_fp32": K * 4 * n / t_dec / 1e9,
            "encode_us": t_enc * 1e6, "decode_sgd_us": t_dec * 1e6,
            "encode_alg_GBps": (4 * n + M) / t_enc / 1e9,
            "decode_alg_GBps": (K * M + 8 * n) / t_dec / 1e9,
            "message_bytes": M, "bits_per_coord_payload": hp.payload_bits_per_coord(code),
            "bits_per_coord_message": 8 * M / n,
        }

    # ---- roofline of the dominant kernel ------------------------------------------------------
    hbm_peak, peak_src = (peaks.get("hbm_gbs"), "measured") if peaks.get("hbm_gbs") else (6650.0, "fallback")
    alg = kernel_algorithmic_bytes(hp, None)
    kern_tab = {k: {"ms_total": v[0], "launches": v[1], "avg_us": 1e3 * v[0] / v[1]} for k, v in kern.items()}
    tot = sum(v[0] for v in kern.values()) or 1.0
    # In the packed form both Elias decoders are launched and one of them returns after reading the
    # payload lengths: that one moved no message bytes and gets no bandwidth figure.
    stood_down = None
    if "decode_elias" in kern_tab and "decode_elias_sparse" in kern_tab:
        stood_down = min(("decode_elias", "decode_elias_sparse"), key=lambda k: kern_tab[k]["avg_us"])
        kern_tab[stood_down]["stood_down"] = True
    for k in kern_tab:
        kern_tab[k]["share"] = kern_tab[k]["ms_total"] / tot
        if k in alg and k != stood_down:
            kern_tab[k]["alg_GBps"] = alg[k] / (kern_tab[k]["avg_us"] * 1e-6) / 1e9
            kern_tab[k]["frac_of_%s_hbm" % peak_src] = kern_tab[k]["alg_GBps"] / hbm_peak
    dom = max(kern, key=lambda k: kern[k][0])
    traffic_tab = load_traffic().get(dom)
    traffic = None
    if traffic_tab and traffic_tab.get("bytes_per_coord") is not None and traffic_tab.get("K", K) == K:
        traffic = traffic_tab["bytes_per_coord"] * n          # ncu capture on a smaller n, scaled per coordinate
    achieved = alg.get(dom, 0) / (kern_tab[dom]["avg_us"] * 1e-6) / 1e9
    roofline = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": achieved / hbm_peak, "peak_source": peak_src, "frac_of_nominal_8000": achieved / 8000.0,
                "traffic": traffic, "alg_bytes_per_launch": alg.get(dom),
                "avg_launch_us": kern_tab[dom]["avg_us"], "share_of_kernel_time": kern_tab[dom]["share"]}

    # ---- end to end: host buffers, copies inside the timed region -----------------------------
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        pinned = [torch.empty(n, dtype=torch.float32).pin_memory() for _ in range(K)]
        for w in range(K):
            pinned[w].copy_(hp.g[w])
        x_host = torch.empty(n, dtype=torch.float32).pin_memory()
        stage = [torch.empty(n, dtype=torch.float32, device=device) for _ in range(2)]
        copy_stream = torch.cuda.Stream(device=device)
        landed = [torch.cuda.Event() for _ in range(2)]       # staging buffer holds worker w's gradient
        taken = [torch.cuda.Event() for _ in range(2)]        # the encode that read it has finished
        main = torch.cuda.current_stream(device)

        def e2e_step(i):
            # the copy of worker w + 1 (copy stream) overlaps the encode of worker w (main stream)
            for code in hp.codes:
                for w in range(K):
                    b = w & 1
                    with torch.cuda.stream(copy_stream):
                        copy_stream.wait_event(taken[b])
                        stage[b].copy_(pinned[w], non_blocking=True)
                        landed[b].record(copy_stream)
                    main.wait_event(landed[b])
                    Q.qsgd_encode(stage[b], hp.d, hp.s, hp.norm, code, PHILOX_SEED, i, w, hp.msgs[code][w],
                                  hp.bits[code][w], hp.ws[code][0], hp.status)
                    taken[b].record(main)
                hp.decode(code)
                x_host.copy_(hp.x, non_blocking=True)
            torch.cuda.synchronize()

        e2e_step(0)
        barrier()
        ev0.record()
        for i in range(e2e_steps):
            e2e_step(1 + i)
        ev1.record()
        barrier()
        t = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device=device)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item()) / e2e_steps
        e2e = {"value": grad_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": len(hp.codes) * K * 4 * n,
               "d2h_bytes_per_step": len(hp.codes) * 4 * n,
               "overlap": "H2D copy of worker w+1 on a second stream under the encode of worker w"}
        del pinned, x_host, stage

    # ---- CPU baseline: the oracle on a bounded sample -----------------------------------------
    cpu = None
    if rank == 0 and not args.no_cpu:
        cpu = run_oracle_sample(wl, steps=1)
        cpu["host_cores"] = os.cpu_count()
        cpu["all_cores"] = run_oracle_parallel(wl)

    if clocks and clocks.get("sm_mhz"):
        # time x median SM clock: how a kernel's duration would move with the clock, were it core-bound
        for k in kern_tab:
            kern_tab[k]["kcycles_at_median_sm_clock"] = kern_tab[k]["avg_us"] * clocks["sm_mhz"] / 1e3

    if rank == 0:
        line = {
            "metric": "QSGD encode + decode+aggregate throughput, fp32 gradient GB/s",
            "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_one_stream": ms_one_stream, "ms_per_step_with_events": ms_events,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload + ": " + wl["desc"], "n": n, "bucket": hp.d, "s": hp.s,
                       "norm": wl["norm"], "codes": wl["codes"], "K": K,
                       "l2": "inputs larger than L2 (K gradients = %.0f MB rotate through 126 MB)" % (K * 4 * n / 1e6),
                       "step": "per code kind: K encodes, fused decode+aggregate+SGD (tables found on the device; "
                               "no host read-back inside a step)",
                       "streams": "the K independent encodes issued round-robin on %d stream(s), a workspace each; "
                                  "the decode after all of them" % hp.n_streams},
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "roofline": roofline, "cpu_baseline": cpu, "phases": phases, "kernels": kern_tab,
        }
        emit(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Bandwidth sweep (n = 2^28 unless --n): bucket x levels x norm x code, K peers. One N(0,1)
    gradient buffer is encoded under K worker ids (K x 1 GiB of distinct gradients is avoided);
    it is 1 GiB, so every encode reads it HBM-cold. Per point: encode and decode+SGD times (median
    of 3), GB/s of fp32 gradient, algorithmic GB/s and fraction of the HBM peak."""
    import torch
    import paper_1610_02132_b200 as Q
    if getattr(args, 'no_chaining', False):
        Q.qsgd_set_launch_chaining(False)
    from paper_1610_02132_b200 import inputs as I
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n = args.n or 2 ** 28
    K = args.K or 16
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm = peaks.get("hbm_gbs") or 6650.0
    g = I.gaussian_device(n, 1.0, seed=1, device=dev)
    x = torch.zeros(n, dtype=torch.float32, device=dev)
    status = Q.new_status(dev)
    points = []
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for d in (128, 512, 4096):
        for s in (1, 3, 15, 255):
            for norm in ("l2", "max"):
                for cname in ("fixed", "elias"):
                    code = CODE[cname]
                    B = (n + d - 1) // d
                    MF = fixed_bytes(n, d, s)
                    cap = MF if code == 0 else min(Q.qsgd_message_capacity(n, d, s, code), 2 * MF + 8 * (B + 1))
                    msgs = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(K)]
                    bits = torch.zeros(K, 4, dtype=torch.int64, device=dev)
                    ws = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code), 16), dtype=torch.uint8, device=dev)
                    t_enc, t_dec, info = [], [], None
                    for rep in range(4):
                        torch.cuda.synchronize()
                        ev[0].record()
                        for w in range(K):
                            Q.qsgd_encode(g, d, s, NORM[norm], code, PHILOX_SEED, rep, w, msgs[w], bits[w], ws, status)
                        ev[1].record()
                        tables = None
                        info = bits.cpu().numpy().view(np.uint64)
                        if code != 0:
                            nb = 8 * (B + 1)
                            tables = [msgs[w][int(info[w, 1]): int(info[w, 1]) + nb].view(torch.int64) for w in range(K)]
                        torch.cuda.synchronize()
                        ev[1].record()
                        Q.qsgd_decode_sgd_step(msgs, tables, n, d, s, code, x, ETA, status)
                        ev[2].record()
                        torch.cuda.synchronize()
                        if rep:                                        # first repetition warms up
                            t_dec.append(ev[1].elapsed_time(ev[2]) * 1e-3)
                        torch.cuda.synchronize()
                        ev[0].record()
                        for w in range(K):
                            Q.qsgd_encode(g, d, s, NORM[norm], code, PHILOX_SEED, rep, w, msgs[w], bits[w], ws, status)
                        ev[1].record()
                        torch.cuda.synchronize()
                        if rep:
                            t_enc.append(ev[0].elapsed_time(ev[1]) * 1e-3 / K)
                    st = int(status.item())
                    assert st == 0, "device status %d at d=%d s=%d %s %s" % (st, d, s, norm, cname)
                    te, td = statistics.median(t_enc), statistics.median(t_dec)
                    M = float(MF) if code == 0 else float(np.mean(info[:, 2].astype(np.float64)))
                    pay_bits = 8.0 * MF / n if code == 0 else float(np.mean(info[:, 0].astype(np.float64))) / n
                    points.append({
                        "d": d, "s": s, "norm": norm, "code": cname,
                        "bits_per_coord_payload": round(pay_bits, 4), "bits_per_coord_message": round(8 * M / n, 4),
                        "encode_us": round(te * 1e6, 1), "decode_sgd_us": round(td * 1e6, 1),
                        "encode_GBps_fp32": round(4 * n / te / 1e9, 1), "decode_sgd_GBps_fp32": round(K * 4 * n / td / 1e9, 1),
                        "encode_alg_GBps": round((4 * n + M) / te / 1e9, 1),
                        "decode_alg_GBps": round((K * M + 8 * n) / td / 1e9, 1),
                        "encode_frac_measured_hbm": round((4 * n + M) / te / 1e9 / hbm, 3),
                        "decode_frac_measured_hbm": round((K * M + 8 * n) / td / 1e9 / hbm, 3),
                        "encode_frac_nominal_8000": round((4 * n + M) / te / 1e9 / 8000.0, 3),
                        "decode_frac_nominal_8000": round((K * M + 8 * n) / td / 1e9 / 8000.0, 3)})
                    del msgs, ws
    ref = [p for p in points if (p["d"], p["s"], p["norm"], p["code"]) == (512, 15, "l2", "fixed")][0]
    value = (2 * K * 4 * n) / (K * ref["encode_us"] * 1e-6 + ref["decode_sgd_us"] * 1e-6) / 1e9
    emit(json.dumps({
        "metric": "QSGD encode + decode+aggregate throughput, fp32 gradient GB/s", "value": value, "unit": "GB/s",
        "n_gpus": 1, "steps": 3, "warmup": 1, "ms_per_step": (K * ref["encode_us"] + ref["decode_sgd_us"]) * 1e-3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "sweep: N(0,1), n=%d, K=%d, bucket x s x norm x code; value quoted at d=512, s=15, "
                               "2-norm, fixed-width" % (n, K), "hbm_peak_GBps": hbm},
        "points": points}))


def run_multi(args):
    """Algorithm 1 across GPUs, K workers on N ranks (N divides K): rank r plays workers
    r * K / N ... and, per step and code kind, encodes their gradients into its slots, all-gathers
    the K messages (NCCL; they land in this GPU's own memory) and runs the same fused decode +
    aggregate + SGD step over all K as the one-GPU bench does. Beside it, timed the same way, the
    uncompressed arm: local sum of the rank's gradients, fp32 all-reduce, plain step."""
    import torch
    import torch.distributed as dist
    import paper_1610_02132_b200 as Q
    if getattr(args, 'no_chaining', False):
        Q.qsgd_set_launch_chaining(False)
    from paper_1610_02132_b200 import exchange as X

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=device)
    wl = dict(WORKLOADS[args.workload])
    for k in ("n", "d", "s", "K"):
        if getattr(args, k) is not None:
            wl[k] = getattr(args, k)
    if args.norm:
        wl["norm"] = args.norm
    if args.codes:
        wl["codes"] = args.codes.split(",")
    if wl.get("policy"):
        raise SystemExit("the per-tensor policy workloads run on one GPU")
    n, d, s, K = wl["n"], wl["d"], wl["s"], wl["K"]
    if K % world:
        raise SystemExit("--gpus %d must divide the workload's K = %d workers" % (world, K))
    W = K // world
    norm = NORM[wl["norm"]]
    B = (n + d - 1) // d
    g = [device_gradient(wl, rank * W + w, device) for w in range(W)]
    x = torch.zeros(n, dtype=torch.float32, device=device)
    x_ref = torch.zeros(n, dtype=torch.float32, device=device)
    gsum = torch.empty(n, dtype=torch.float32, device=device)
    status = Q.new_status(device)
    ex, ws = {}, {}
    for cname in wl["codes"]:
        code = CODE[cname]
        cap = Q.qsgd_message_capacity(n, d, s, code)
        if code != 0:        # an Elias message longer than twice the fixed-width one is not worth sending
            cap = min(cap, 2 * fixed_bytes(n, d, s) + 8 * (B + 1))
        ex[code] = X.Exchange(cap, W, device)
        ws[code] = torch.empty(max(Q.qsgd_workspace_bytes(n, d, s, code), 16), dtype=torch.uint8, device=device)
    exact = not args.capacity_slots

    def step(i):
        for cname in wl["codes"]:
            code = CODE[cname]
            e = ex[code]
            for w in range(W):
                out, info = e.local_slot(w)
                Q.qsgd_encode(g[w], d, s, norm, code, PHILOX_SEED, i, rank * W + w, out, info, ws[code], status)
            msgs, infos, nbytes = e.run(exact=exact and code != 0, with_info=code != 0)
            Q.qsgd_decode_sgd_step_packed(msgs, infos if code != 0 else None, n, d, s, code, x, ETA, status,
                                          msg_bytes=nbytes)

    def step_allreduce():
        for _ in wl["codes"]:
            torch.add(g[0], g[1], out=gsum) if W > 1 else gsum.copy_(g[0])
            for w in range(2, W):
                gsum.add_(g[w])
            dist.all_reduce(gsum)
            x_ref.add_(gsum, alpha=-ETA / K)

    def timed(fn, steps):
        dist.barrier(); torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for i in range(steps):
            fn(i)
        ev1.record()
        dist.barrier(); torch.cuda.synchronize()
        t = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item()) / steps

    for i in range(args.warmup):
        step(i)
        step_allreduce()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    l0 = Q.qsgd_launch_count()
    ms_step = timed(lambda i: step(args.warmup + i), args.steps)
    launches = Q.qsgd_launch_count() - l0
    clocks = sampler.stop() if rank == 0 else None
    ms_allreduce = timed(lambda i: step_allreduce(), args.steps)
    assert int(status.item()) == 0, "device status %d" % int(status.item())
    sizes = {c: ex[CODE[c]].infos[:, 2].double().mean().item() if CODE[c] != 0 else float(fixed_bytes(n, d, s))
             for c in wl["codes"]}
    # fp32 gradient bytes through Encode (each worker once) plus through Decode (all K on every rank)
    grad_bytes = len(wl["codes"]) * (K * 4 * n + world * K * 4 * n)
    if rank == 0:
        emit(json.dumps({
            "metric": "QSGD encode + decode+aggregate throughput, fp32 gradient GB/s",
            "value": grad_bytes / (ms_step * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload + ": " + wl["desc"], "n": n, "bucket": d, "s": s,
                       "norm": wl["norm"], "codes": wl["codes"], "K": K,
                       "parallelism": "rank plays K/N = %d workers; NCCL all-gather of the K messages into local "
                                      "memory; every rank decodes all K" % W,
                       "slots": "exact (one 32-byte-per-message read-back per Elias exchange)" if exact
                                else "capacity (no host synchronisation)",
                       "l2": "inputs larger than L2 between steps"},
            "gpu_launches": int(launches), "clocks": clocks,
            "message_bytes": sizes,
            "allreduce_fp32": {"ms_per_step": ms_allreduce, "what": "per code kind: local sum of the rank's "
                               "gradients, dist.all_reduce of n fp32 values, x -= (eta/K) sum",
                               "speedup_of_qsgd_step": ms_allreduce / ms_step}}))
    dist.destroy_process_group()


def spawn_ranks(n_gpus):
    """`python bench.py --gpus N` without a launcher: start N ranks on this node, one per GPU."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "VERSION")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd, env=env, stdout=_REAL_STDOUT))     # the ranks' JSON line goes to our real stdout


# ------------------------------------------------------------------------------------------------
# the reference arm / CPU baseline: the oracle, as it stands, on host cores
# ------------------------------------------------------------------------------------------------
def run_oracle_sample(wl, steps=1, workers=2):
    """Times the oracle on a bounded sample: the first `workers` of the K workers' gradients at
    full n (capped at 2^25 coordinates), every code kind of the workload: encode each, then
    decode + aggregate + SGD step."""
    from oracle import oracle as O
    plan = None
    if wl.get("policy"):                              # the policy needs the whole tensor list
        n = wl["n"]
        plan = O.policy_plan(policy_sizes(wl["policy"]), wl["d"])
    else:
        n = min(wl["n"], 2 ** 25)
        n -= n % wl["d"] if n > wl["d"] else 0
    d, s, norm = wl["d"], wl["s"], NORM[wl["norm"]]
    gs = [host_gradient(wl, w, n) for w in range(workers)]
    x = np.zeros(n, dtype=np.float32)
    t_total, bytes_total = 0.0, 0
    for it in range(steps):
        for code_name in wl["codes"]:
            code = CODE[code_name]
            t0 = time.perf_counter()
            msgs, tabs, infos = [], [], []
            for w, g in enumerate(gs):
                if plan is not None:
                    m, info = O.policy_encode(g, plan, s, norm, code, PHILOX_SEED, it, w)
                else:
                    m, info = O.encode(g, d, s, norm, code, PHILOX_SEED, it, w)
                    tabs.append(None if code == 0 else O.message_table(m, info, n, d))
                msgs.append(m)
                infos.append(info)
            if plan is not None:
                st, acc = O.policy_decode_accumulate(msgs, infos, plan, s, code)
            else:
                st, acc = O.decode_accumulate(msgs, None if code == 0 else tabs, n, d, s, code)
            x = O.sgd_step(x, acc, ETA, workers)
            t_total += time.perf_counter() - t0
            bytes_total += 2 * workers * 4 * n
    return {"value": bytes_total / t_total / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "seconds": t_total,
            "sample": "%d of %d workers, first %d of %d coordinates, codes %s, %d step(s)" % (
                workers, wl["K"], n, wl["n"], ",".join(wl["codes"]), steps)}


def run_oracle_parallel(wl, n_cap=2 ** 23):
    """Second CPU figure: min(K, host cores) independent oracle instances, one thread each (the
    oracle itself is single-threaded; its C calls release the interpreter lock). An instance encodes
    one worker's gradient (first n_cap coordinates) under every code kind of the workload and decodes
    that message into a step."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle as O
    if wl.get("policy"):
        return None
    T = max(1, min(wl["K"], os.cpu_count() or 1))
    n = min(wl["n"], n_cap)
    n -= n % wl["d"] if n > wl["d"] else 0
    d, s, norm = wl["d"], wl["s"], NORM[wl["norm"]]
    gs = [host_gradient(wl, w, n) for w in range(T)]

    def instance(w):
        x = np.zeros(n, dtype=np.float32)
        for code_name in wl["codes"]:
            code = CODE[code_name]
            m, info = O.encode(gs[w], d, s, norm, code, PHILOX_SEED, 0, w)
            tabs = None if code == 0 else [O.message_table(m, info, n, d)]
            st, acc = O.decode_accumulate([m], tabs, n, d, s, code)
            x = O.sgd_step(x, acc, ETA, 1)
        return x[0]

    t0 = time.perf_counter()
    with ThreadPoolExecutor(T) as pool:
        list(pool.map(instance, range(T)))
    dt = time.perf_counter() - t0
    return {"value": T * len(wl["codes"]) * 2 * 4 * n / dt / 1e9, "unit": "GB/s", "cores": T,
            "host_cores": os.cpu_count(), "kind": "oracle, %d independent instances on %d threads" % (T, T),
            "seconds": dt, "sample": "each instance: 1 worker, first %d of %d coordinates, codes %s" % (
                n, wl["n"], ",".join(wl["codes"]))}


def run_qsvrg(args):
    """QSVRG (Section 3.3) on a synthetic ridge least-squares problem, n = 4096 (one bucket, s = 64),
    K = 8 processors, dense code: time per inner iteration (K encodes + one fused decode + the torch
    gradient arithmetic). Vectors of 16 KB make this launch-bound; reported for completeness."""
    import torch
    import paper_1610_02132_b200 as Q
    if getattr(args, 'no_chaining', False):
        Q.qsgd_set_launch_chaining(False)
    from paper_1610_02132_b200 import inputs as I
    from paper_1610_02132_b200 import qsvrg as GV
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    n, m, K, lam = 4096, 16384, 8, 0.1
    A, b = I.least_squares_problem(m, n, seed=1)
    gs, gj = GV.least_squares_gradients(torch.from_numpy(A).cuda(), torch.from_numpy(b).cuda(), lam, K)
    T = max(args.steps, 1) * 20
    idx = I.sample_indices(2, T, K, m, seed=3)
    eta = 0.1 / (1 + lam)
    GV.qsvrg(gs, gj, n, K, 1, max(args.warmup, 3) * 5, eta, idx, np.zeros(n, np.float32))      # warm-up
    torch.cuda.synchronize()
    l0 = Q.qsgd_launch_count()
    t0 = time.perf_counter()
    out = GV.qsvrg(gs, gj, n, K, 1, T, eta, idx, np.zeros(n, np.float32))
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    A64, b64 = A.astype(np.float64), b.astype(np.float64)
    f = lambda x: 0.5 * np.mean((A64 @ x - b64) ** 2) + 0.5 * lam * np.dot(x, x)  # noqa: E731
    line = {
        "metric": "QSGD encode + decode+aggregate throughput, fp32 gradient GB/s",
        "value": 2 * K * 4 * n * (T + 1) / dt / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": T, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / (T + 1), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "qsvrg: ridge least squares, unit rows, one epoch", "n": n, "bucket": n, "s": 64,
                   "norm": "l2", "codes": ["elias_dense"], "K": K, "m": m, "T": T},
        "gpu_launches": int(Q.qsgd_launch_count() - l0),
        "bits_per_processor": int(out["bits"][0]), "bound_bits": float((32 + 2.8 * n) * (T + 1)),
        "f_start": float(f(np.zeros(n))), "f_after_epoch": float(f(out["y"][-1].astype(np.float64))),
    }
    emit(json.dumps(line))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = dict(WORKLOADS[args.workload])
    for k in ("n", "d", "s", "K"):
        if getattr(args, k) is not None:
            wl[k] = getattr(args, k)
    for i in range(args.warmup):
        run_oracle_sample(wl, steps=1, workers=1)
        break                                         # one warm-up pass pages the library in
    t0 = time.perf_counter()
    cpu = run_oracle_sample(wl, steps=args.steps, workers=2)
    dt = time.perf_counter() - t0
    line = {
        "impl": "reference", "metric": "QSGD encode + decode+aggregate throughput, fp32 gradient GB/s",
        "value": cpu["value"], "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cpu["seconds"] / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "wall_s": dt,
        "config": {"workload": args.workload + ": " + wl["desc"], "n": wl["n"], "bucket": wl["d"],
                   "s": wl["s"], "norm": wl["norm"], "codes": wl["codes"], "K": wl["K"]},
        "cpu_baseline": cpu,
        "e2e": {"value": cpu["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    emit(json.dumps(line))


def main():
    claim_stdout()
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS) + ["sweep", "qsvrg"])
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--d", type=int, default=None)
    ap.add_argument("--s", type=int, default=None)
    ap.add_argument("--K", type=int, default=None)
    ap.add_argument("--norm", default=None, choices=["l2", "max"])
    ap.add_argument("--codes", default=None, help="comma list of fixed,elias,elias_dense")
    ap.add_argument("--streams", type=int, default=2,
                    help="streams the K independent encodes of a step are issued on (1 = everything on one stream)")
    ap.add_argument("--no-chaining", action="store_true",
                    help="plain stream-ordered launches (no programmatic dependent launch)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--replicas", action="store_true",
                    help="with more than one GPU: independent replicas of the one-GPU workload (no collective) "
                         "instead of Algorithm 1 across the GPUs")
    ap.add_argument("--exchange", action="store_true",
                    help="run the multi-GPU path (encode into slots, NCCL all-gather, packed decode, all-reduce arm) "
                         "even with a single rank: exercises that path on one GPU")
    ap.add_argument("--capacity-slots", action="store_true",
                    help="multi-GPU: all-gather whole capacity slots (no host synchronisation) instead of slots "
                         "cut to the longest message of the step")
    ap.add_argument("--capture", action="store_true",
                    help="for runs under a profiler: keep --warmup as given, skip e2e and the CPU baseline")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 1 if args.steps is None else min(args.steps, 4)
        run_reference(args)
        return
    world = int(os.environ.get("WORLD_SIZE", "0"))
    if world == 0 and args.gpus > 1:
        spawn_ranks(args.gpus)
    if args.steps is None:
        args.steps = 10
    if args.capture:
        args.no_e2e = args.no_cpu = True
    else:
        args.warmup = max(args.warmup, 3)
    if args.workload == "sweep":
        run_sweep(args)
    elif args.workload == "qsvrg":
        run_qsvrg(args)
    elif (max(world, 1) > 1 and not args.replicas) or args.exchange:
        run_multi(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
