#!/usr/bin/env python
"""Benchmark of the DQ-SGD quantizer hot path on B200.

One step = one communication round of Algorithm 1 on one batch of synthetic
gradients, all through the C-ABI library: bucket norms and quantize+pack in one
pass with the bit width chosen after the previous round, unpack+dequantize+average,
and the bit rule for the next round beside the average.

The workload is the largest single-GPU point of the bandwidth sweep: one flat
N(0,1) fp32 gradient of d = 2^26 elements per worker, M = 32 workers (8 GiB of
gradients per step), bucket 512.  The headline step runs at the paper's operating
point b = 4 (chosen on the device by the rule of Eq. 17, calibrated so); the
``per_b`` table repeats the three hot kernels -- quantize+pack, norms+quantize+pack
in one pass, unpack+average -- for a list of bit widths, each as a train of launches
and as single event-bracketed launches, with achieved GB/s of algorithmic bytes, the
fraction of the measured copy bandwidth and of 8 TB/s, and which roof binds.
``size_sweep`` times the fused quantizer and the average on the other axes of the
sweep (M = 1 at d = 2^24 .. 2^30; buckets of 128 and 4096 at d = 2^26, M = 32), and the
model-shaped workloads (ResNet-18 M = 8, VGG-16 M = 16, text classifier M = 16)
are timed as secondary figures.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  ``value`` is GB/s of fp32 gradient processed
(4 * M * d bytes per step over the step time), inputs resident in HBM;
``e2e`` is the same with pinned host buffers and the copies timed.
``--impl reference`` times the CPU checker on the host cores instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "quantize+pack and unpack+average GB/s of fp32 gradient"
UNIT = "GB/s"
MAIN_D, MAIN_M, MAIN_BUCKET = 1 << 26, 32, 512
HEADLINE_B = 4
PER_B = (2, 3, 4, 5, 6, 8, 12, 16)
WORKLOAD = ("bandwidth sweep point: flat N(0,1) gradient, d=2^26 fp32/worker, M=32 workers (8 GiB/step), bucket=512, "
            "l2 norms, b=%d chosen on the device by the rule of Eq. 17" % HEADLINE_B)
SEED = 2107
NOMINAL_HBM_GBS = 8000.0
SCHEDULERS_PER_SM = 4          # one warp instruction per scheduler and cycle is the issue roof


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs); of measured"
    return 6650.0, "fallback (earlier measurement on this pool); of fallback"


# Sources whose text decides what each timed call moves through DRAM and how many instructions
# it issues: a counter capture stays valid only while their digest is the one stored beside it.
KERNEL_SOURCES = {
    "norms_quantize_pack": ["dq_fused.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"],
    "quantize_pack": ["dq_quantize.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"],
    "bucket_norms": ["dq_norms.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"],
    "unpack_dequant_average": ["dq_unpack.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"],
    "choose_bits": ["dq_bits.cu", "dq_common.cuh"],
}


def _sources_digest(kernel_key: str) -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel_key]:
        with open(os.path.join(ROOT, "paper_2107_14575_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _counters(kernel_key: str):
    """The committed ncu counters of a kernel (DRAM bytes and warp instructions per unit of work), or
    None if one of the kernel's sources changed since the capture."""
    path = os.path.join(ROOT, "profiles", "counters.json")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        rec = json.load(fh).get(kernel_key)
    if not rec or rec.get("sha256") != _sources_digest(kernel_key):
        return None
    return rec


def _interp(table: dict, b: int):
    """Value at bit width b of a {"b": value} table measured at a few b (linear between neighbours)."""
    if not table:
        return None
    pts = sorted((int(k), float(v)) for k, v in table.items())
    if b <= pts[0][0]:
        return pts[0][1]
    for (b0, v0), (b1, v1) in zip(pts, pts[1:]):
        if b <= b1:
            return v0 + (v1 - v0) * (b - b0) / (b1 - b0)
    return pts[-1][1]


class ClockSampler:
    """Samples SM clocks and clock-event reasons through NVML (read-only) from a thread while the timed
    region runs; only samples taken between ``start`` and ``stop`` count."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, uuid: str, period_s: float = 0.002):
        self.uuid, self.period = uuid, period_s
        self.samples = []
        self.handle = None
        self._run = False
        self._active = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:                       # no NVML: the line says so instead of guessing
            self.handle = None

    def _one(self):
        nv = self.nv
        mhz = float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
        try:
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
        except Exception:
            mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
        self.samples.append((mhz, mask))

    def _loop(self):
        while self._run:
            if self._active:
                try:
                    self._one()
                except Exception:
                    pass
            time.sleep(self.period)

    def start(self):
        """Opens a sampling window.  The thread is started once, ahead of the first window, and idles between
        windows, so that a window of a few tens of milliseconds is sampled from its first period on."""
        if self.handle is None:
            return
        if not self._run:
            self._run = True
            self._active = False
            self.thread = threading.Thread(target=self._loop, daemon=True)
            self.thread.start()
            try:
                self._one()                      # the first NVML queries of a process are the slow ones
            except Exception:
                pass
        self.samples = []
        self._active = True

    def stop(self):
        if self.handle is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["NVML unavailable"]}
        self._active = False
        time.sleep(self.period)                  # a query in flight ends
        sm = [m for m, _ in self.samples]
        reasons = set()
        for _, mask in self.samples:
            for bit, name in self.REASONS.items():
                if mask & bit:
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------
# the CPU checker on the host cores (reference arm and cpu_baseline leg)
# --------------------------------------------------------------------------

def _calibrated_eps(G2: float, T: int, x: float) -> float:
    """eps_hat for which the rule's x = sqrt(T / eps_hat) * G-bar equals `x` at alpha = 1."""
    return T * G2 / (x * x)


def _x_for(b: int) -> float:
    """A value of x that the rule rounds up to exactly b bits: half a level below s(b) = 2^(b-1) - 1."""
    return ((1 << (b - 1)) - 1) - 0.5


def _oracle_round(oracle, ref, g, T, t, eps_hat):
    norms = oracle.bucket_norms(ref, g)
    b, s, _ = oracle.choose_bits(norms, T, t, eps_hat, 1.0)
    packed = oracle.quantize_pack(ref, g, norms, b, SEED, t)
    out = oracle.unpack_dequant_average(ref, packed, norms, b)
    return b, out


def _oracle_rate(grads, seconds: float, min_steps: int, max_steps: int, fixed_steps=None, warmup: int = 0):
    """Times whole rounds of the CPU checker on `grads` [M, d] (numpy); returns (GB/s, steps, s, b, cores)."""
    import numpy as np

    import oracle
    M, d = grads.shape
    ref = oracle.Layout([d], MAIN_BUCKET)
    cores = os.cpu_count() or 1
    oracle.set_threads(cores)
    n0 = oracle.bucket_norms(ref, grads)
    G2 = float((n0.astype(np.float64) ** 2).sum() / M)
    eps_hat = _calibrated_eps(G2, 100, _x_for(HEADLINE_B))
    b = 0
    for i in range(warmup):
        b, _ = _oracle_round(oracle, ref, grads, 100, i % 100, eps_hat)
    steps, dt = 0, 0.0
    while (steps < fixed_steps) if fixed_steps is not None else (steps < min_steps or (dt < seconds and steps < max_steps)):
        t0 = time.perf_counter()
        b, _ = _oracle_round(oracle, ref, grads, 100, steps % 100, eps_hat)
        dt += time.perf_counter() - t0
        steps += 1
    return 4.0 * M * d * steps / dt / 1e9, steps, dt, b, cores


def run_reference(args) -> dict:
    import numpy as np
    d_sample = 1 << 21
    rng = np.random.Generator(np.random.PCG64(SEED))
    g = rng.standard_normal((MAIN_M, d_sample), dtype=np.float32)
    gbs, steps, dt, b, cores = _oracle_rate(g, 0.0, 0, 0, fixed_steps=args.steps, warmup=args.warmup)
    sample = ("each step = one whole round of the CPU checker on a prefix of the workload: the first 2^21 of the 2^26 "
              "elements of all M=32 workers (268 MB of gradients), b=%d from its own bit rule" % b)
    return {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


# --------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------

class Timer:
    """CUDA-event timing on torch's current stream (the stream every library call is launched on)."""

    def __init__(self, torch, warmup: int):
        self.torch, self.warmup = torch, max(3, warmup)

    def train(self, fn, n: int) -> float:
        """ms per call of `n` calls launched back to back between two events."""
        torch = self.torch
        for i in range(self.warmup):
            fn(i)
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for i in range(n):
            fn(i)
        e.record()
        torch.cuda.synchronize()
        return s.elapsed_time(e) / n

    def single(self, fn, n: int) -> float:
        """mean ms of `n` calls each bracketed by its own pair of events (sees the launch latency too)."""
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        torch.cuda.synchronize()
        for i, (s, e) in enumerate(ev):
            s.record()
            fn(i)
            e.record()
        torch.cuda.synchronize()
        return sum(s.elapsed_time(e) for s, e in ev) / n


def _bound(kernel_key, b, alg_bytes, units, ms, peak_gbs, sm_count, sm_mhz):
    """Which roof binds a launch that took `ms`: the time its algorithmic bytes need at the measured copy
    bandwidth, or the time its warp instructions need at one instruction per scheduler and cycle
    (instructions per unit from the committed ncu counters x units, at the sampled SM clock)."""
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    rec = {"ms": round(ms, 5), "achieved_gbs": round(gbs, 1), "frac_of_measured": round(gbs / peak_gbs, 4),
           "frac_of_8tbs": round(gbs / NOMINAL_HBM_GBS, 4), "algorithmic_bytes": alg_bytes, "bound": "hbm",
           "issue": None}
    c = _counters(kernel_key)
    ipu = _interp((c or {}).get("warp_instructions_per_group"), b)
    if ipu is not None and sm_mhz:
        issue_peak = sm_count * SCHEDULERS_PER_SM * sm_mhz * 1e6            # warp instructions per second
        inst = ipu * units
        t_issue_ms = inst / issue_peak * 1e3
        t_hbm_ms = alg_bytes / (peak_gbs * 1e9) * 1e3
        rec["issue"] = {"warp_instructions_per_group": round(ipu, 1), "warp_instructions": inst,
                        "roof_ms": round(t_issue_ms, 5), "hbm_roof_ms": round(t_hbm_ms, 5),
                        "frac_of_issue_roof": round(t_issue_ms / ms, 4), "sm_mhz": sm_mhz}
        if t_issue_ms > t_hbm_ms:
            rec["bound"] = "alu"
    return rec


def _gen_resnet(torch, gen, w, L, dev, step):
    """Laplace(0, scale_l * 0.98^step) per tensor l, zero on padding; [M, D32] fp32 on the device."""
    nseg = len(w.segments)
    scale_vec = torch.zeros(L.D32, dtype=torch.float32, device=dev)
    for i, n in enumerate(w.segments):
        scale_vec[L.offsets[i]: L.offsets[i] + n] = 1e-2 * 10.0 ** (-i / (nseg - 1))
    u = torch.rand((w.M, L.D32), generator=gen, device=dev, dtype=torch.float32) - 0.5
    g = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_(max=0.4999999))
    g.mul_(scale_vec * (0.98 ** step))
    return g


def _gen_vgg(torch, gen, w, L, dev, step):
    """Gaussian values, 1% of the entries scaled x100; zero on padding."""
    mask = torch.zeros(L.D32, dtype=torch.float32, device=dev)
    for i, n in enumerate(w.segments):
        mask[L.offsets[i]: L.offsets[i] + n] = 1.0
    g = torch.randn((w.M, L.D32), generator=gen, device=dev, dtype=torch.float32) * 1e-2
    big = torch.rand((w.M, L.D32), generator=gen, device=dev, dtype=torch.float32) < 0.01
    g = torch.where(big, g * 100.0, g)
    return g * mask


def _gen_text(torch, gen, w, L, dev, step):
    """Embedding 30000 x 300 with 97% of the rows exactly zero (fresh subset per worker), dense LSTM and head."""
    g = torch.randn((w.M, L.D32), generator=gen, device=dev, dtype=torch.float32) * 1e-2
    mask = torch.zeros(L.D32, dtype=torch.float32, device=dev)
    for i, n in enumerate(w.segments):
        mask[L.offsets[i]: L.offsets[i] + n] = 1.0
    g = g * mask
    rows, cols = 30000, 300
    emb = g[:, L.offsets[0]: L.offsets[0] + rows * cols].view(w.M, rows, cols)
    keep = torch.rand((w.M, rows, 1), generator=gen, device=dev) < 0.03
    emb.mul_(keep.to(torch.float32))
    return g


def _model_workload(torch, dq, Round, timer, w, gen_fn, dev, K, peak):
    """Algorithm-1 steps of a model-shaped workload with the dynamic schedule of its config; returns the
    per-step time, the bit widths seen, and the event-bracketed time of each call."""
    rnd = Round(w.segments, w.bucket, w.M, device=str(dev))
    L = rnd.layout
    gen = torch.Generator(device=dev)
    gen.manual_seed(SEED + 17)
    npool = 3
    pool = [gen_fn(torch, gen, w, L, dev, p) for p in range(npool)]
    rnd.norms_(pool[0])
    G2 = float((rnd.norms.double() ** 2).sum().item() / w.M)
    T, alpha = w.T, w.alpha
    eps_hat = T * alpha ** (T - 1) * G2 / w.x0 ** 2

    def rule_for(i):
        return dq.Rule.dynamic(T, i % T, eps_hat, alpha)

    rnd.bits_(rule_for(0))
    b0 = rnd.bits()
    ms = timer.train(lambda i: rnd.step_fused(pool[i % npool], rule_for(i + 1), SEED, i), K)
    b1 = rnd.bits()
    # per call at the b the schedule has reached: event-bracketed single launches (the bracket leaves the GPU idle
    # for some microseconds around every launch, which counts) and trains of launches; the trains rotate through
    # `npool` sets of buffers (gradients for the quantizer, words and outputs for the average), more than the L2 holds
    elems = w.M * L.D32
    t_f = timer.single(lambda i: rnd.norms_quantize_(pool[i % npool], SEED, i), min(K, 10))
    t_a = timer.single(lambda i: rnd.average_(), min(K, 10))
    rounds = [rnd] + [Round(w.segments, w.bucket, w.M, device=str(dev)) for _ in range(npool - 1)]
    for r, g in zip(rounds, pool):
        r.bits_(dq.Rule.fixed(b1))
        r.norms_quantize_(g, SEED, 0)
    t_f_train = timer.train(lambda i: rnd.norms_quantize_(pool[i % npool], SEED, i), 3 * K)
    t_a_train = timer.train(lambda i: rounds[i % npool].average_(), 3 * K)
    for r in rounds:
        assert r.read_status() == 0, "device status %d" % r.read_status()
    bytes_f = (4.0 + b1 / 8.0) * elems
    bytes_a = (w.M * b1 / 8.0 + 4.0) * L.D32
    out = {"workload": "%s: %d tensors, d=%d fp32/worker, M=%d, bucket=%d, dynamic b over T=%d"
                       % (w.name, len(w.segments), w.d, w.M, w.bucket, w.T),
           "ms_per_step": round(ms, 5), "value": round(4.0 * w.M * w.d / (ms * 1e-3) / 1e9, 1),
           "bits_first_last": [b0, b1], "mb_per_step": (4 * elems) >> 20,
           "norms_quantize_pack": {"b": b1, "ms": round(t_f, 5),
                                   "frac_of_measured": round(bytes_f / (t_f * 1e-3) / 1e9 / peak, 4),
                                   "train_ms": round(t_f_train, 5),
                                   "train_frac_of_measured": round(bytes_f / (t_f_train * 1e-3) / 1e9 / peak, 4)},
           "unpack_dequant_average": {"b": b1, "ms": round(t_a, 5),
                                      "frac_of_measured": round(bytes_a / (t_a * 1e-3) / 1e9 / peak, 4),
                                      "train_ms": round(t_a_train, 5),
                                      "train_frac_of_measured": round(bytes_a / (t_a_train * 1e-3) / 1e9 / peak, 4)}}
    del rounds
    del pool, rnd
    torch.cuda.empty_cache()
    return out


SWEEP_B = (2, 4, 8)
# the other axes of the bandwidth sweep: (M, log2 d, bucket); the per-b table covers (32, 26, 512)
SWEEP_POINTS = ((1, 24, 512), (1, 26, 512), (1, 28, 512), (1, 30, 512), (32, 26, 128), (32, 26, 4096))


def _sweep_point(torch, dq, Round, timer, M, log2d, bucket, K, dev, peak):
    """Trains of the fused quantizer and of the average at one (M, d, bucket) of the bandwidth sweep.
    Small cases rotate through several sets of buffers so that every launch reads more than the L2 holds
    since it last saw the same addresses."""
    d = 1 << log2d
    n_rot = max(1, min(8, -(-(1 << 29) // (4 * M * d))))
    rounds = [Round([d], bucket, M, device=str(dev)) for _ in range(n_rot)]
    D32 = rounds[0].layout.D32
    gen = torch.Generator(device=dev)
    gen.manual_seed(SEED + log2d + bucket)
    grads = [torch.randn((M, D32), generator=gen, device=dev, dtype=torch.float32) for _ in range(n_rot)]
    elems = M * D32
    rec = {"M": M, "d": d, "bucket": bucket, "buffer_sets": n_rot, "mb_per_launch": (4 * elems) >> 20, "b": {}}
    for b in SWEEP_B:
        for r, g in zip(rounds, grads):
            r.bits_(dq.Rule.fixed(b))
            r.norms_quantize_(g, SEED, 0)
        t_f = timer.train(lambda i: rounds[i % n_rot].norms_quantize_(grads[i % n_rot], SEED, i), K)
        t_a = timer.train(lambda i: rounds[i % n_rot].average_(), K)
        bytes_f = (4.0 + b / 8.0) * elems
        bytes_a = (M * b / 8.0 + 4.0) * D32
        rec["b"][str(b)] = {
            "norms_quantize_pack": {"ms": round(t_f, 5), "achieved_gbs": round(bytes_f / (t_f * 1e-3) / 1e9, 1),
                                    "frac_of_measured": round(bytes_f / (t_f * 1e-3) / 1e9 / peak, 4)},
            "unpack_dequant_average": {"ms": round(t_a, 5), "achieved_gbs": round(bytes_a / (t_a * 1e-3) / 1e9, 1),
                                       "frac_of_measured": round(bytes_a / (t_a * 1e-3) / 1e9 / peak, 4)}}
        for r in rounds:
            assert r.read_status() == 0, "device status %d" % r.read_status()
    del rounds, grads
    torch.cuda.empty_cache()
    return rec


def run_cuda(args) -> dict:
    import torch
    import torch.distributed as dist

    from paper_2107_14575_b200 import dq, replicas, workloads
    from paper_2107_14575_b200.pipeline import Round

    rank, world, local = replicas.env_rank()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    K, W = args.steps, max(3, args.warmup)
    M, d = MAIN_M, MAIN_D
    rnd = Round([d], MAIN_BUCKET, M, device=str(dev))
    L = rnd.layout
    D32 = L.D32
    elems = M * D32
    groups = elems // 32
    gen = torch.Generator(device=dev)
    gen.manual_seed(SEED + 1000 * rank)
    grads = torch.randn((M, D32), generator=gen, device=dev, dtype=torch.float32)      # 8 GiB: far larger than the L2
    rnd.norms_(grads)
    G2 = float((rnd.norms.double() ** 2).sum().item() / M)
    T = 100

    def rule_b(b, t=0):
        """The dynamic rule of Eq. 17 with eps_hat calibrated so that it lands on b for these norms."""
        return dq.Rule.dynamic(T, t % T, _calibrated_eps(G2, T, _x_for(b)), 1.0)

    def set_b(b):
        rnd.bits_(rule_b(b))
        got = rnd.bits()
        assert got == b, "the device rule chose b=%d where the calibration aims at %d" % (got, b)

    peak, peak_src = _peaks()
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    timer = Timer(torch, W)
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", ""))

    # ---- headline: K steps in the order of Algorithm 1 at b = 4
    set_b(HEADLINE_B)
    for i in range(W):
        rnd.step_fused(grads, rule_b(HEADLINE_B, i + 1), SEED, i, overlap=(False if args.no_overlap else None))
    torch.cuda.synchronize()
    assert rnd.read_status() == 0, "device status %d" % rnd.read_status()
    nev = 5
    ev_stride = max(1, K // 12)
    ev = {i: [torch.cuda.Event(enable_timing=True) for _ in range(nev)] for i in range(0, K, ev_stride)}
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    start.record()
    h0 = time.perf_counter()
    for i in range(K):
        rnd.step_fused(grads, rule_b(HEADLINE_B, i + 1), SEED, i, overlap=(False if args.no_overlap else None), events=ev.get(i))
    end.record()
    host_submit_ms = (time.perf_counter() - h0) * 1e3 / K
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_total = replicas.max_over_ranks(start.elapsed_time(end), dev)
    assert rnd.read_status() == 0 and rnd.bits() == HEADLINE_B
    sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz")
    spans = {"norms_quantize_pack": (0, 1), "unpack_dequant_average": (1, 2), "choose_bits": (3, 4)}
    step_ms = {n: sum(e[p].elapsed_time(e[q]) for e in ev.values()) / len(ev) for n, (p, q) in spans.items()}
    alg_bytes = {
        "bucket_norms": lambda b: 4.0 * elems,
        "quantize_pack": lambda b: (4.0 + b / 8.0) * elems,
        "norms_quantize_pack": lambda b: (4.0 + b / 8.0) * elems,
        "unpack_dequant_average": lambda b: (M * b / 8.0 + 4.0) * D32,
    }
    # units of the instruction model: 32-element groups a launch processes (per worker for the
    # quantizers; for the average a group of M x 32 codes)
    units = {"bucket_norms": groups, "quantize_pack": groups, "norms_quantize_pack": groups,
             "unpack_dequant_average": D32 // 32}
    kernels = {n: _bound(n, HEADLINE_B, alg_bytes[n](HEADLINE_B), units[n], step_ms[n], peak, sm_count, sm_mhz)
               for n in ("norms_quantize_pack", "unpack_dequant_average")}
    path_ms = sum(step_ms[n] for n in kernels)
    for n in kernels:
        kernels[n]["share"] = round(step_ms[n] / path_ms, 4)
    kernels["choose_bits"] = {"ms": round(step_ms["choose_bits"], 5), "share": None,
                              "runs_beside": "unpack_dequant_average (second stream)" if not args.no_overlap else None,
                              "algorithmic_bytes": 4.0 * M * L.nb}
    dominant = max(("norms_quantize_pack", "unpack_dequant_average"), key=lambda n: step_ms[n])
    dk = kernels[dominant]
    cnt = _counters(dominant)
    traffic = _interp((cnt or {}).get("dram_bytes_per_group"), HEADLINE_B)
    roofline = {"kernel": dominant, "b": HEADLINE_B, "bound": dk["bound"], "unit": "GB/s", "achieved": dk["achieved_gbs"],
                "peak": peak, "frac": dk["frac_of_measured"], "peak_source": peak_src,
                "traffic": traffic * units[dominant] if traffic is not None else None,
                "algorithmic_bytes_per_launch": dk["algorithmic_bytes"], "frac_of_nominal_8tbs": dk["frac_of_8tbs"],
                "hbm": {"achieved_gbs": dk["achieved_gbs"], "frac_of_measured": dk["frac_of_measured"]},
                "kernels": kernels,
                "timing": "CUDA events on the launching stream around each call of every %d-th timed step (%d samples)"
                          % (ev_stride, len(ev))}
    if dk["bound"] == "alu":
        # the instruction roof binds: report against it (lane instructions per second; peak = SMs x 128 lanes x
        # sampled SM clock), the HBM figures stay beside it under "hbm"
        iss = dk["issue"]
        roofline.update({"unit": "Ginst/s", "achieved": round(iss["warp_instructions"] * 32 / (dk["ms"] * 1e-3) / 1e9, 1),
                         "peak": round(sm_count * SCHEDULERS_PER_SM * 32 * sm_mhz * 1e6 / 1e9, 1),
                         "frac": iss["frac_of_issue_roof"],
                         "peak_source": "SMs x 4 schedulers x 32 lanes x sampled SM clock (one warp instruction per "
                                        "scheduler and cycle); instructions per group from profiles/counters.json"})

    # ---- the same step with the parameter update of Eq. 2 applied by the averaging kernel (x <- x - eta * average)
    with_update = None
    if not args.no_per_b:
        x = torch.zeros(D32, dtype=torch.float32, device=dev)
        evu = [[torch.cuda.Event(enable_timing=True) for _ in range(nev)] for _ in range(min(K, 8))]
        for i in range(W):
            rnd.step_fused(grads, rule_b(HEADLINE_B, i + 1), SEED, i, params=x, lr=1e-3)
        torch.cuda.synchronize()
        su, eu = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        su.record()
        for i in range(K):
            rnd.step_fused(grads, rule_b(HEADLINE_B, i + 1), SEED, i, params=x, lr=1e-3,
                           events=evu[i] if i < len(evu) else None)
        eu.record()
        torch.cuda.synchronize()
        assert rnd.read_status() == 0 and rnd.bits() == HEADLINE_B
        t_u = sum(e[1].elapsed_time(e[2]) for e in evu) / len(evu)
        bytes_u = (M * HEADLINE_B / 8.0 + 8.0) * D32            # the words of M workers, x read and written
        with_update = {"ms_per_step": round(su.elapsed_time(eu) / K, 5),
                       "value": round(4.0 * M * d * K / (su.elapsed_time(eu) * 1e-3) / 1e9, 1),
                       "unpack_average_update": {"ms": round(t_u, 5), "algorithmic_bytes": bytes_u,
                                                 "achieved_gbs": round(bytes_u / (t_u * 1e-3) / 1e9, 1),
                                                 "frac_of_measured": round(bytes_u / (t_u * 1e-3) / 1e9 / peak, 4)}}
        del x

    # ---- per b: the three hot kernels, trains of K launches and single event-bracketed launches
    per_b = {}
    n_single = min(K, 8)
    norms_ms = timer.train(lambda i: rnd.norms_(grads), K)
    for b in (() if args.no_per_b else PER_B):
        set_b(b)
        rec = {}
        rnd.norms_(grads)
        for name, fn in (("quantize_pack", lambda i: rnd.quantize_(grads, SEED, i)),
                         ("norms_quantize_pack", lambda i: rnd.norms_quantize_(grads, SEED, i)),
                         ("unpack_dequant_average", lambda i: rnd.average_())):
            # a train of launches runs long enough for the power cap to pull the SM clock down: the clock
            # is sampled per train and the instruction roof of the point uses that sample
            sampler.start()
            t_train = timer.train(fn, K)
            clk = sampler.stop()
            t_single = timer.single(fn, n_single)
            r = _bound(name, b, alg_bytes[name](b), units[name], t_train, peak, sm_count, clk.get("sm_mhz") or sm_mhz)
            r["sm_mhz"] = clk.get("sm_mhz")
            r["clock_reasons"] = clk.get("reasons")
            r["single_launch_ms"] = round(t_single, 5)
            r["single_launch_frac_of_measured"] = round(alg_bytes[name](b) / (t_single * 1e-3) / 1e9 / peak, 4)
            r["gradient_gbs"] = round(4.0 * M * d / (t_train * 1e-3) / 1e9, 1)
            rec[name] = r
        step = timer.train(lambda i: rnd.step_fused(grads, rule_b(b, i + 1), SEED, i, overlap=(False if args.no_overlap else None)), K)
        rec["step_ms"] = round(step, 5)
        rec["step_gradient_gbs"] = round(4.0 * M * d / (step * 1e-3) / 1e9, 1)
        per_b[str(b)] = rec
        assert rnd.read_status() == 0 and rnd.bits() == b
    set_b(HEADLINE_B)

    value = replicas.whole_job_rate(4.0 * M * d * K, world, ms_total) / 1e9

    # ---- end to end: pinned host gradients in, averaged gradient out, copies timed
    e2e = None
    if not args.no_e2e:
        e2e = _end_to_end(torch, dist, rnd, grads, rule_b, K, world, dev, M, d, D32)

    # ---- the model-shaped workloads, then the other sizes and bucket lengths of the bandwidth sweep (secondary)
    other = None
    sweep = None
    if not (args.no_models and args.no_sweep):
        del grads
        rnd = None
        torch.cuda.empty_cache()
    if not args.no_models:
        other = {}
        for w, gen_fn in ((workloads.config_resnet18(), _gen_resnet), (workloads.config_vgg16(), _gen_vgg),
                          (workloads.config_text(), _gen_text)):
            other[w.name] = _model_workload(torch, dq, Round, timer, w, gen_fn, dev, K, peak)
    if not args.no_sweep:
        sweep = [_sweep_point(torch, dq, Round, timer, m_, l_, bk_, K, dev, peak) for m_, l_, bk_ in SWEEP_POINTS]

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD,
                   "order": "Algorithm 1: norms+quantize+pack in one pass with b_t, average, b_{t+1} from this step's norms"
                            + ("" if args.no_overlap else " (bit rule on a second stream beside the average)"),
                   "l2": "inputs larger than L2 (%d MB of gradients per step)" % ((4 * elems) >> 20),
                   "per_b": "b in %s: trains of %d launches and %d single event-bracketed launches per kernel"
                            % (list(PER_B), K, n_single),
                   "size_sweep": "M=1 at d=2^24..2^30 and buckets 128/4096 at d=2^26, M=32, b in %s: trains of %d launches, "
                                 "buffers rotated where one set would fit in the L2" % (list(SWEEP_B), K),
                   "multi_gpu": "independent replicas, no collective" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 4 * K, "roofline": roofline,
        "per_b": per_b, "bucket_norms": _bound("bucket_norms", 0, 4.0 * elems, groups, norms_ms, peak, sm_count, sm_mhz),
        # what the workers would put on the wire per step (Eq. 7: d * b bits per worker, plus the fp32 norms)
        "wire": {"bytes_per_step": M * (d * HEADLINE_B / 8.0 + 4.0 * L.nb), "fp32_bytes_per_step": 4.0 * M * d,
                 "ratio": round((d * HEADLINE_B / 8.0 + 4.0 * L.nb) / (4.0 * d), 4)},
        "with_parameter_update": with_update, "size_sweep": sweep, "model_workloads": other, "host_submit_ms_per_step": round(host_submit_ms, 5),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = _cpu_baseline(torch, gen, dev)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out if rank == 0 else {}


def _end_to_end(torch, dist, rnd, grads, rule_b, K, world, dev, M, d, D32) -> dict:
    from paper_2107_14575_b200 import replicas
    Ke = max(2, min(K, 4))
    host = torch.empty((M, D32), dtype=torch.float32, pin_memory=True)
    host.copy_(grads)
    torch.cuda.synchronize()
    for i in range(2):
        rnd.step_host(host, rule_b(HEADLINE_B, i + 1), SEED, i)
    rnd.sync_host()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for i in range(Ke):
        res = rnd.step_host(host, rule_b(HEADLINE_B, i + 1), SEED, i)
    rnd.join_host()                        # the last download ends inside the timed region
    e2.record()
    rnd.sync_host()
    torch.cuda.synchronize()
    checksum = float(res[:1024].double().abs().sum())        # the result is read on the host
    ms2 = replicas.max_over_ranks(s2.elapsed_time(e2), dev)
    return {"value": replicas.whole_job_rate(4.0 * M * d * Ke, world, ms2) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": 4 * M * D32, "d2h_bytes_per_step": 4 * D32, "steps": Ke,
            "ms_per_step": ms2 / Ke, "checksum": checksum,
            "api": "pipeline.Round.step_host: pinned host gradients in, averaged gradient back in pinned host memory"}


def _cpu_baseline(torch, gen, dev) -> dict:
    """The CPU checker timed on whole rounds over a prefix of the same workload (drawn by the same
    generator): about twelve seconds of work, at least two rounds."""
    d_sample = 1 << 23
    g = torch.randn((MAIN_M, d_sample), generator=gen, device=dev, dtype=torch.float32).cpu().numpy()
    gbs, steps, dt, b, cores = _oracle_rate(g, 12.0, 2, 16)
    return {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d whole rounds (norms, bit rule, quantize+pack, unpack+average; b=%d) on 2^23 of the 2^26 elements "
                      "of all %d workers (1 GiB of gradients per round), %.1f s" % (steps, b, MAIN_M, dt)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU checker timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the M = 1 sizes and the other bucket lengths of the bandwidth sweep")
    ap.add_argument("--no-models", action="store_true", help="skip the secondary timing of the model-shaped workloads")
    ap.add_argument("--no-per-b", action="store_true", help="skip the per-b table (profiling runs)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="run the bit rule after the average on the same stream instead of beside it")
    ap.add_argument("--source-digests", action="store_true",
                    help="print the digest of each kernel's sources (stored beside a counter capture) and exit")
    args = ap.parse_args()
    if args.source_digests:
        print(json.dumps({k: _sources_digest(k) for k in KERNEL_SOURCES}, indent=1))
        return
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return
        print(json.dumps(run_reference(args)))
        return
    out = run_cuda(args)
    if out:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
