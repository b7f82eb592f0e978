#!/usr/bin/env python
"""Benchmark of the DQ-SGD quantizer hot path on B200.

One step = one communication round of Algorithm 1 on one batch of synthetic
gradients, all through the C-ABI library: bucket norms and quantize+pack in one
pass with the bit width chosen after the previous round, unpack+dequantize+average,
and the bit rule for the next round beside the average.  The same steps as four
separate calls (norms -> bit rule -> quantize+pack -> average) and with the
parameter update folded into the average are timed as secondary figures.
The workload is the ResNet-18-shaped gradient
(62 tensors, 11,173,962 fp32 per worker, M = 8 workers, bucket 512, Laplace
values, dynamic b over T = 100 steps, norms shrinking by 0.98 per step).

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
WORKLOAD = "resnet18-cifar10 gradient, 62 tensors, d=11173962 fp32/worker, M=8, bucket=512, Laplace, dynamic b, T=100"
SEED = 2107
POOL_BYTES = 40 << 30          # device memory the pre-generated inputs may take


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# Sources whose text decides what each timed call moves through DRAM: a counter capture
# stays valid only while their digest is the one stored beside it.
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


def _traffic(kernel_key: str):
    """DRAM bytes per launch from the committed ncu capture, or None if one of the
    kernel's sources changed since the capture."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        rec = json.load(fh).get(kernel_key)
    if not rec or rec.get("sha256") != _sources_digest(kernel_key):
        return None
    return rec


class ClockSampler:
    """Samples SM clocks and clock-event reasons through NVML (read-only) from a thread while the timed
    region runs; only samples taken between ``start`` and ``stop`` count."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, uuid: str, period_s: float = 0.004):
        self.uuid, self.period = uuid, period_s
        self.samples = []
        self.handle = None
        self._run = False
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
            try:
                self._one()
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.handle is None:
            return
        self.samples = []
        self._run = True
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def stop(self):
        if self.handle is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["NVML unavailable"]}
        self._run = False
        self.thread.join(timeout=2)
        sm = [m for m, _ in self.samples]
        reasons = set()
        for _, mask in self.samples:
            for bit, name in self.REASONS.items():
                if mask & bit:
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------
# reference arm: the CPU checker, as it stands, on the host cores
# --------------------------------------------------------------------------

def _oracle_round(oracle, np, w, ref, g, t, eps_hat, alpha):
    norms = oracle.bucket_norms(ref, g)
    b, s, _ = oracle.choose_bits(norms, w.T, t, eps_hat, alpha)
    packed = oracle.quantize_pack(ref, g, norms, b, SEED, t)
    out = oracle.unpack_dequant_average(ref, packed, norms, b)
    return b, out


def run_reference(args) -> dict:
    import numpy as np

    import oracle
    from paper_2107_14575_b200 import workloads
    factor = 16
    full = workloads.config_resnet18()
    w = workloads.scaled_down(full, factor)
    ref = oracle.Layout(w.segments, w.bucket)
    cores = os.cpu_count() or 1
    oracle.set_threads(cores)
    pool = [workloads.make_grads(w, ref.offsets, ref.D32, step=t) for t in range(4)]
    n0 = oracle.bucket_norms(ref, pool[0])
    G2 = float((n0.astype(np.float64) ** 2).sum() / w.M)
    alpha = full.alpha
    eps_hat = full.T * alpha ** (full.T - 1) * G2 / full.x0 ** 2
    for i in range(args.warmup):
        _oracle_round(oracle, np, w, ref, pool[i % 4], i % full.T, eps_hat, alpha)
    t0 = time.perf_counter()
    for i in range(args.steps):
        _oracle_round(oracle, np, w, ref, pool[i % 4], i % full.T, eps_hat, alpha)
    dt = time.perf_counter() - t0
    gbs = 4.0 * w.M * w.d * args.steps / dt / 1e9
    sample = "every tensor of the workload cut to 1/%d of its size (d=%d per worker), all M=8 workers" % (factor, w.d)
    return {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


# --------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------

def _gen_step(torch, gen, scale_vec, M, D32, step):
    """Laplace(0, scale_l * 0.98^step) per tensor l, zero on padding; [M, D32] fp32 on the device."""
    u = torch.rand((M, D32), generator=gen, device=scale_vec.device, dtype=torch.float32) - 0.5
    g = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_(max=0.4999999))
    g.mul_(scale_vec * (0.98 ** step))
    return g


def run_cuda(args) -> dict:
    import numpy as np
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

    w = workloads.config_resnet18()
    rnd = Round(w.segments, w.bucket, w.M, device=str(dev))
    L = rnd.layout
    M, D32, T = w.M, L.D32, w.T
    nseg = len(w.segments)

    scale_vec = torch.zeros(D32, dtype=torch.float32, device=dev)
    for i, n in enumerate(w.segments):
        scale_vec[L.offsets[i]: L.offsets[i] + n] = 1e-2 * 10.0 ** (-i / (nseg - 1))

    K, W = args.steps, args.warmup
    step_bytes = 4 * M * D32
    npool = max(2, min(K + W, POOL_BYTES // step_bytes))
    if npool > T:
        npool = T                              # one input set per schedule step: set i % T belongs to step t = i % T
    gen = torch.Generator(device=dev)
    gen.manual_seed(SEED + 1000 * rank)
    # pool entry p is the input of every step i with i % npool == p; it carries the
    # norm decay of schedule step t = p % T
    pool = [_gen_step(torch, gen, scale_vec, M, D32, p % T) for p in range(npool)]

    # calibrate eps_hat so that x(t = 0) = x0 (b = 4 at the start of the schedule)
    rnd.norms_(pool[0])
    G2 = float((rnd.norms.double() ** 2).sum().item() / M)
    alpha = w.alpha
    eps_hat = T * alpha ** (T - 1) * G2 / w.x0 ** 2

    def rule_for(i):
        return dq.Rule.dynamic(T, i % T, eps_hat, alpha)

    peak, peak_src = _peaks()
    elems = M * D32

    def b_of(norm_set, t):
        """b the rule gives at schedule step t for the norms of input set `norm_set` (synchronises)."""
        rnd.norms_(pool[norm_set % npool])
        rnd.bits_(dq.Rule.dynamic(T, t % T, eps_hat, alpha))
        return rnd.bits()

    # Two orders of the same four steps (both supported by the library):
    #  "algorithm1": as Algorithm 1 of the paper runs -- quantize with b_t, which was chosen from the
    #     previous step's norms, in ONE pass together with the norms (dq_norms_quantize_pack), average,
    #     then choose b_{t+1} from this step's norms.  This is the timed headline.
    #  "four_call": norms, bit rule on this step's own norms, quantize (second pass), average.
    host_ms = {}

    def run_order(order, sampler=None):
        if order in ("algorithm1", "algorithm1_update"):
            names = ["norms_quantize_pack", "unpack_dequant_average" if order == "algorithm1" else "unpack_average_update",
                     "choose_bits"]
            bits = [b_of(0, 0)] + [b_of(i - 1, i) for i in range(1, K)]          # untimed: b of every step
        else:
            names = ["bucket_norms", "choose_bits", "quantize_pack", "unpack_dequant_average"]
            bits = [b_of(i, i) for i in range(K)]

        def one_step(i, e):
            g = pool[i % npool]
            if order == "algorithm1":
                rnd.step_fused(g, rule_for(i + 1), SEED, i, overlap=not args.no_overlap, events=e)
            elif order == "algorithm1_update":
                rnd.step_fused(g, rule_for(i + 1), SEED, i, overlap=not args.no_overlap, events=e, params=params,
                               lr=1e-3)
            else:
                rec = (lambda j: e[j].record()) if e else (lambda j: None)
                rec(0); rnd.norms_(g)
                rec(1); rnd.bits_(rule_for(i))
                rec(2); rnd.quantize_(g, SEED, i)
                rec(3); rnd.average_()
                rec(4)

        nev = 5
        b_of(0, 0)                                  # dev_b holds b_0 before the first step
        dummy = [torch.cuda.Event(enable_timing=True) for _ in range(nev)]
        for i in range(max(W, 3)):
            one_step(i, dummy)
        b_of(0, 0)
        torch.cuda.synchronize()
        assert rnd.read_status() == 0, "device status %d" % rnd.read_status()
        # Per-call events cost about 3 us of device time each (the stream drains around them), so only
        # every `ev_stride`-th timed step carries them; the others run as a user's steps do.
        ev_stride = max(1, K // 12)
        ev = {i: [torch.cuda.Event(enable_timing=True) for _ in range(nev)] for i in range(0, K, ev_stride)}
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler:
            sampler.start()
        start.record()
        h0 = time.perf_counter()
        for i in range(K):
            one_step(i, ev.get(i))
        end.record()
        host_ms[order] = (time.perf_counter() - h0) * 1e3 / K      # host time to submit one step
        torch.cuda.synchronize()
        clk = sampler.stop() if sampler else None
        t_ms = start.elapsed_time(end)
        assert rnd.read_status() == 0
        t_ms = replicas.max_over_ranks(t_ms, dev)
        # algorithm1: events 0-1 bracket the fused call, 1-2 the average, 3-4 the bit rule (on its own
        # stream when it overlaps the average); four_call: 0-1-2-3-4 in sequence
        spans = [(0, 1), (1, 2), (3, 4)] if order != "four_call" else [(0, 1), (1, 2), (2, 3), (3, 4)]
        totals = {n: sum(e[p].elapsed_time(e[q]) for e in ev.values()) for n, (p, q) in zip(names, spans)}
        nsamp = len(ev)
        mean_b = sum(bits) / len(bits)
        mean_bs = sum(bits[i] for i in ev) / nsamp                 # of the steps that carried events
        alg_bytes = {
            "bucket_norms": 4.0 * elems,
            "choose_bits": 4.0 * M * L.nb,
            "quantize_pack": (4.0 + mean_bs / 8.0) * elems,
            "norms_quantize_pack": (4.0 + mean_bs / 8.0) * elems,
            "unpack_dequant_average": (M * mean_bs / 8.0 + 4.0) * D32,
            "unpack_average_update": (M * mean_bs / 8.0 + 8.0) * D32,
        }
        # shares are of the time on the main stream; a bit rule that runs beside the average on the
        # second stream is not on that path (its interval there includes waiting for room on the SMs)
        beside = order != "four_call" and not args.no_overlap
        on_path = [n for n in names if not (beside and n == "choose_bits")]
        path_total = sum(totals[n] for n in on_path)
        kernels = {}
        for n in names:
            avg_ms = totals[n] / nsamp
            gbs = alg_bytes[n] / (avg_ms * 1e-3) / 1e9
            kernels[n] = {"avg_ms": round(avg_ms, 5), "achieved_gbs": round(gbs, 1), "frac": round(gbs / peak, 4),
                          "share": round(totals[n] / path_total, 4) if n in on_path else None,
                          "algorithmic_bytes_per_launch": alg_bytes[n]}
            if n not in on_path:
                kernels[n]["runs_beside"] = names[1]
        return t_ms, bits, mean_b, kernels, clk, len(names) + (1 if "choose_bits" in names else 0)

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", ""))
    ms, bits, mean_b, kernels, clocks, launches_per_step = run_order("algorithm1", sampler)
    dominant = max(kernels, key=lambda n: kernels[n]["avg_ms"])
    tr = _traffic(dominant)
    roofline = {
        "kernel": dominant, "bound": "hbm", "achieved": kernels[dominant]["achieved_gbs"], "peak": peak,
        "unit": "GB/s", "frac": kernels[dominant]["frac"], "traffic": (tr or {}).get("bytes_per_launch"),
        "peak_source": peak_src + "; of measured" if peak_src.startswith("measured") else peak_src + "; of fallback",
        "algorithmic_bytes_per_launch": kernels[dominant]["algorithmic_bytes_per_launch"], "mean_b": round(mean_b, 3),
        "frac_of_nominal_8tbs": round(kernels[dominant]["achieved_gbs"] / 8000.0, 4),
        "kernels": kernels,
    }
    # The events that bracket a single launch also see its launch latency (the stream drains at
    # every record).  For context, the same kernel launched back to back between two events:
    if dominant == "norms_quantize_pack":
        nb2b = 10
        b_last = bits[-1]
        rnd.bits_(dq.Rule.fixed(b_last))
        for i in range(3):
            rnd.norms_quantize_(pool[i % npool], SEED, i)
        torch.cuda.synchronize()
        s3, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s3.record()
        for i in range(nb2b):
            rnd.norms_quantize_(pool[i % npool], SEED, i)
        e3.record()
        torch.cuda.synchronize()
        b2b_ms = s3.elapsed_time(e3) / nb2b
        b2b_bytes = (4.0 + b_last / 8.0) * elems
        roofline["back_to_back"] = {"launches": nb2b, "b": b_last, "avg_ms": round(b2b_ms, 5),
                                    "achieved": round(b2b_bytes / (b2b_ms * 1e-3) / 1e9, 1),
                                    "frac": round(b2b_bytes / (b2b_ms * 1e-3) / 1e9 / peak, 4)}
    upd = None
    if not args.no_four_call:
        # the same order with the parameter update of Eq. 2 folded into the server step
        params = torch.zeros(D32, dtype=torch.float32, device=dev)
        msu, _, mean_bu, kernelsu, _, _ = run_order("algorithm1_update")
        upd = {"ms_per_step": msu / K, "value": replicas.whole_job_rate(4.0 * M * w.d * K, world, msu) / 1e9,
               "mean_bits": round(mean_bu, 3), "kernels": kernelsu}
    four = None
    if not args.no_four_call:
        ms4, bits4, mean_b4, kernels4, _, _ = run_order("four_call")
        four = {"ms_per_step": ms4 / K, "value": replicas.whole_job_rate(4.0 * M * w.d * K, world, ms4) / 1e9,
                "mean_bits": round(mean_b4, 3), "kernels": kernels4}

    value = replicas.whole_job_rate(4.0 * M * w.d * K, world, ms) / 1e9

    # ---- end to end: pinned host gradients in, averaged gradient out, copies timed ----
    e2e = None
    if not args.no_e2e:
        e2e = _end_to_end(torch, dist, rnd, pool, rule_for, K, world, dev, M, w.d, D32)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(W, 3),
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "bits_first_last": [bits[0], bits[-1]], "mean_bits": round(mean_b, 3),
                   "order": "Algorithm 1: norms+quantize+pack in one pass with b_t, average, b_{t+1} from this step's norms"
                            + ("" if args.no_overlap else " (bit rule on a second stream beside the average)"),
                   "l2": "inputs larger than L2 (%d MB per step, %d rotating input sets)" % (step_bytes >> 20, npool),
                   "kernel_events": "CUDA events around each call on every %d-th timed step (%d samples)"
                                    % (max(1, K // 12), len(range(0, K, max(1, K // 12)))),
                   "multi_gpu": "independent replicas, no collective" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * K, "roofline": roofline,
        # what the workers would put on the wire per step (Eq. 7: d * b bits per worker, plus the fp32 norms)
        "wire": {"bytes_per_step": M * (w.d * mean_b / 8.0 + 4.0 * L.nb), "fp32_bytes_per_step": 4.0 * M * w.d,
                 "ratio": round((w.d * mean_b / 8.0 + 4.0 * L.nb) / (4.0 * w.d), 4)},
        "four_call_order": four, "with_parameter_update": upd,
        "host_submit_ms_per_step": round(host_ms["algorithm1"], 5),
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = _cpu_baseline(pool, w, eps_hat, alpha)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out if rank == 0 else {}


def _end_to_end(torch, dist, rnd, pool, rule_for, K, world, dev, M, d, D32) -> dict:
    from paper_2107_14575_b200 import replicas
    Ke = min(K, 10)
    host = [pool[p].cpu().pin_memory() for p in range(2)]
    for i in range(2):
        rnd.step_host(host[i % 2], rule_for(i + 1), SEED, i)
    rnd.sync_host()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for i in range(Ke):
        res = rnd.step_host(host[i % 2], rule_for(i + 1), SEED, i)
    rnd.join_host()                        # the last download ends inside the timed region
    e2.record()
    rnd.sync_host()
    torch.cuda.synchronize()
    checksum = float(res[:1024].double().abs().sum())        # the result is read on the host
    ms2 = s2.elapsed_time(e2)
    ms2 = replicas.max_over_ranks(ms2, dev)
    return {"value": replicas.whole_job_rate(4.0 * M * d * Ke, world, ms2) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": 4 * M * D32, "d2h_bytes_per_step": 4 * D32, "steps": Ke,
            "ms_per_step": ms2 / Ke, "checksum": checksum}


def _cpu_baseline(pool, w, eps_hat, alpha) -> dict:
    """The CPU checker timed on full steps of the same workload (same arrays): as many steps as
    fit about twelve seconds, at least two."""
    import numpy as np

    import oracle
    ref = oracle.Layout(w.segments, w.bucket)
    cores = os.cpu_count() or 1
    oracle.set_threads(cores)
    grads = [pool[p].cpu().numpy() for p in range(min(4, len(pool)))]
    steps, dt = 0, 0.0
    while steps < 2 or (dt < 12.0 and steps < 64):
        t0 = time.perf_counter()
        _oracle_round(oracle, np, w, ref, grads[steps % len(grads)], steps % w.T, eps_hat, alpha)
        dt += time.perf_counter() - t0
        steps += 1
    out = {"value": 4.0 * w.M * w.d * steps / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "%d full steps (all %d workers, all %d tensors, t = 0..%d), %.1f s"
                     % (steps, w.M, len(w.segments), steps - 1, dt)}
    # the same checker on one thread, on one worker's share of a step
    import copy
    w1 = copy.copy(w)
    w1.M = 1
    oracle.set_threads(1)
    t0 = time.perf_counter()
    _oracle_round(oracle, np, w1, ref, grads[0][:1], 0, eps_hat, alpha)
    dt1 = time.perf_counter() - t0
    oracle.set_threads(cores)
    out["one_thread"] = {"value": 4.0 * w.d / dt1 / 1e9, "unit": UNIT, "cores": 1,
                         "sample": "one step of one worker (all %d tensors), %.1f s" % (len(w.segments), dt1)}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU checker timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-four-call", action="store_true", help="skip the secondary timing of the four separate calls")
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
