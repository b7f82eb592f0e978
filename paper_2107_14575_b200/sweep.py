"""Bandwidth sweep of the kernels on flat N(0, 1) gradients, through the C ABI.

    python -m paper_2107_14575_b200.sweep [--quick] [--out sweep.json]

Sizes d = 2^20 ... 2^30 at M = 1 and d = 2^26 at M = 32, bit widths 1..16 at bucket 512
and {2, 4, 8, 16} at buckets 128 and 4096; at bucket 512 also the l_inf norms (alone and fused
with the quantizer) and one norm per tensor (``dq_tensor_norms``).  Every kernel is timed alone with CUDA events
(3 warm-up launches, median of 8-20), over rotating inputs that together exceed the L2,
and once more as a train of launches between two events (the sustained rate: launch latency
overlaps the previous launch).  Each row gives both times, GB/s of algorithmic bytes (norms 4, quantizers 4 + b/8 per
element and worker, average M b/8 + 4 per element) and GB/s of fp32 gradient (4 M d).
Points below a few hundred microseconds are bound by the host's launch cost, not by the GPU.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import dq
from .pipeline import Round


def _time(fn, reps):
    for i in range(3):
        fn(i)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for i in range(reps):
        evs[i][0].record()
        fn(i)
        evs[i][1].record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    # sustained: the same launches back to back between two events
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return ts[len(ts) // 2] * 1e3, ts[0] * 1e3, a.elapsed_time(b) * 1e3 / reps


def run(quick: bool = False):
    rows = []
    points = [(1 << e, 1) for e in (20, 22, 24, 26, 28, 30)] + [(1 << 26, 32)]
    for d, M in points:
        for bucket in (128, 512, 4096):
            if quick and bucket != 512:
                continue
            bits = list(range(1, 17)) if (bucket == 512 and not quick) else [2, 4, 8, 16]
            rnd = Round([d], bucket, M)
            D32 = rnd.layout.D32
            step_bytes = 4 * M * D32
            nbuf = max(1, min(8, (256 << 20) // step_bytes + 1, (24 << 30) // step_bytes))
            gs = [torch.randn((M, D32), device="cuda") for _ in range(nbuf)]
            reps = 20 if d * M <= (1 << 28) else 8

            def add(kernel, b, med, best, train, nbytes):
                rows.append({"kernel": kernel, "d": d, "M": M, "bucket": bucket, "b": b, "med_us": med, "best_us": best,
                             "train_us": train, "gbs": nbytes / med / 1e3, "train_gbs": nbytes / train / 1e3,
                             "grad_gbs": 4.0 * M * d / med / 1e3})

            add("bucket_norms", 0, *_time(lambda i: rnd.norms_(gs[i % nbuf]), reps), 4.0 * M * D32)
            for b in bits:
                rnd.bits_(dq.Rule.fixed(b))
                add("quantize_pack", b, *_time(lambda i: rnd.quantize_(gs[i % nbuf], 1, i), reps), (4.0 + b / 8.0) * M * D32)
                add("norms_quantize_pack", b, *_time(lambda i: rnd.norms_quantize_(gs[i % nbuf], 1, i), reps),
                    (4.0 + b / 8.0) * M * D32)
                add("unpack_dequant_average", b, *_time(lambda i: rnd.average_(), reps), (M * b / 8.0 + 4.0) * D32)
            torch.cuda.synchronize()
            if rnd.read_status() != 0:
                raise RuntimeError("device status %d" % rnd.read_status())
            del rnd
            if bucket == 512:
                # the other members of the norm family on the same inputs: l_inf buckets, one norm per tensor
                for norm, tag in ((dq.NORM_LINF, "_linf"),):
                    alt = Round([d], bucket, M, norm=norm)
                    add("bucket_norms" + tag, 0, *_time(lambda i: alt.norms_(gs[i % nbuf]), reps), 4.0 * M * D32)
                    for b in (2, 4, 8, 16):
                        alt.bits_(dq.Rule.fixed(b))
                        add("norms_quantize_pack" + tag, b, *_time(lambda i: alt.norms_quantize_(gs[i % nbuf], 1, i), reps),
                            (4.0 + b / 8.0) * M * D32)
                    del alt
                for norm, tag in ((dq.NORM_L2, ""), (dq.NORM_LINF, "_linf")):
                    whole = Round([d], dq.BUCKET_WHOLE_TENSOR, M, max_bits=1, norm=norm)
                    add("tensor_norms" + tag, 0, *_time(lambda i: whole.norms_(gs[i % nbuf]), reps), 4.0 * M * D32)
                    torch.cuda.synchronize()
                    if whole.read_status() != 0:
                        raise RuntimeError("device status %d" % whole.read_status())
                    del whole
            del gs
            torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="bucket 512 and four bit widths only")
    ap.add_argument("--out", default=None, help="write the rows as JSON to this file")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device (there is no CPU fallback)")
    rows = run(args.quick)
    if args.out:
        with open(args.out, "w") as fh:
            json.dump(rows, fh)
    for r in rows:
        sys.stdout.write("%-24s d=2^%-2d M=%-2d bucket=%-4d b=%-2d %9.1f us %7.0f GB/s | in a train %9.1f us %7.0f GB/s | "
                         "gradient %7.0f GB/s\n" % (r["kernel"], r["d"].bit_length() - 1, r["M"], r["bucket"], r["b"],
                                                    r["med_us"], r["gbs"], r["train_us"], r["train_gbs"], r["grad_gbs"]))


if __name__ == "__main__":
    main()
