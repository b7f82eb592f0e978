"""Throughput of the path on the model-shaped workloads, one table row per configuration and bit width.

    python -m paper_2107_14575_b200.config_times [--out times.json]

Configurations: the flat d = 2^20, M = 4 case, the ResNet-18 shape (M = 8, bucket 512), the VGG-16
shape (M = 16, bucket 2048, 1% outliers) and the text-classifier shape (M = 16, bucket 1024, 97% of
the embedding rows zero), with the value distributions of ``workloads``.  For each of them and for
b in {2, 4, 6, 8}: the fused norms+quantize+pack call, the average, and the two alternating as a step
does, each as a train of launches between two CUDA events over rotating input sets, plus the b the
paper's rule picks at the first and last step of the configuration's schedule.  Reported: microseconds,
GB/s of fp32 gradient (4 M d per step) and GB/s of algorithmic bytes (4 + b/8 per element and worker
for the quantizer, M b/8 + 4 per element for the average).
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import dq, workloads
from .pipeline import Round


def _train(fn, reps):
    for i in range(3):
        fn(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / reps


def run():
    rows = []
    configs = [workloads.config_flat(), workloads.config_resnet18(), workloads.config_vgg16(), workloads.config_text()]
    for w in configs:
        rnd = Round(w.segments, w.bucket, w.M)
        L = rnd.layout
        D32, M = L.D32, w.M
        nset = max(2, min(6, (512 << 20) // (4 * M * D32) + 1))          # rotating inputs, together beyond the L2
        pool = [torch.from_numpy(workloads.make_grads(w, L.offsets, D32, step=t)).cuda() for t in range(nset)]
        # b of the paper's rule at the ends of the schedule (x(t = 0) calibrated to x0, constant norms)
        rnd.norms_(pool[0])
        G2 = float((rnd.norms.double() ** 2).sum().item() / M)
        sched = None
        if w.T > 1 and G2 > 0:
            eps_hat = w.T * w.alpha ** (w.T - 1) * G2 / w.x0 ** 2
            sched = []
            for t in (0, w.T - 1):
                rnd.bits_(dq.Rule.dynamic(w.T, t, eps_hat, w.alpha))
                sched.append(rnd.bits())
        reps = 200 if M * D32 < (1 << 26) else 60
        for b in (2, 4, 6, 8):
            rnd.bits_(dq.Rule.fixed(b))
            t_q = _train(lambda i: rnd.norms_quantize_(pool[i % nset], 1, i), reps)
            t_a = _train(lambda i: rnd.average_(), reps)

            def pair(i):
                rnd.norms_quantize_(pool[i % nset], 1, i)
                rnd.average_()
            t_p = _train(pair, reps)
            rows.append({"config": w.name, "d": w.d, "M": M, "bucket": w.bucket, "b": b, "rule_b_first_last": sched,
                         "quantize_us": t_q, "average_us": t_a, "step_us": t_p,
                         "quantize_alg_gbs": (4.0 + b / 8.0) * M * D32 / t_q / 1e3,
                         "average_alg_gbs": (M * b / 8.0 + 4.0) * D32 / t_a / 1e3,
                         "step_grad_gbs": 4.0 * M * w.d / t_p / 1e3})
        torch.cuda.synchronize()
        if rnd.read_status() != 0:
            raise RuntimeError("device status %d" % rnd.read_status())
        del pool, rnd
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None, help="write the rows as JSON to this file")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("this needs a CUDA device (there is no CPU fallback)")
    rows = run()
    if args.out:
        with open(args.out, "w") as fh:
            json.dump(rows, fh)
    for r in rows:
        sys.stdout.write("%-9s d=%-9d M=%-2d bucket=%-4d b=%d rule b %s | quantize %7.1f us %6.0f GB/s | average %7.1f us "
                         "%6.0f GB/s | step %7.1f us %6.0f GB/s of gradient\n"
                         % (r["config"], r["d"], r["M"], r["bucket"], r["b"], r["rule_b_first_last"], r["quantize_us"],
                            r["quantize_alg_gbs"], r["average_us"], r["average_alg_gbs"], r["step_us"], r["step_grad_gbs"]))


if __name__ == "__main__":
    main()
