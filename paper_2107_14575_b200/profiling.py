"""Profiling helpers of the library: a small driver that launches ONE kernel on a stated case (the
command an ``ncu`` capture wraps), and the code that turns a capture into the short summaries and
counters kept under ``profiles/``.

    # launch a kernel a few times (bounded case; this is what ncu wraps)
    python -m paper_2107_14575_b200.profiling run --kernel unpack_dequant_average --log2d 24 --M 32 --b 4 --n 3

    # summarise a capture: ncu -i REP --page raw --csv > capture.csv, then
    python -m paper_2107_14575_b200.profiling summarize capture.csv --kernel unpack_dequant_average \
        --log2d 24 --M 32 --b 4 --command "<the full ncu command>" [--update-counters]

    # the per-b table of a bench line as markdown
    python -m paper_2107_14575_b200.profiling table bench_line.json > profiles/bench_per_b.md

    # per kernel launches / time / share from an `ncu --metrics gpu__time_duration.sum --csv --log-file` run
    python -m paper_2107_14575_b200.profiling launches launches.csv --command "<the ncu command>" > profiles/bench_launch_list.md

``run`` needs a GPU; the other two run anywhere.  Nothing here is on the product path.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)

KERNELS = {
    # key -> (substring of the kernel's name in a capture, source files that decide its counters)
    "norms_quantize_pack": ("norms_quantize_pack_", ["dq_fused.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"]),
    "quantize_pack": ("quantize_pack_kernel", ["dq_quantize.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"]),
    "bucket_norms": ("bucket_norms_", ["dq_norms.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"]),
    "unpack_dequant_average": ("unpack_average_kernel", ["dq_unpack.cu", "dq_device.cuh", "dq_tma.cuh", "dq_common.cuh"]),
}


def sources_digest(key: str) -> str:
    h = hashlib.sha256()
    for name in KERNELS[key][1]:
        with open(os.path.join(PKG, "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def algorithmic_bytes(key: str, d32: int, M: int, b: int) -> float:
    """Bytes the method itself must move per launch (norms traffic left out: below 1 %)."""
    if key == "bucket_norms":
        return 4.0 * M * d32
    if key in ("quantize_pack", "norms_quantize_pack"):
        return (4.0 + b / 8.0) * M * d32
    return (M * b / 8.0 + 4.0) * d32


def groups(key: str, d32: int, M: int) -> int:
    """Units of the per-group counters: 32-element groups per launch (for the average a group is 32
    output elements, i.e. M x 32 codes)."""
    return d32 // 32 if key == "unpack_dequant_average" else M * d32 // 32


# ------------------------------------------------------------------ run

def cmd_run(a) -> None:
    import torch

    from . import dq
    from .pipeline import Round
    if not torch.cuda.is_available():
        raise RuntimeError("`run` needs a CUDA device (there is no CPU fallback)")
    rnd = Round([1 << a.log2d], a.bucket, a.M)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2107)
    g = torch.randn((a.M, rnd.layout.D32), generator=gen, device="cuda")
    rnd.bits_(dq.Rule.fixed(a.b))
    rnd.norms_quantize_(g, 2107, 0)                  # norms and words for the kernels that read them
    fn = {"norms_quantize_pack": lambda i: rnd.norms_quantize_(g, 2107, i),
          "quantize_pack": lambda i: rnd.quantize_(g, 2107, i),
          "bucket_norms": lambda i: rnd.norms_(g),
          "unpack_dequant_average": lambda i: rnd.average_()}[a.kernel]
    torch.cuda.synchronize()
    for i in range(a.n):
        fn(i)
    torch.cuda.synchronize()
    st = rnd.read_status()
    print("kernel %s d=2^%d M=%d bucket=%d b=%d launches=%d status=%d" % (a.kernel, a.log2d, a.M, a.bucket, a.b, a.n, st))
    if st:
        raise SystemExit(1)


# ------------------------------------------------------------ summarize

FIGURES = [
    ("duration", "gpu__time_duration.sum"), ("grid", "launch__grid_size"), ("block", "launch__block_size"),
    ("registers/thread", "launch__registers_per_thread"), ("dynamic smem/block", "launch__shared_mem_per_block_dynamic"),
    ("occupancy limit (registers), CTAs/SM", "launch__occupancy_limit_registers"),
    ("occupancy limit (smem), CTAs/SM", "launch__occupancy_limit_shared_mem"),
    ("DRAM read", "dram__bytes_read.sum"), ("DRAM write", "dram__bytes_write.sum"),
    ("DRAM throughput % of peak", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed"),
    ("L2 hit rate %", "lts__t_sector_hit_rate.pct"),
    ("achieved occupancy %", "sm__warps_active.avg.pct_of_peak_sustained_active"),
    ("warp instructions", "smsp__inst_executed.sum"),
    ("issue slots busy per cycle (per scheduler)", "smsp__issue_active.avg.per_cycle_active"),
    ("eligible warps per cycle (per scheduler)", "smsp__warps_eligible.avg.per_cycle_active"),
    ("ALU pipe active %", "sm__pipe_alu_cycles_active.avg.pct_of_peak_sustained_active"),
    ("FMA pipe active %", "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_active"),
    ("LSU pipe instructions %", "sm__inst_executed_pipe_lsu.avg.pct_of_peak_sustained_active"),
    ("shared-memory bank conflicts", "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum"),
] + [("stall %s / issue" % n, "smsp__average_warps_issue_stalled_%s_per_issue_active.ratio" % k) for n, k in (
    ("long scoreboard", "long_scoreboard"), ("short scoreboard", "short_scoreboard"),
    ("math pipe throttle", "math_pipe_throttle"), ("dispatch", "dispatch_stall"), ("wait", "wait"),
    ("barrier", "barrier"), ("not selected", "not_selected"), ("branch resolving", "branch_resolving"),
    ("no instruction", "no_instruction"))]

SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6}


def _peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured copy bandwidth"
    return 6650.0, "fallback copy bandwidth"


def cmd_summarize(a) -> None:
    with open(a.csv, newline="") as fh:
        rows = [r for r in csv.reader(fh) if r]
    start = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    hdr, units, body = rows[start], rows[start + 1], rows[start + 2:]
    ki = hdr.index("Kernel Name")
    pattern = KERNELS[a.kernel][0]
    sel = [r for r in body if pattern in r[ki]]
    if not sel:
        raise SystemExit("no launch of %s in %s" % (pattern, a.csv))

    def col(name):
        i = hdr.index(name)
        return [float(r[i].replace(",", "")) for r in sel], units[i]

    lines = []
    for label, metric in FIGURES:
        if metric not in hdr:
            continue
        v, u = col(metric)
        mean = sum(v) / len(v)
        rng = "" if max(v) == min(v) else " (%.4g..%.4g)" % (min(v), max(v))
        lines.append("| %s | %.4g %s%s |" % (label, mean, u, rng))
    if "sm__cycles_active.avg" in hdr and "sm__cycles_elapsed.max" in hdr:
        act, _ = col("sm__cycles_active.avg")
        ela, _ = col("sm__cycles_elapsed.max")
        lines.append("| SM active cycles / elapsed cycles | %.3f |" % (sum(x / y for x, y in zip(act, ela)) / len(act)))

    def total(name):
        v, u = col(name)
        return sum(v) / len(v) * SCALE[u]

    d32 = 1 << a.log2d
    alg = algorithmic_bytes(a.kernel, d32, a.M, a.b)
    n_groups = groups(a.kernel, d32, a.M)
    dur_us = total("gpu__time_duration.sum")
    traffic = total("dram__bytes_read.sum") + total("dram__bytes_write.sum") if "dram__bytes_read.sum" in hdr else None
    inst = total_plain(col, "smsp__inst_executed.sum") if "smsp__inst_executed.sum" in hdr else None
    peak, peak_name = _peak()
    gbs = alg / (dur_us * 1e-6) / 1e9
    out = ["# %s: d = 2^%d, M = %d, bucket %d, b = %d" % (sel[0][ki].split("(")[0], a.log2d, a.M, a.bucket, a.b), "",
           "Flat N(0,1) gradient of 2^%d fp32 elements per worker, M = %d workers, bucket %d, l2 norms, b = %d."
           % (a.log2d, a.M, a.bucket, a.b), "",
           "Command (one B200; the same command line had exited 0 without ncu directly before):", "", "```",
           a.command, "```", "",
           "Read back with `ncu -i <report> --page raw --csv`; %d captured launch(es), the table gives their mean "
           "(min..max where they differ)." % len(sel), "", "| figure | value |", "|---|---|"] + lines + [""]
    out.append("Algorithmic bytes per launch: %.1f MB (%s)." % (alg / 1e6, {
        "bucket_norms": "4 B x M x d read", "quantize_pack": "(4 + b/8) B x M x d",
        "norms_quantize_pack": "(4 + b/8) B x M x d", "unpack_dequant_average": "(M b/8 + 4) B x d"}[a.kernel]))
    if traffic is not None:
        out.append("DRAM traffic per launch (read + write): %.1f MB (%.2f x algorithmic; ncu flushes the caches before "
                   "each replayed launch, and output lines still dirty in L2 at the kernel's end are not counted)."
                   % (traffic / 1e6, traffic / alg))
    if inst is not None:
        out.append("Warp instructions per 32-element group: %.1f (%d groups per launch)." % (inst / n_groups, n_groups))
    out.append("Under ncu (serialised, cold caches) the launch took %.1f us = %.0f GB/s of algorithmic bytes, %.1f%% of "
               "the %s %.0f GB/s; bench.py's live CUDA-event figure is the one that counts." %
               (dur_us, gbs, 100 * gbs / peak, peak_name, peak))
    if a.note:
        out += ["", a.note]
    name = a.out or os.path.join(ROOT, "profiles", "%s_flat_d%d_m%d_b%d.md" % (pattern.rstrip("_"), a.log2d, a.M, a.b))
    if not a.counters_only:
        with open(name, "w") as fh:
            fh.write("\n".join(out) + "\n")
        print("wrote", name)
    if a.update_counters:
        path = os.path.join(ROOT, "profiles", "counters.json")
        rec = {}
        if os.path.exists(path):
            with open(path) as fh:
                rec = json.load(fh)
        digest = sources_digest(a.kernel)
        cur = rec.get(a.kernel)
        if not cur or cur.get("sha256") != digest:
            cur = {"sha256": digest, "sources": KERNELS[a.kernel][1], "warp_instructions_per_group": {},
                   "dram_bytes_per_group": {}, "cases": {}}
        if inst is not None:
            cur["warp_instructions_per_group"][str(a.b)] = round(inst / n_groups, 2)
        if traffic is not None:
            cur["dram_bytes_per_group"][str(a.b)] = round(traffic / n_groups, 2)
        cur["cases"][str(a.b)] = {"log2d": a.log2d, "M": a.M, "bucket": a.bucket, "command": a.command}
        if not a.counters_only:
            cur["cases"][str(a.b)]["summary"] = os.path.relpath(name, ROOT)
        rec[a.kernel] = cur
        with open(path, "w") as fh:
            json.dump(rec, fh, indent=1, sort_keys=True)
        print("updated", path)


def total_plain(col, name):
    v, _ = col(name)
    return sum(v) / len(v)


# ---------------------------------------------------------------- table

def cmd_table(a) -> None:
    with open(a.json) as fh:
        text = fh.read()
    line = json.loads(text[text.index("{"):])
    per_b = line["per_b"]
    print("# Per-b figures of the bench workload\n")
    print(line["config"]["workload"] + ".  From one `python bench.py --steps %d --warmup %d` line; `train` = launches "
          "back to back between two CUDA events, `single` = one launch between its own events; fractions are of the "
          "copy bandwidth %.0f GB/s (%s).  `SM MHz` is the median NVML sample during the train: these trains run into "
          "the 1000 W power cap (`sw_power_cap`), which pulls the clock below its 1965 MHz maximum, and the "
          "instruction-bound kernels slow down with it.\n" % (line["steps"], line["warmup"], line["roofline"]["hbm"]["achieved_gbs"] /
                                              max(line["roofline"]["hbm"]["frac_of_measured"], 1e-9),
                                              line["roofline"].get("peak_source", "")))
    names = ("quantize_pack", "norms_quantize_pack", "unpack_dequant_average")
    print("| b | " + " | ".join("%s train ms / GB/s / frac / bound / SM MHz | single ms / frac" % n for n in names) +
          " | step ms | step GB/s of gradient |")
    print("|---|" + "---|---|" * len(names) + "---|---|")
    for b in sorted(per_b, key=int):
        r = per_b[b]
        cells = []
        for n in names:
            k = r[n]
            cells.append("%.3f / %.0f / %.3f / %s / %s | %.3f / %.3f" % (k["ms"], k["achieved_gbs"], k["frac_of_measured"],
                                                                        k["bound"], ("%.0f" % k["sm_mhz"]) if k.get("sm_mhz") else "-",
                                                                        k["single_launch_ms"],
                                                                        k["single_launch_frac_of_measured"]))
        print("| %s | %s | %.3f | %.0f |" % (b, " | ".join(cells), r["step_ms"], r["step_gradient_gbs"]))
    if line.get("with_parameter_update"):
        u = line["with_parameter_update"]
        k = u["unpack_average_update"]
        print("\nThe headline step with the parameter update of Eq. 2 applied by the averaging kernel: %.3f ms per step "
              "(%.0f GB/s of gradient); the update kernel %.3f ms = %.0f GB/s of its algorithmic bytes "
              "((M b/8 + 8) B per element), %.3f of the copy bandwidth." % (u["ms_per_step"], u["value"], k["ms"],
                                                                          k["achieved_gbs"], k["frac_of_measured"]))
    if line.get("size_sweep"):
        print("\n## Other sizes and bucket lengths of the bandwidth sweep\n")
        print("Trains of launches; cases whose buffers would fit in the L2 rotate through `sets` sets of buffers.  "
              "Cells: ms per launch / GB/s of algorithmic bytes / fraction of the copy bandwidth.\n")
        bs = sorted(line["size_sweep"][0]["b"], key=int)
        print("| M | d | bucket | MB/launch | sets | " + " | ".join("fused b=%s | average b=%s" % (b, b) for b in bs) + " |")
        print("|---|---|---|---|---|" + "---|---|" * len(bs))
        for pt in line["size_sweep"]:
            cells = []
            for b in bs:
                for n in ("norms_quantize_pack", "unpack_dequant_average"):
                    k = pt["b"][b][n]
                    cells.append("%.4f / %.0f / %.3f" % (k["ms"], k["achieved_gbs"], k["frac_of_measured"]))
            print("| %d | 2^%d | %d | %d | %d | %s |" % (pt["M"], pt["d"].bit_length() - 1, pt["bucket"], pt["mb_per_launch"],
                                                      pt["buffer_sets"], " | ".join(cells)))
    if line.get("model_workloads"):
        print("\n## Model-shaped workloads (Algorithm-1 order, dynamic b)\n")
        print("`single` = one launch between its own pair of events (the bracket leaves the GPU idle for some microseconds "
              "around the launch); `train` = launches back to back, rotating through three sets of buffers.\n")
        print("| workload | MB/step | ms/step | GB/s of gradient | b first..last | fused single ms (frac) | fused train ms (frac) "
              "| average single ms (frac) | average train ms (frac) |")
        print("|---|---|---|---|---|---|---|---|---|")
        for name, w in line["model_workloads"].items():
            f, v = w["norms_quantize_pack"], w["unpack_dequant_average"]
            print("| %s | %d | %.4f | %.0f | %s | %.4f (%.3f) | %.4f (%.3f) | %.4f (%.3f) | %.4f (%.3f) |" % (
                w["workload"], w["mb_per_step"], w["ms_per_step"], w["value"], w["bits_first_last"],
                f["ms"], f["frac_of_measured"], f.get("train_ms", float("nan")), f.get("train_frac_of_measured", float("nan")),
                v["ms"], v["frac_of_measured"], v.get("train_ms", float("nan")), v.get("train_frac_of_measured", float("nan"))))


def cmd_launches(a) -> None:
    """Per kernel: launches, total time and share, from the CSV log of an
    ``ncu --metrics gpu__time_duration.sum --csv --log-file`` run (one row per launch)."""
    with open(a.csv, newline="") as fh:
        rows = [r for r in csv.reader(l for l in fh if not l.startswith("==")) if r]
    hdr, body = rows[0], rows[1:]
    ki, vi, ui = hdr.index("Kernel Name"), hdr.index("Metric Value"), hdr.index("Metric Unit")
    per = {}
    for r in body:
        full = r[ki].replace("(anonymous namespace)::", "").replace("<unnamed>::", "")
        name = full.split("(")[0].split("<")[0].replace("void ", "").strip().split("::")[-1]
        t = float(r[vi].replace(",", "")) * {"ns": 1e-3, "us": 1.0, "ms": 1e3}[r[ui]]
        n, tot = per.get(name, (0, 0.0))
        per[name] = (n + 1, tot + t)
    library = ("norms_quantize_pack", "quantize_pack_kernel", "bucket_norms", "unpack_average_kernel", "tensor_norms_join",
               "norm_square_partials", "apply_rule")
    ours = {k: v for k, v in per.items() if any(k.startswith(p) for p in library)}
    total_ours = sum(t for _, t in ours.values())
    total_all = sum(t for _, t in per.values())
    print("# Launch list of the bench command\n")
    print("Command (one B200; the same command line had exited 0 without ncu directly before):\n\n```\n%s\n```\n" % a.command)
    print("Every launch of the process with its device time (ncu serialises the launches and flushes the caches, so the "
          "absolute times are cold-cache figures: the SHARES are what the bench line's must agree with).  %d launches, "
          "%.1f us in the library's kernels, %.1f us in all kernels (the rest is torch: the generator, fills, copies).\n"
          % (len(body), total_ours, total_all))
    print("| kernel | launches | total us | mean us | share of the library's kernels |")
    print("|---|---|---|---|---|")
    for k, (n, t) in sorted(per.items(), key=lambda kv: -kv[1][1]):
        share = "%.3f" % (t / total_ours) if k in ours else "(torch)"
        print("| %s | %d | %.1f | %.1f | %s |" % (k, n, t, t / n, share))
    if a.note:
        print("\n" + a.note)


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(prog="python -m paper_2107_14575_b200.profiling")
    sub = ap.add_subparsers(dest="cmd", required=True)

    def case(p):
        p.add_argument("--kernel", required=True, choices=sorted(KERNELS))
        p.add_argument("--log2d", type=int, default=24)
        p.add_argument("--M", type=int, default=32)
        p.add_argument("--bucket", type=int, default=512)
        p.add_argument("--b", type=int, default=4)

    r = sub.add_parser("run")
    case(r)
    r.add_argument("--n", type=int, default=3)
    s = sub.add_parser("summarize")
    s.add_argument("csv")
    case(s)
    s.add_argument("--command", required=True)
    s.add_argument("--note", default="")
    s.add_argument("--out", default=None)
    s.add_argument("--update-counters", action="store_true")
    s.add_argument("--counters-only", action="store_true", help="no summary file, only profiles/counters.json")
    t = sub.add_parser("table")
    t.add_argument("json")
    l = sub.add_parser("launches")
    l.add_argument("csv")
    l.add_argument("--command", required=True)
    l.add_argument("--note", default="")
    a = ap.parse_args(argv)
    {"run": cmd_run, "summarize": cmd_summarize, "table": cmd_table, "launches": cmd_launches}[a.cmd](a)


if __name__ == "__main__":
    main()
