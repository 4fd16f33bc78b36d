"""Where the Newton-Schulz kernel's cycles go: runs the Newton-Schulz phase of a synthetic parameter set through the
profiling build of the library (libmona_trace.so, compiled with -DMONA_TRACE) and prints what every role of the kernel
waited for, and the MMA issuer's cycles per k-slice for every kind of tile.

    python -m paper_2605_26842_b200.trace_report --config 3 --layers 2 [--bucket wide|tall|square] [--json]

The profiling build computes exactly what the ordinary build computes (the step's status and launch count are checked
here, parity is a test); its clock reads make the kernel a few per cent slower, so absolute times come from bench.py
and only the split comes from here.  Needs a B200; there is no CPU path."""
from __future__ import annotations

import argparse
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
KINDS = ["XXt off-diagonal", "XXt diagonal", "bA+cA^2+aI off-diagonal", "bA+cA^2+aI diagonal", "B'X macro-tile", "B'X single tile"]
# 256 x 256 x 64 MMAs per k-slice of a tile of each kind, at 512 SM cycles each when the tensor pipe never idles
TILES_PER_KSLICE = [1, 1, 1, 1, 2, 1]
ROLE_WAITS = [("producer", 3, [(1, "free operand slabs"), (2, "next item")]),
              ("MMA issuer", 5, [(4, "next item")]),
              ("scheduler", 8, [(6, "dependency (previous GEMM of the matrix)"), (7, "free ring slot (it is ahead)")]),
              ("epilogue warps (x8)", 12, [(9, "finished accumulator"), (10, "staging buffer"), (11, "next item")]),
              ("store warp", 14, [(13, "staged phase")])]


def collect(config: int, layers: int, bucket: str | None, steps: int, delay: int | None):
    import torch

    import paper_2605_26842_b200 as pkg
    from paper_2605_26842_b200 import binding, build, synth

    # the binding loads its library on first use: point it at the profiling build unless the caller chose one
    if not os.environ.get("MONA_LIBRARY"):
        binding._LIB_PATH = build.build(trace=True)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = synth.workload(config, layers)
    if bucket:
        # keep only the matrices of one aspect (wide and tall experts, square attention weights), all layers of them
        pick = {"wide": lambda s: s.rows < s.cols, "tall": lambda s: s.rows > s.cols, "square": lambda s: s.rows == s.cols}[bucket]
        wl.specs = [s for s in wl.specs if pick(s)]
        if not wl.specs:
            raise SystemExit(f"config {config} has no {bucket} matrices")
    params = synth.init_params(wl, dev)
    gp = synth.GradientProcess(wl, dev, keep_fp32_shadow=False)
    options = pkg.default_options(**({"ns_delay": delay} if delay is not None else {}))
    opt = pkg.MonaOptimizer(params, options=options)
    hp = pkg.default_hparams(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha)
    gp.next()
    for _ in range(2):                       # whole steps: state warm, clocks settled
        opt.step(hp, params, gp.grads)
    torch.cuda.synchronize()
    binding.trace_read(reset=True, rows=0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        opt.step_ex(hp, params, gp.grads, None, 2)      # phase mask 2: the Newton-Schulz phase alone
    e1.record()
    torch.cuda.synchronize()
    launches = opt.last_launch_count()
    rows = binding.trace_read(reset=True)
    status, bad = opt.poll_status()
    executed, _ = opt.last_ns_flops()
    ms = e0.elapsed_time(e1) / steps
    opt.close()
    return {"workload": wl.name, "bucket": bucket or "all", "matrices": sum(s.batch for s in wl.specs), "steps": steps, "status": status,
            "launches_per_pass": launches, "ns_pass_ms": ms, "tflops_executed": executed / (ms * 1e-3) / 1e12, "rows": rows}


def summarise(res):
    rows = [r for r in res["rows"] if r[0] > 0]          # CTAs that ran
    lead, peer = rows[0::2], rows[1::2]
    mean = lambda rs, k: sum(r[k] for r in rs) / max(1, len(rs))
    out = {k: res[k] for k in res if k != "rows"}
    out["ctas"] = len(rows)
    out["kernel_cycles_per_cta"] = mean(rows, 0)
    out["items"] = sum(r[15] for r in lead)
    roles = {}
    for name, total, waits in ROLE_WAITS:
        group = lead if name in ("MMA issuer", "scheduler") else rows
        t = mean(group, total)
        roles[name] = {"cycles": t, "waits_pct": {label: 100.0 * mean(group, k) / t if t else 0.0 for k, label in waits}}
    out["roles"] = roles
    tiles = {}
    for kind, label in enumerate(KINDS):
        b = 16 + 4 * kind
        cyc, ks, wf, wa = (sum(r[b + j] for r in lead) for j in range(4))
        if ks:
            ideal = 512.0 * TILES_PER_KSLICE[kind]
            tiles[label] = {"k_slices": ks, "cycles_per_k_slice": cyc / ks, "waiting_operands": wf / ks, "waiting_accumulator": wa / ks,
                            "issuing": (cyc - wf - wa) / ks, "tensor_peak_cycles": ideal, "share_of_issuer_time_pct": 0.0}
    total = sum(v["cycles_per_k_slice"] * v["k_slices"] for v in tiles.values())
    for v in tiles.values():
        v["share_of_issuer_time_pct"] = 100.0 * v["cycles_per_k_slice"] * v["k_slices"] / total
    out["tiles"] = tiles
    epi = {}
    for kind, label in enumerate(KINDS):
        b = 40 + 4 * kind
        cyc, n, wa, ws = (sum(r[b + j] for r in rows) for j in range(4))
        if n:
            epi[label] = {"items_per_warp": n / 8, "cycles_per_item": cyc / n, "waiting_accumulator": wa / n, "waiting_staging": ws / n,
                          "working": (cyc - wa - ws) / n}
    out["epilogue"] = epi
    issuer = mean(lead, 5)
    out["mma_issuer_inside_tiles_pct"] = 100.0 * total / len(lead) / issuer if issuer else 0.0
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--bucket", choices=["wide", "tall", "square"], default=None)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--ns-delay", type=int, default=None)
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    s = summarise(collect(a.config, a.layers, a.bucket, a.steps, a.ns_delay))
    if a.json:
        print(json.dumps(s))
        return 0
    print(f"{s['workload']} ({s['bucket']}, {s['matrices']} matrices): Newton-Schulz pass {s['ns_pass_ms']:.3f} ms, "
          f"{s['tflops_executed']:.0f} TFLOP/s executed (profiling build), {s['launches_per_pass']} launches, status {s['status']}, "
          f"{s['ctas']} CTAs, {s['items']} work items in {s['steps']} passes")
    for name, r in s["roles"].items():
        waits = ";  ".join(f"{label} {pct:.1f} %" for label, pct in r["waits_pct"].items())
        print(f"  {name:<22s} waits, % of its time:  {waits}")
    print(f"  MMA issuer inside tiles: {s['mma_issuer_inside_tiles_pct']:.1f} % of its time (the rest: between tiles and waiting for items)")
    print("  per k-slice (64 of the inner dimension) of the MMA issuer, SM cycles:")
    for label, v in s["tiles"].items():
        print(f"    {label:<26s} {v['k_slices']:>9d} k-slices  {v['cycles_per_k_slice']:7.1f} cycles "
              f"(tensor peak {v['tensor_peak_cycles']:.0f}) = issuing {v['issuing']:6.1f} + operands {v['waiting_operands']:6.1f} "
              f"+ accumulator {v['waiting_accumulator']:6.1f};  {v['share_of_issuer_time_pct']:4.1f} % of the time inside tiles")
    print("  per work item of an epilogue warp, SM cycles (a CTA's 128 rows of the tile or macro-tile):")
    for label, v in s["epilogue"].items():
        print(f"    {label:<26s} {v['cycles_per_item']:8.0f} cycles = working {v['working']:6.0f} + accumulator {v['waiting_accumulator']:6.0f} "
              f"+ staging buffer {v['waiting_staging']:6.0f}")
    return 0 if s["status"] == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
