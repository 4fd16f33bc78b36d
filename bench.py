#!/usr/bin/env python
"""Benchmark of the MONA optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--layers L] [--impl reference]

A step is one pass of the whole hot path (fused prologue, Newton-Schulz, parameter update) over every
matrix of a synthetic parameter set (see paper_2605_26842_b200/synth.py).  Prints ONE JSON line.

Timing: CUDA events on the launching stream around each mona_step; between timed steps the gradient
buffers advance one step of the AR(1) process and a buffer larger than L2 is rewritten (both untimed).
The per-phase figures (prologue GB/s, Newton-Schulz TFLOP/s, update GB/s) come from extra passes that
run one phase alone through mona_step_ex's phase mask.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mona_optimizer_steps_per_s"
UNIT = "steps/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the Newton-Schulz kernel from the ncu capture
# summarised in profiles/ns_chunk_kernel_moe7b_1L.md: the launch over a 93-matrix 768x2048 chunk, the launch shape that
# makes up most of the default workload (40 of its 56 launches per step are of this shape or its tall twin).  Valid only
# for the kernel source the counters were taken with (hash of ns_tc.cu + ns_tc.cuh).
NCU_TRAFFIC = {"source_sha256_16": "d420627d482a0ead", "bytes_per_launch": 6.690e9,
               "unit": "DRAM bytes of one launch over a 93-matrix 768x2048 chunk (ncu; 2.153 TFLOP executed in that launch)"}


def kernel_traffic():
    """DRAM bytes per GEMM launch from the committed ncu capture, or None once the kernel source has changed."""
    import hashlib
    try:
        src = b"".join(open(os.path.join(ROOT, "paper_2605_26842_b200", "csrc", f), "rb").read() for f in ("ns_tc.cu", "ns_tc.cuh"))
    except OSError:
        return None
    return NCU_TRAFFIC["bytes_per_launch"] if hashlib.sha256(src).hexdigest()[:16] == NCU_TRAFFIC["source_sha256_16"] else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


_POWER_FIELD = None


def power_field(index: int) -> str:
    """`power.draw.instant` where this driver's nvidia-smi knows it (power.draw is a one-second average), else `power.draw`."""
    global _POWER_FIELD
    if _POWER_FIELD is None:
        _POWER_FIELD = "power.draw"
        try:
            r = subprocess.run(["nvidia-smi", f"--id={index}", "--query-gpu=power.draw.instant", "--format=csv,noheader,nounits"],
                               capture_output=True, text=True, timeout=20)
            if r.returncode == 0:
                float(r.stdout.strip().splitlines()[0])
                _POWER_FIELD = "power.draw.instant"
        except Exception:
            pass
    return _POWER_FIELD


class ClockSampler:
    """Samples SM clock, board power and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,{power},clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.Q = ClockSampler.Q.format(power=power_field(index))
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ts, row in self.rows:
            if t0 is not None and not (t0 <= ts <= t1 + 0.15):
                continue
            f = [x.strip() for x in row.split(",")]
            if len(f) < 7:
                continue
            try:
                vals = (float(f[0]), float(f[1]), float(f[2]))
            except ValueError:
                continue
            sm.append(vals[0]); mx.append(vals[1]); power.append(vals[2])
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "power_w_median": statistics.median(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def sustained(torch, dev, index, fn, flops_per_call, seconds=2.5):
    """Runs fn() back to back for about `seconds` with clock and power sampling: sustained TFLOP/s, median watts and
    clock over the window (its first 0.5 s left out of the medians), and joules per TFLOP."""
    fn()
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(index)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    calls = 0
    e0.record()
    while time.time() - t0 < seconds:
        fn()
        calls += 1
        if calls % 4 == 0:
            torch.cuda.synchronize(dev)      # keep the host a few calls ahead at most, so the window is what was asked for
    e1.record()
    torch.cuda.synchronize(dev)
    t1 = time.time()
    c = sampler.stop(t0 + 0.5, t1)
    tflops = flops_per_call * calls / (e0.elapsed_time(e1) * 1e-3) / 1e12
    w = c.get("power_w_median")
    return {"tflops": tflops, "watts_median": w, "sm_mhz_median": c.get("sm_mhz"), "samples": c.get("samples"),
            "reasons": c.get("reasons"), "joules_per_tflop": (w / tflops) if w and tflops else None, "seconds": t1 - t0}


def oracle_sample(wl, budget_s: float = 12.0):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: one full step on matrices of
    every distinct shape, repeated round-robin over the shapes until about `budget_s` seconds of CPU work
    are spent, then extrapolated to the whole set by matrix count.  Returns (steps/s, description, threads)."""
    import numpy as np
    import oracle.mona_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    counts = {}
    for s in wl.specs:
        counts[(s.rows, s.cols)] = counts.get((s.rows, s.cols), 0) + s.batch
    rng = np.random.default_rng(wl.seed)
    hp = orc.Hyper(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha)
    times = {k: [] for k in counts}
    spent = 0.0
    while True:
        for (m, n) in counts:
            W = rng.standard_normal((m, n)) * 0.02
            G = rng.standard_normal((m, n)) * wl.sigma
            st = orc.OracleState(m, n)
            t0 = time.perf_counter()
            orc.mona_step(W, G, st, hp)
            dt = time.perf_counter() - t0
            times[(m, n)].append(dt)
            spent += dt
        if spent >= budget_s or len(next(iter(times.values()))) >= 64:
            break
    total, parts = 0.0, []
    for (m, n), cnt in counts.items():
        t = sum(times[(m, n)]) / len(times[(m, n)])
        total += cnt * t
        parts.append(f"{m}x{n}: {t * 1e3:.1f} ms x {cnt}")
    reps = len(next(iter(times.values())))
    desc = (f"fp64 numpy oracle, {reps} matrices of every distinct shape, one full step each ({spent:.1f} s of CPU work), "
            f"extrapolated by matrix count: " + "; ".join(parts))
    return 1.0 / total, desc, threads


def pick_workload(index, layers, free_bytes):
    """The requested configuration, with the layer count reduced until it fits the device."""
    from paper_2605_26842_b200 import synth
    wl = synth.workload(index, layers)
    note = ""
    if layers is None and index in (1, 2, 3, 4, 5, 6, 7):
        nominal = {1: 12, 2: 16, 3: 24, 4: 8, 5: 10, 6: 10, 7: 14}[index]
        L = nominal
        # W, state, G resident + ~3 GB for workspace, generator temporaries and the L2 flush buffer
        while L > 1 and synth.resident_bytes(synth.workload(index, L)) + (3 << 30) > free_bytes:
            L -= 1
        if L != nominal:
            note = f"layer count reduced from {nominal} to {L} to fit device memory; per-matrix shapes unchanged"
            wl = synth.workload(index, L)
    return wl, note


def run_reference(args):
    """`--impl reference`: the oracle on the host cores, same metric and configuration."""
    from paper_2605_26842_b200 import shard, synth
    if shard.env_rank()[0] != 0:
        return
    wl = synth.workload(args.config, args.layers)
    vals = []
    desc = ""
    threads = 1
    for i in range(args.warmup + args.steps):
        v, desc, threads = oracle_sample(wl, 10.0)
        if i >= args.warmup:
            vals.append(v)
    value = len(vals) / sum(1.0 / v for v in vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "matrices": wl.n_matrices, "params": wl.n_params},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def library_yardstick(torch, dev, wl, chunk_budget=768 << 20, index=None):
    """Diagnostic only (never on the product path): the library batched GEMM (torch.bmm, bf16) on the three GEMM
    shapes of the workload's dominant bucket, one chunk's worth of matrices, timed back to back with CUDA events.
    Dense products: the library computes all of X X^T and A A, not their lower triangles.  With `index` (the device's
    nvidia-smi index) the three products are also run back to back for a few seconds with power sampling."""
    best = None
    for sp in wl.specs:
        s_, l_ = min(sp.rows, sp.cols), max(sp.rows, sp.cols)
        cost = sp.batch * (4.0 * s_ * s_ * l_ + 2.0 * s_ ** 3)
        if s_ >= 64 and (best is None or cost > best[0]):
            best = (cost, s_, l_)
    if best is None:
        return None
    _, s_, l_ = best
    C = max(1, min(512, chunk_budget // ((2 * s_ * l_ + 2 * s_ * s_) * 2)))
    X = torch.randn(C, s_, l_, device=dev, dtype=torch.bfloat16)
    A = torch.randn(C, s_, s_, device=dev, dtype=torch.bfloat16)
    Xn, A2 = torch.empty_like(X), torch.empty_like(A)

    def t(fn, n=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / n * 1e-3
    t1 = t(lambda: torch.bmm(X, X.transpose(1, 2), out=A2))
    t2 = t(lambda: torch.bmm(A, A, out=A2))
    t3 = t(lambda: torch.bmm(A, X, out=Xn))
    f1, f2, f3 = 2.0 * C * s_ * s_ * l_, 2.0 * C * s_ ** 3, 2.0 * C * s_ * s_ * l_
    out = {"shape": f"{C} x ({s_} x {l_})", "what": "torch.bmm bf16, dense products, back to back",
           "XXt": f1 / t1 / 1e12, "AA": f2 / t2 / 1e12, "BX": f3 / t3 / 1e12, "all_three": (f1 + f2 + f3) / (t1 + t2 + t3) / 1e12}
    if index is not None:
        def three():
            torch.bmm(X, X.transpose(1, 2), out=A2)
            torch.bmm(A, A, out=A2)
            torch.bmm(A, X, out=Xn)
        out["sustained"] = sustained(torch, dev, index, three, f1 + f2 + f3)
    del X, A, Xn, A2
    return out


def run_workload(torch, pkg, synth, shard, args, dev, local_rank, rank, world, dist, index, layers, steps, warmup, full):
    """Times one parameter set.  `full`: the headline configuration (clock sampling over the timed steps, yardstick,
    end-to-end and CPU legs); otherwise a short run that returns the compact figures of the other configurations."""
    free_bytes, _ = torch.cuda.mem_get_info(dev)
    wl, fit_note = pick_workload(index, layers, free_bytes)
    options = pkg.default_options()
    if args.chunk_mb:
        options.chunk_budget_bytes = args.chunk_mb << 20
    if args.no_overlap:
        options.chunk_overlap = 0
    if args.fuse:
        options.fuse_update = 1
    if args.ns_delay:
        options.ns_delay = args.ns_delay
    if args.macro_min_k:
        options.macro_tile_min_k = args.macro_min_k
    # every rank owns an independent parameter set of this shape (weak scaling, no data-path collective)
    params = synth.init_params(wl, dev, seed_offset=rank)
    gp = synth.GradientProcess(wl, dev, keep_fp32_shadow=False)
    opt = pkg.MonaOptimizer(params, grad_dtype=wl.grad_dtype, device=local_rank, options=options,
                            state_dtype=pkg.MONA_STATE_COMBINED if args.single_buffer else (torch.bfloat16 if args.lite else torch.float32))
    hp = pkg.default_hparams(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha, algorithm=1 if args.muon else 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    g_elem = 2 if wl.grad_dtype == torch.bfloat16 else 4
    aux = 2 if args.lite else 4                     # bytes per element of A_k and of G_{k-1}

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed_steps(n, mask=7, refresh=True):
        evs = []
        for _ in range(n):
            if refresh:
                gp.next()
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            if mask == 7:
                opt.step(hp, params, gp.grads)
            else:
                opt.step_ex(hp, params, gp.grads, None, mask)
            e1.record(stream)
            evs.append((e0, e1))
        torch.cuda.synchronize(dev)
        return [a.elapsed_time(b) for a, b in evs]

    gp.next()
    timed_steps(warmup)
    barrier()
    sampler = ClockSampler(local_rank) if full else None
    if sampler:
        sampler.start()
    t_wall0 = time.time()
    ms = timed_steps(steps)
    t_wall1 = time.time()
    barrier()
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    st, bad = opt.poll_status()
    if st != 0:
        raise RuntimeError(f"device status {pkg.STATUS_NAMES[st]} at matrix {bad}")
    launches_per_step = opt.last_launch_count()
    total_ms = shard.max_over_ranks(sum(ms), dist, dev)
    ms_per_step = total_ms / steps
    value = shard.whole_job_rate(1.0, world, ms_per_step * 1e-3)

    # ---- per-phase passes (one phase alone; state keeps evolving, which does not change the work) ----
    n_phase = max(2, min(steps, 3))
    ns_clocks = None
    timed_steps(1, mask=1, refresh=False)
    ms_pro = statistics.median(timed_steps(n_phase, mask=1, refresh=False))
    # The Newton-Schulz kernel alone (mask 2: O_k stored in bf16) and together with the update (mask 6: in the kernel's last
    # epilogue when fuse_update is on, as a separate kernel otherwise).  The pass that times the kernel as it runs inside the
    # step is the one whose clocks are sampled.
    fused = bool(opt.options.fuse_update)
    passes = {}
    for mask in ((2, 6) if fused else (6, 2)):
        timed_steps(1, mask=mask, refresh=False)
        sampled = full and mask == (6 if fused else 2)
        ns_sampler = ClockSampler(local_rank) if sampled else None
        if ns_sampler:
            ns_sampler.start()
        t_ns0 = time.time()
        passes[mask] = statistics.median(timed_steps(max(n_phase, 5) if sampled else n_phase, mask=mask, refresh=False))
        t_ns1 = time.time()
        if ns_sampler:
            ns_clocks = ns_sampler.stop(t_ns0, t_ns1)
        if mask == 2:
            ns_launches = opt.last_launch_count()
    ms_nsu, ms_ns = passes[6], passes[2]
    flops_exec, flops_dense = opt.last_ns_flops()
    flops_useful = opt.last_ns_useful_flops()
    timed_steps(1, mask=4, refresh=False)
    ms_upd = statistics.median(timed_steps(n_phase, mask=4, refresh=False))
    st, bad = opt.poll_status()   # phase-only passes may see stale iterates; clear whatever they latched

    peaks, peak_src = load_peaks()
    n = wl.n_params
    pro_elem = g_elem + 2 * aux + 4 + 2 * aux + 4 + 2   # read G, G_prev, A, M; write G_prev, A, M, bf16 X
    if args.single_buffer:
        pro_elem = g_elem + 4 + 4 + 4 + 4 + 2           # read G, Z, M; write Z, M, bf16 X
    if args.muon:
        pro_elem = g_elem + 4 + 4 + 2                   # read G, M; write M, bf16 X
    pro_gbs = n * pro_elem / (ms_pro * 1e-3) / 1e9
    upd_gbs = n * (4 + 2 + 4) / (ms_upd * 1e-3) / 1e9   # read W, bf16 O; write W
    ms_kernel = ms_nsu if fused else ms_ns
    ns_tflops = flops_exec / (ms_kernel * 1e-3) / 1e12
    phases = {"prologue_ms": ms_pro, "prologue_gbs": pro_gbs, "prologue_frac_of_hbm_peak": pro_gbs / peaks["hbm_gbs"],
              "prologue_frac_of_nominal_8000": pro_gbs / 8000.0, "prologue_bytes_per_elem": pro_elem,
              "ns_with_update_ms": ms_nsu, "ns_store_bf16_ms": ms_ns, "separate_update_ms": ms_upd,
              "ns_tflops_executed": ns_tflops, "ns_tflops_useful": flops_useful / (ms_kernel * 1e-3) / 1e12,
              "ns_tflops_executed_without_update": flops_exec / (ms_ns * 1e-3) / 1e12,
              "separate_update_gbs": upd_gbs, "separate_update_frac_of_hbm_peak": upd_gbs / peaks["hbm_gbs"],
              "update": "in the epilogue of the last GEMM of the Newton-Schulz kernel" if fused else "separate kernel",
              "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peak_src}
    result = {"wl": wl, "fit_note": fit_note, "value": value, "ms_per_step": ms_per_step, "ms": ms, "clocks": clocks,
              "launches_per_step": launches_per_step, "phases": phases, "hp": hp, "options": opt.options}
    if not full:
        opt.close()
        del params, gp, flush, opt
        torch.cuda.empty_cache()
        return result

    # the Newton-Schulz kernel runs inside a long step: compare with the sustained GEMM peak
    mhz = (ns_clocks or {}).get("sm_mhz")
    roofline = {"kernel": "ns_chunk_kernel (all Newton-Schulz GEMMs of a chunk in one launch"
                          + (", parameter update in the last epilogue)" if fused else ")"), "bound": "tensor",
                "achieved": ns_tflops, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": ns_tflops / peaks["bf16_tflops_sustained"], "peak_source": peak_src + " (sustained bf16 GEMM)",
                "frac_of_burst_peak": ns_tflops / peaks["bf16_tflops"], "frac_of_nominal_2250": ns_tflops / 2250.0,
                "flops": "executed tile MMAs (padding and upper halves of diagonal tiles included)",
                "useful_tflops": flops_useful / (ms_kernel * 1e-3) / 1e12, "useful_flops_per_matrix_iteration": "3 s^2 l + s^3",
                "flops_per_launch": flops_exec / max(1, ns_launches), "launches_per_step": ns_launches,
                "avg_launch_us": ms_kernel * 1e3 / max(1, ns_launches), "traffic": kernel_traffic(),
                "traffic_unit": NCU_TRAFFIC["unit"],
                "dense_equivalent_tflops": flops_dense / (ms_kernel * 1e-3) / 1e12,
                "sm_mhz_during_pass": mhz, "clock_reasons_during_pass": (ns_clocks or {}).get("reasons"),
                "util_per_clock": (ns_tflops / (2250.0 * mhz / 1965.0)) if mhz else None,
                "util_per_clock_note": "achieved / (2250 TFLOP/s x median SM MHz during the pass / 1965)"}
    if full and world == 1 and not args.no_yardstick:
        # Diagnostic: the Newton-Schulz pass back to back for a few seconds with power sampling, to put joules per executed
        # TFLOP beside the library's on the same shapes (main() adds that leg).  Runs after every timed figure above.
        try:
            roofline["energy"] = {"ns_kernel": sustained(torch, dev, local_rank, lambda: opt.step_ex(hp, params, gp.grads, None, 2), flops_exec),
                                  "power_field": power_field(local_rank),
                                  "note": "Newton-Schulz pass (executed flops) and the library's dense products of the dominant bucket, "
                                          "each run back to back for ~2.5 s; watts = median nvidia-smi sample after the first 0.5 s"}
            opt.poll_status()
        except Exception as exc:
            roofline["energy"] = {"error": str(exc)[:200]}
    result["roofline"] = roofline
    result.update({"opt": opt, "params": params, "gp": gp, "stream": stream, "barrier": barrier})
    return result


def run_sharded(torch, pkg, synth, shard, args, dev, local_rank, rank, world, dist):
    """--shard: ONE parameter set split over the ranks by whole matrices (ZeRO-1 style).  Every rank holds the full
    parameters, the state and gradients of its own share only, steps its share and then takes part in the exchange
    of the updated slices.  Reports the step time with and without the exchange."""
    wl = synth.workload(args.config, args.layers)
    shapes = [(s.batch, s.rows, s.cols) for s in wl.specs]
    all_shares = shard.partition(shapes, world)
    mine = all_shares[rank]
    params = synth.init_params(wl, dev, seed_offset=0)                  # same full set on every rank
    my_params = shard.local_views(params, mine)
    sub = synth.Workload(wl.name + f"_share{rank}", [synth.MatrixSpec(f"s{i}", r, c, b) for i, (b, r, c) in
                                                      enumerate(shard.share_shapes(shapes, mine))], steps=wl.steps,
                         rho=wl.rho, sigma=wl.sigma, dist=wl.dist, grad_dtype=wl.grad_dtype, accel_beta=wl.accel_beta,
                         seed=wl.seed + 100 * rank)
    gp = synth.GradientProcess(sub, dev, keep_fp32_shadow=False)
    opt = pkg.MonaOptimizer(my_params, grad_dtype=wl.grad_dtype, device=local_rank)
    hp = pkg.default_hparams(accel_beta=wl.accel_beta, accel_alpha=wl.accel_alpha)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def run(n, with_exchange):
        times = []
        for _ in range(n):
            gp.next()
            flush.zero_()
            torch.cuda.synchronize(dev)
            if dist is not None:
                dist.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            opt.step(hp, my_params, gp.grads)
            if with_exchange:
                shard.exchange(params, all_shares, dist)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            times.append(e0.elapsed_time(e1))
        return shard.max_over_ranks(sum(times), dist, dev) / n
    run(args.warmup, True)
    ms_with = run(args.steps, True)
    ms_without = run(args.steps, False)
    st, bad = opt.poll_status()
    if st != 0:
        raise RuntimeError(f"device status {pkg.STATUS_NAMES[st]} at matrix {bad}")
    total = sum(b * r * c * 4 for b, r, c in shapes)
    owned = sum(b * r * c * 4 for b, r, c in shard.share_shapes(shapes, mine))
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": 1e3 / ms_with, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms_with, "ms_per_step_without_exchange": ms_without,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16 tensor-core Newton-Schulz; fp32 state and parameters",
                          "data": "synthetic", "config": {"workload": wl.name, "config_index": args.config, "matrices": wl.n_matrices,
                                                          "params": wl.n_params, "parallelism": f"one parameter set partitioned by whole matrices over {world} rank(s); updated fp32 slices broadcast from their owners",
                                                          "matrices_on_rank0": sum(s.count for s in mine)},
                          "exchange_bytes_received_per_step_rank0": total - owned, "gpu_launches": opt.last_launch_count() * args.steps}))
    opt.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, help="parameter set 0..7 (default 3: the ~7B MoE set; 5-7: the paper's own expert shapes)")
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--impl", default="mona", choices=["mona", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-yardstick", action="store_true", help="skip the library-GEMM diagnostic")
    ap.add_argument("--chunk-mb", type=int, default=None, help="override the chunk budget (MiB)")
    ap.add_argument("--no-overlap", action="store_true", help="keep all chunks on one stream")
    ap.add_argument("--fuse", action="store_true", help="apply the parameter update in the epilogue of the last GEMM instead of a separate kernel")
    ap.add_argument("--ns-delay", type=int, default=None, help="work-order distance between consecutive GEMMs of one matrix")
    ap.add_argument("--macro-min-k", type=int, default=None, help="shortest inner dimension for which X' = B'X uses 256x512 macro-tiles")
    ap.add_argument("--shard", action="store_true", help="one parameter set partitioned over the ranks, parameters exchanged after the step")
    ap.add_argument("--muon", action="store_true", help="plain Muon step (no acceleration term): the baseline of the paper's timing claim")
    ap.add_argument("--single-buffer", action="store_true", help="state kept as M and Z = beta_a A - (1 - beta_a) G (one fp32 buffer instead of A and G_prev)")
    ap.add_argument("--lite", action="store_true", help="MONA-Lite storage: A_k and G_{k-1} kept in bfloat16")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2605_26842_b200 as pkg
    from paper_2605_26842_b200 import shard, synth
    rank, local_rank, world = shard.env_rank()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if args.shard:
        run_sharded(torch, pkg, synth, shard, args, dev, local_rank, rank, world, dist)
        if dist is not None:
            dist.destroy_process_group()
        return

    r = run_workload(torch, pkg, synth, shard, args, dev, local_rank, rank, world, dist, args.config, args.layers,
                     args.steps, args.warmup, full=True)
    wl, opt, params, gp, stream, barrier, hp = r["wl"], r["opt"], r["params"], r["gp"], r["stream"], r["barrier"], r["hp"]
    if rank == 0 and world == 1 and not args.no_yardstick:
        try:
            lib = library_yardstick(torch, dev, wl, int(r["options"].chunk_budget_bytes), index=local_rank)
            r["roofline"]["library_same_shape_tflops"] = lib
            if lib and "sustained" in lib and isinstance(r["roofline"].get("energy"), dict) and "ns_kernel" in r["roofline"]["energy"]:
                r["roofline"]["energy"]["library_same_shape"] = lib.pop("sustained")
        except Exception as exc:     # a diagnostic must not take the benchmark down (e.g. no memory left for its operands)
            r["roofline"]["library_same_shape_tflops"] = {"error": str(exc)[:200]}

    # ---- end to end: host gradients in, host parameters out, through mona_step_host ----
    e2e = None
    if not args.no_e2e:
        # the pinned host copies of all gradients and parameters must fit the node for every rank at once
        need = sum(g.numel() * g.element_size() for g in gp.grads) + sum(p.numel() * p.element_size() for p in params)
        try:
            import psutil
            avail = psutil.virtual_memory().available
        except Exception:
            avail = None
        if dist is not None:    # every rank must take the same branch: use the smallest figure any rank saw
            avail = -shard.max_over_ranks(-float(avail if avail is not None else 0.0), dist, dev)
        if avail is not None and need * world > 0.6 * avail:
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                   "error": f"skipped: {world} rank(s) x {need / 1e9:.1f} GB of pinned host memory against {avail / 1e9:.1f} GB available"}
    if not args.no_e2e and e2e is None:
        try:
            g_host = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True) for g in gp.grads]
            p_host = [torch.empty(p.shape, dtype=p.dtype, pin_memory=True) for p in params]
            for h_, g in zip(g_host, gp.grads):
                h_.copy_(g)
            torch.cuda.synchronize(dev)
            h2d = sum(g.numel() * g.element_size() for g in gp.grads)
            d2h = sum(p.numel() * p.element_size() for p in params)
            n_e2e = max(1, min(args.steps, 3))
            e_ms = []
            for i in range(1 + n_e2e):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                barrier()
                e0.record(stream)
                opt.step_host(hp, params, gp.grads, g_host, p_host)
                e1.record(stream)
                torch.cuda.synchronize(dev)
                if i > 0:
                    e_ms.append(e0.elapsed_time(e1))
            e_total = shard.max_over_ranks(sum(e_ms), dist, dev)
            e2e = {"value": shard.whole_job_rate(1.0, world, e_total / n_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "steps": n_e2e, "api": "mona_step_host (pinned host gradients in, updated parameters out)"}
            del g_host, p_host
        except Exception as exc:   # e.g. not enough pinned host memory
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "error": str(exc)[:200]}
    opt.close()
    del opt, params, gp
    r.pop("opt"); r.pop("params"); r.pop("gp")
    torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        v, desc, threads = oracle_sample(wl, 15.0)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    # ---- the other benchmark configurations, briefly (one GPU only; the headline stays the configuration above) ----
    others = None
    if world == 1 and not args.no_others and args.config == 3 and args.layers is None:
        others = {}
        for idx in (1, 2, 4, 5):       # 5: the paper-shaped 256 x 768 expert set (its smallest model's experts)
            try:
                o = run_workload(torch, pkg, synth, shard, args, dev, local_rank, rank, world, dist, idx, None, 3, 3, full=False)
                ph = o["phases"]
                others[o["wl"].name] = {"config_index": idx, "params": o["wl"].n_params, "steps_per_s": o["value"], "ms_per_step": o["ms_per_step"],
                                        "ns_tflops_executed": ph["ns_tflops_executed"], "ns_tflops_useful": ph["ns_tflops_useful"],
                                        "prologue_gbs": ph["prologue_gbs"], "prologue_bytes_per_elem": ph["prologue_bytes_per_elem"],
                                        "separate_update_gbs": ph["separate_update_gbs"], "note": o["fit_note"]}
            except Exception as exc:
                others[f"config_{idx}"] = {"error": str(exc)[:200]}

    if rank == 0:
        line = {"metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16 tensor-core Newton-Schulz with fp32 accumulate; fp32 state and parameters",
                "data": "synthetic",
                "config": {"workload": wl.name, "config_index": args.config, "matrices": wl.n_matrices, "params": wl.n_params,
                           "grad_dtype": str(wl.grad_dtype).replace("torch.", ""), "gradient_process":
                           f"AR(1) rho={wl.rho} sigma={wl.sigma} {wl.dist}", "ns_steps": hp.ns_steps,
                           "accel_beta": wl.accel_beta, "accel_alpha": wl.accel_alpha,
                           "state_storage": "single fp32 buffer Z" if args.single_buffer else ("bf16 A_k and G_{k-1} (MONA-Lite)" if args.lite else "fp32"),
                           "algorithm": "Muon (no acceleration term)" if args.muon else "MONA", "parallelism":
                           "independent parameter set per GPU, no collective" if world > 1 else "single GPU",
                           "l2": "inputs larger than L2 and a 256 MiB buffer rewritten between timed steps",
                           "timing": "CUDA events around each mona_step; gradient refresh between steps untimed",
                           "note": r["fit_note"]},
                "gpu_launches": r["launches_per_step"] * args.steps, "launches_per_step": r["launches_per_step"],
                "step_ms_each": r["ms"], "clocks": r["clocks"], "roofline": r["roofline"], "phases": r["phases"], "e2e": e2e,
                "cpu_baseline": cpu, "other_configs": others}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
