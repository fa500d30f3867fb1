#!/usr/bin/env python
"""Benchmark of the SSN stage-boundary codec on B200.

One *step* is one pass of the whole hot path over one microbatch of the 8B-class stage
boundary (d=4096, k=40, vocab 128256, 32 x 2048 = 65536 tokens, bf16, Zipf(1.1) token ids):

    compress  Z  = (X - E[ids] - P) U          (sender, forward)
    decompress Xhat = Z U^T + E[ids] + P       (receiver, forward)
    grad-project dZ = G U                      (backward)
    weight re-projection W <- (W U) U^T of one transformer block's attention out-projection
        [4096 x 4096] and MLP down-projection [14336 x 4096]   (after the optimizer step)

The metric is tokens per second through that step.  Every rank runs its own replica on its own
microbatch (tokens are independent, so there is no collective on the data path): weak scaling.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

`--impl reference` times the CPU oracle (test infrastructure, as it stands) on a bounded sample.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ssn_codec_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")


def recorded_traffic(config_name, default_size):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) that an earlier ncu
    capture of this same workload recorded, read from profiles/dram_traffic.json (written next to
    the ncu summaries).  A recorded capture, not a measurement of this run; {} for any other
    workload size."""
    if not default_size:
        return {}
    try:
        with open(TRAFFIC_FILE) as fh:
            return json.load(fh).get(config_name, {})
    except (OSError, ValueError):
        return {}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", choices=["stage8b", "mid"], default="stage8b",
                    help="stage8b: the 8B-class stage boundary the metric is quoted on (d=4096, k=40, "
                         "65536 tokens, Zipf ids); mid: d=2048, k=32, vocab 32000, 32768 tokens, uniform "
                         "ids, re-projection of W [2048 x 8192] on the left")
    ap.add_argument("--batch", type=int, default=None, help="sequences per microbatch (default: the config's)")
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the sustained run behind the clock_sensitivity object (0: skip it)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tables", action="store_true",
                    help="the step's compress reads the prepared tables E U, P U instead of gathering "
                         "the E and P rows (the default step gathers; the table variant is always "
                         "timed beside it as compress_prepared_tables)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sweep", choices=["compress", "reproject", "reparam", "wire", "dp", "small", "fusions"],
                    default=None,
                    help="instead of the step: time the compress sweep (d, k, tokens) or the "
                         "re-projection sweep (k, weight shape, 32 layers); one JSON line per point")
    return ap.parse_args()


def workload(args):
    from paper_2607_13332_b200 import synth

    wl = synth.WORKLOADS[args.config]
    if args.batch is not None:
        wl = wl.scaled(batch=args.batch)
    return wl


def reproject_weights(wl):
    """(side, [(rows, cols), ...]) of the step's weight re-projection: the 8B block's out-proj and
    down-proj with the subspace on the columns, or the mid config's W [d x 8192] with it on the rows."""
    if wl.name == "mid":
        return "left", [(wl.d, 8192)]
    return "right", [(4096, wl.d), (14336, wl.d)]


def config_of(wl, world, tables=False):
    side, shapes = reproject_weights(wl)
    ids = f"Zipf({wl.zipf_s})" if wl.ids_law == "zipf" else "uniform"
    title = "8B-class stage boundary" if wl.name == "stage8b" else f"{wl.name} codec"
    return {
        "compress_terms": "prepared tables EU=E.U, PU=P.U (fp32, made once before the timed region)"
                          if tables else "E and P rows gathered every step",
        "workload": f"{title}: d={wl.d}, k={wl.k}, vocab={wl.vocab}, "
                    f"{wl.batch}x{wl.seq_len}={wl.n_tokens} tokens, bf16, {ids} ids; "
                    "compress + decompress + grad-project + re-projection of "
                    + " and ".join(f"[{r}x{c}]" for r, c in shapes) + f" ({side}) per step",
        "d": wl.d, "k": wl.k, "vocab": wl.vocab, "tokens_per_rank": wl.n_tokens,
        "replicas": world,
        "l2": f"inputs larger than L2 (X, G: {wl.n_tokens * wl.d * 2 / 1e6:.0f} MB each, "
              f"E: {wl.vocab * wl.d * 2 / 1e6:.0f} MB)",
    }


# ----------------------------------------------------------------------------------------------
# compulsory ("algorithmic") bytes of one launch: each distinct table row counted once
# ----------------------------------------------------------------------------------------------
def algorithmic_bytes(wl, ids, step, tables=False):
    b = 2
    n, d, k = wl.n_tokens, wl.d, wl.k
    uniq = int(np.unique(ids).size)
    shift = uniq * d * b + min(wl.seq_len, n) * d * b
    if step == "compress" and tables:     # X, ids, one fp32 table row per distinct id / position, U, Z
        return n * d * b + n * 4 + (uniq + min(wl.seq_len, n)) * k * 4 + d * k * b + n * k * b
    if step in ("compress", "decompress"):
        return n * d * b + shift + d * k * b + n * k * b
    if step == "grad_project":
        return n * d * b + d * k * b + n * k * b
    if step == "weight_reproject":        # every weight read once and written once
        _, shapes = reproject_weights(wl)
        return 2 * sum(r * c for r, c in shapes) * b + 2 * d * k * b
    raise ValueError(step)


# ----------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline of the GPU arm, and the whole of --impl reference)
# ----------------------------------------------------------------------------------------------
def oracle_tokens_per_s(wl, seconds, seed=0x5EED + 32):
    """Times the oracle, as it stands, on a bounded SAMPLE of the step: `sample` tokens through
    compress, decompress and grad-project plus the same fraction of the re-projected weights, on
    all host threads numpy's BLAS uses and once more on one thread.  tokens/s of the full step is
    extrapolated from the sample (every token, row and column is independent)."""
    from threadpoolctl import threadpool_info, threadpool_limits

    from oracle import ssn_oracle as oracle
    from paper_2607_13332_b200 import synth

    sample = min(wl.n_tokens, 4096)
    small = synth.Workload("sample", wl.d, wl.k, min(wl.vocab, 16384), 1, sample, wl.dtype,
                           wl.ids_law, wl.zipf_s)
    t = synth.codec_inputs(small, seed=seed)
    pos = oracle.token_positions(sample, wl.seq_len)
    P = synth.to_storage(synth.sinusoidal_positions(wl.seq_len, wl.d), wl.dtype)
    side, shapes = reproject_weights(wl)
    free_extent = sum(r if side == "right" else c for r, c in shapes)
    w_extent = max(1, free_extent * sample // wl.n_tokens)
    W = synth.projection_weight(w_extent, wl.d, seed, wl.dtype)     # [extent x d]; transposed for the left side

    f = lambda a: synth.to_f64(a, wl.dtype)
    U, E, Pf = f(t["U"]), f(t["E"]), f(P)      # the shared tables are set up once, untimed

    def one_pass():
        Z, _ = oracle.compress(f(t["X"]), U, E, t["ids"], Pf, pos)
        oracle.decompress(Z, U, E, t["ids"], Pf, pos)
        oracle.grad_project_coeff(f(t["G"]), U)
        Wf = f(W)
        oracle.weight_reproject(Wf if side == "right" else np.ascontiguousarray(Wf.T), U, side)

    def rate(budget):
        one_pass()
        t0 = time.perf_counter()
        one_pass()
        per_pass = time.perf_counter() - t0
        reps = max(1, int(budget / max(per_pass, 1e-3)))
        t0 = time.perf_counter()
        for _ in range(reps):
            one_pass()
        elapsed = time.perf_counter() - t0
        return sample * reps / elapsed, reps, elapsed

    value, reps, elapsed = rate(seconds)
    cores = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    with threadpool_limits(limits=1):
        value_1, _, _ = rate(max(1.0, seconds / 4))
    return {
        "value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle", "extrapolated": True,
        "value_1_thread": value_1,
        "sample": f"{reps} passes over a {sample}-token sample (+{w_extent} weight {'rows' if side == 'right' else 'columns'}) "
                  f"of the step, numpy fp64, {elapsed:.1f} s; tokens/s of the full step extrapolated from "
                  "the sample (tokens are independent)",
    }, elapsed / reps


# ----------------------------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.lines = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [l for (ts, l) in self.lines if (t_begin is None or t_begin <= ts <= t_end + 0.1)]
        if not rows:
            rows = [l for (_, l) in self.lines]
        sm, smax, reasons = [], [], set()
        for row in rows:
            parts = [p.strip() for p in row.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, flag in zip(self.NAMES, parts[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload(args)
    total_steps = args.warmup + args.steps
    per_step_seconds = max(1.0, min(args.cpu_seconds, 120.0 / max(1, total_steps)))
    values, last = [], None
    for i in range(total_steps):
        last, per_pass = oracle_tokens_per_s(wl, per_step_seconds)
        if i >= args.warmup:
            values.append(last["value"])
    value = float(np.mean(values))
    last["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.n_tokens / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(wl, 1), "cpu_baseline": last,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args):
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    from paper_2607_13332_b200 import binding, dist_util, synth
    from paper_2607_13332_b200.runner import Codec, to_device

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SSN codec has no CPU path")
    rank, world, local = dist_util.rank_world()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    wl = workload(args)
    default_size = args.batch is None
    dt = wl.dtype
    t = synth.codec_inputs(wl, seed=0x5EED + 32 + 1000 * rank)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    tables = args.tables
    codec_t = Codec(dt, codec.U, codec.E, codec.P)
    codec_t.prepare_tables()        # constants of the codec, like U, E and P: set up once
    compress_codec = codec_t if tables else codec
    n, d, k = wl.n_tokens, wl.d, wl.k
    ids_h = torch.from_numpy(t["ids"]).pin_memory()
    X_h = torch.from_numpy(t["X"].view(np.int16)).view(torch.bfloat16).pin_memory()
    G_h = torch.from_numpy(t["G"].view(np.int16)).view(torch.bfloat16).pin_memory()
    X, G, ids = X_h.cuda(), G_h.cuda(), ids_h.cuda()
    Z = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
    dZ = torch.empty_like(Z)
    Xh = torch.empty_like(X)
    Z_h, dZ_h = Z.cpu().pin_memory(), dZ.cpu().pin_memory()
    side, shapes = reproject_weights(wl)
    weights = [to_device(synth.projection_weight(r, c, 0x5EED, dt, layer=i), dt)
               for i, (r, c) in enumerate(shapes)]
    del t["X"], t["G"], t["E"]

    stream = torch.cuda.current_stream()

    def reproject():     # every weight of the step in one call (and one launch)
        codec.weight_reproject_list(weights, side)

    calls = (("compress", lambda: compress_codec.compress(X, ids, seq_len=wl.seq_len, out=Z)),
             ("decompress", lambda: codec.decompress(Z, ids, seq_len=wl.seq_len, out=Xh)),
             ("grad_project", lambda: codec.grad_project(G, out=dZ)),
             ("weight_reproject", reproject))
    kernel_events = []

    def step(record=False):
        for name, call in calls:
            if record:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            call()
            if record:
                e1.record(stream)
                kernel_events.append((name, e0, e1))

    def e2e_step():
        X.copy_(X_h, non_blocking=True)
        G.copy_(G_h, non_blocking=True)
        ids.copy_(ids_h, non_blocking=True)
        step()
        Z_h.copy_(Z, non_blocking=True)
        dZ_h.copy_(dZ, non_blocking=True)

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, per_step=None, **kw):
        """Device time of `steps` calls of fn, max over ranks; per_step (a list) also receives one
        event pair per call."""
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(steps):
            if per_step is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            fn(**kw)
            if per_step is not None:
                e1.record(stream)
                per_step.append((e0, e1))
        b.record(stream)
        barrier()
        return dist_util.max_over_ranks(a.elapsed_time(b), device="cuda")

    for _ in range(max(3, args.warmup)):
        step()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = binding.ssn_launch_count()
    t_begin = time.perf_counter()
    ms_total = timed(step, args.steps)
    launches = binding.ssn_launch_count() - launches0
    # the same loop with an event pair around every step (median / min), then around every call
    # (events add small gaps, so neither pass is the one that gives `value`)
    step_events = []
    timed(step, args.steps, per_step=step_events)
    step_ms = sorted(a.elapsed_time(b) for a, b in step_events)
    timed(step, args.steps, record=True)
    per_call = {name: sorted(a.elapsed_time(b) for n_, a, b in kernel_events if n_ == name) for name, _ in calls}
    kernel_ms = {name: float(np.mean(v)) for name, v in per_call.items()}
    # the compress variant that is not in the step, timed alone the same way
    other = codec if tables else codec_t
    other_name = "compress_rows" if tables else "compress_prepared_tables"
    other_ms = timed(lambda: other.compress(X, ids, seq_len=wl.seq_len, out=Z), args.steps) / args.steps
    for _ in range(2):
        e2e_step()
    ms_e2e = timed(e2e_step, args.steps)
    t_end = time.perf_counter()
    # the clock record spans all the timed passes above (device-resident, per-step, per-kernel, end to end)
    clocks = sampler.stop(t_begin, t_end) if sampler else None

    # host time of one enqueue (argument marshalling, tensor maps, launch): 1000 calls, no device wait
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(250):
        step()
    host_us_per_call = (time.perf_counter() - t0) / 1000 * 1e6
    torch.cuda.synchronize()

    sensitivity = None
    if rank == 0 and world == 1 and args.sustain_seconds > 0:
        sensitivity = clock_sensitivity(args, wl, calls, kernel_ms, clocks, local, timed)

    status = codec.take_status()
    status |= codec_t.take_status()
    if status != 0:
        raise RuntimeError(f"device status {status}: {Codec.describe_status(status)}")

    if rank == 0:
        ms_per_step = ms_total / args.steps
        value = world * n / (ms_per_step * 1e-3)
        peak, peak_kind = measured_hbm_peak()
        traffic = recorded_traffic(wl.name, default_size)
        kernels = {}
        for name, ms in kernel_ms.items():
            algo_k = algorithmic_bytes(wl, t["ids"], name, tables)
            gbs = algo_k / (ms * 1e-3) / 1e9
            key = "compress_prepared_tables" if (name == "compress" and tables) else name
            kernels[name] = {"ms": ms, "ms_median": float(np.median(per_call[name])), "ms_min": per_call[name][0],
                             "algorithmic_bytes": algo_k, "achieved": gbs, "frac": gbs / peak,
                             "frac_of_8TBps": gbs / 8000.0, "traffic": traffic.get(key)}
        algo_o = algorithmic_bytes(wl, t["ids"], "compress", not tables)
        kernels[other_name] = {"ms": other_ms, "algorithmic_bytes": algo_o,
                               "achieved": algo_o / (other_ms * 1e-3) / 1e9,
                               "frac": algo_o / (other_ms * 1e-3) / 1e9 / peak,
                               "frac_of_8TBps": algo_o / (other_ms * 1e-3) / 1e9 / 8000.0,
                               "traffic": traffic.get("compress" if tables else "compress_prepared_tables"),
                               "note": "not part of the step; back-to-back launches"}
        # the roofline object describes the call that takes the largest share of the step
        dominant = max(kernel_ms, key=kernel_ms.get)
        algo, achieved = kernels[dominant]["algorithmic_bytes"], kernels[dominant]["achieved"]
        h2d = X_h.numel() * 2 + G_h.numel() * 2 + ids_h.numel() * 4
        d2h = Z_h.numel() * 2 + dZ_h.numel() * 2
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
            "ms_per_step_median": float(np.median(step_ms)), "ms_per_step_min": step_ms[0],
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(wl, world, tables),
            "roofline": {"bound": "hbm", "kernel": "ssn_" + dominant, "achieved": achieved,
                         "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_8TBps": achieved / 8000.0,
                         "peak_kind": peak_kind, "algorithmic_bytes": algo,
                         "kernel_ms": kernel_ms[dominant], "traffic": kernels[dominant]["traffic"],
                         "traffic_source": "recorded ncu capture of this workload (profiles/dram_traffic.json)"
                                           if kernels[dominant]["traffic"] else None,
                         "kernels": kernels},
            "e2e": {"value": world * n / (ms_e2e / args.steps * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "host_us_per_call": host_us_per_call,
            "clocks": clocks,
        }
        if sensitivity is not None:
            out["clock_sensitivity"] = sensitivity
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"], _ = oracle_tokens_per_s(wl, args.cpu_seconds)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def clock_sensitivity(args, wl, calls, burst_ms, burst_clocks, gpu_index, timed):
    """How the step and each call depend on the SM clock, with the clocks the box gives (none is
    set here).  The timed region of the bench lasts milliseconds and sees the boost clock; a run of
    `--sustain-seconds` of back-to-back steps, and then of each call alone, sees whatever clock the
    power cap leaves.  For each: time, median SM MHz while it ran, and their product (thousands
    of SM clocks per launch).  A call whose product stays put while its time grows is bound on the
    SM side (issue, shared memory); one whose time stays put is bound by HBM."""
    import torch

    def sustained(fn, seconds, block=None):
        fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        fn()
        torch.cuda.synchronize()
        once = max(time.perf_counter() - t0, 1e-5)
        block = block or max(10, int(seconds / 20 / once))
        sampler = ClockSampler(gpu_index)
        time.sleep(0.05)
        t_begin = time.perf_counter()
        blocks = [timed(fn, block) / block for _ in range(20)]
        t_end = time.perf_counter()
        clocks = sampler.stop(t_begin, t_end)
        return {"ms_median": float(np.median(blocks)), "ms_min": float(min(blocks)), "launches_per_block": block,
                "blocks": 20, "sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"],
                "seconds": round(t_end - t_begin, 2)}

    def step():
        for _, call in calls:
            call()

    out = {"burst_sm_mhz": burst_clocks["sm_mhz"] if burst_clocks else None,
           "step": sustained(step, args.sustain_seconds), "kernels": {}}
    for name, call in calls:
        r = sustained(call, max(0.4, args.sustain_seconds / 4))
        mhz, burst_mhz = r["sm_mhz"], (burst_clocks or {}).get("sm_mhz")
        r["kclocks_sustained"] = r["ms_median"] * mhz if mhz else None
        r["burst_ms"] = burst_ms[name]
        r["kclocks_burst"] = burst_ms[name] * burst_mhz if burst_mhz else None
        out["kernels"][name] = r
    return out


def run_sweep(args):
    """Benchmark definition's sweeps, one GPU: device-resident inputs larger than L2 where the
    point allows, CUDA events around `reps` back-to-back launches after 3 warm-up launches."""
    import torch

    import __graft_entry__ as entry
    entry.build()
    from paper_2607_13332_b200 import binding, synth
    from paper_2607_13332_b200.runner import Codec, to_device

    peak, _ = measured_hbm_peak()
    dt, vocab, seq = synth.BF16, 128256, 2048
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)

    def timed_us(fn, reps):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / reps

    if args.sweep == "compress":
        # every point's output is compared with the oracle on sampled tokens by
        # tests/test_gpu_sweep_parity.py, which draws the same inputs from synth_device
        from paper_2607_13332_b200 import synth_device
        for d in (1024, 2048, 4096, 8192):
            gen = synth_device.generator(d)
            E = synth_device.embedding_table(vocab, d, gen)
            P = synth_device.positions_table(seq, d)
            for k in (8, 32, 64, 128):
                U = synth_device.basis(d, k, 1)
                codec, codec_t = Codec(dt, U, E, P), Codec(dt, U, E, P)
                codec_t.prepare_tables()
                for n in (4096, 65536, 524288):
                    ids_np = synth_device.uniform_ids(n, vocab, n + d + k)
                    ids = torch.from_numpy(ids_np).cuda()
                    X = synth_device.activations(n, d, gen)
                    Z = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
                    uniq = int(np.unique(ids_np).size)
                    reps = 20 if n <= 65536 else 5
                    out = {"sweep": "compress", "d": d, "k": k, "tokens": n, "distinct_ids": uniq}
                    for name, c, algo in (
                            ("rows", codec, n * d * 2 + uniq * d * 2 + min(seq, n) * d * 2 + d * k * 2 + n * k * 2),
                            ("tables", codec_t, n * d * 2 + n * 4 + (uniq + min(seq, n)) * k * 4 + d * k * 2 + n * k * 2)):
                        us = timed_us(lambda: c.compress(X, ids, seq_len=seq, out=Z), reps)
                        out[name] = {"us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                                     "frac_of_measured": round(algo / us / 1e3 / peak, 3)}
                    out["status"] = Codec.describe_status(codec.take_status() | codec_t.take_status())
                    print(json.dumps(out), flush=True)
                    del X, Z, ids
            del E, P
    elif args.sweep == "small":
        # the call sizes of the paper's per-stage timing table (1 to 3 coalesced sequences of 4096
        # tokens per call) at the 8B-class boundary; several input sets are rotated so that L2 does
        # not hold a call's input from the call before; host_us is the enqueue cost of one call
        from paper_2607_13332_b200 import synth_device
        d, k = 4096, 40
        gen = synth_device.generator(1)
        E = synth_device.embedding_table(vocab, d, gen)
        P = synth_device.positions_table(seq, d)
        U = synth_device.basis(d, k, 1)
        codec, codec_t = Codec(dt, U, E, P), Codec(dt, U, E, P)
        codec_t.prepare_tables()
        for n in (4096, 8192, 12288, 16384):
            ids_np = synth.zipf_ids(n, vocab, 1.1, seed=n)
            ids = torch.from_numpy(ids_np).cuda()
            uniq = int(np.unique(ids_np).size)
            nset = max(2, (512 << 20) // (n * d * 2))
            Xs = [synth_device.activations(n, d, gen) for _ in range(nset)]
            Zs = [synth_device.activations(n, k, gen) for _ in range(nset)]
            Xh = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
            Zo = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
            turn = [0]

            def nxt(sets):
                turn[0] += 1
                return sets[turn[0] % nset]

            rows_bytes = n * d * 2 + uniq * d * 2 + min(seq, n) * d * 2 + d * k * 2 + n * k * 2
            for name, fn, algo in (
                    ("compress (rows)", lambda: codec.compress(nxt(Xs), ids, seq_len=seq, out=Zo), rows_bytes),
                    ("compress (prepared tables)", lambda: codec_t.compress(nxt(Xs), ids, seq_len=seq, out=Zo),
                     n * d * 2 + n * 4 + (uniq + min(seq, n)) * k * 4 + d * k * 2 + n * k * 2),
                    ("grad_project", lambda: codec.grad_project(nxt(Xs), out=Zo), n * d * 2 + d * k * 2 + n * k * 2),
                    ("decompress", lambda: codec.decompress(nxt(Zs), ids, seq_len=seq, out=Xh), rows_bytes)):
                us = timed_us(fn, 40)
                fam, var = binding.ssn_last_kernel()
                t0 = time.perf_counter()
                for _ in range(200):
                    fn()
                host_us = (time.perf_counter() - t0) / 200 * 1e6
                torch.cuda.synchronize()
                # the same calls replayed from a CUDA graph: device time without the host's enqueue gaps
                graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    fn()
                    with torch.cuda.graph(graph, stream=side):
                        for _ in range(2 * nset):
                            fn()
                torch.cuda.current_stream().wait_stream(side)
                graph_us = timed_us(graph.replay, 10) / (2 * nset)
                print(json.dumps({"sweep": "small", "op": name, "tokens": n, "d": d, "k": k, "us": round(us, 1),
                                  "graph_us": round(graph_us, 1), "host_us": round(host_us, 1),
                                  "GBps": round(algo / min(us, graph_us) / 1e3, 0),
                                  "frac_of_measured": round(algo / min(us, graph_us) / 1e3 / peak, 3),
                                  "kernel_family": fam, "kernel_variant": var}), flush=True)
            del Xs, Zs, Xh
    elif args.sweep == "fusions":
        # decompress with the RMSNorm row statistic of the receiving block, against decompress
        # followed by a separate reduction over the rows it wrote (a library reduction stands in for
        # the norm's first pass)
        from paper_2607_13332_b200 import synth_device
        d, k, n = 4096, 40, 65536
        gen = synth_device.generator(2)
        E = synth_device.embedding_table(vocab, d, gen)
        P = synth_device.positions_table(seq, d)
        codec = Codec(dt, synth_device.basis(d, k, 1), E, P)
        ids_np = synth.token_ids(synth.STAGE_8B, 3)
        ids = torch.from_numpy(ids_np).cuda()
        uniq = int(np.unique(ids_np).size)
        Z = synth_device.activations(n, k, gen)
        Xh = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
        ss = torch.empty(n, dtype=torch.float32, device="cuda")
        algo = n * k * 2 + n * 4 + uniq * d * 2 + seq * d * 2 + d * k * 2 + n * d * 2
        for name, fn, extra in (
                ("decompress", lambda: codec.decompress(Z, ids, seq_len=seq, out=Xh), 0),
                ("decompress_rowsumsq (fused)",
                 lambda: codec.decompress_rowsumsq(Z, ids, seq_len=seq, out=Xh, rowsumsq=ss), n * 4),
                ("decompress, then a separate sum of squares over Xhat",
                 lambda: (codec.decompress(Z, ids, seq_len=seq, out=Xh), torch.linalg.vector_norm(Xh, dim=1, dtype=torch.float32, out=ss)),
                 n * 4)):
            us = timed_us(fn, 10)
            print(json.dumps({"sweep": "fusions", "op": name, "tokens": n, "d": d, "k": k, "us": round(us, 1),
                              "GBps": round((algo + extra) / us / 1e3, 0),
                              "frac_of_measured": round((algo + extra) / us / 1e3 / peak, 3)}), flush=True)
    elif args.sweep == "reparam":
        # reparameterized SSN (Eq. reparam): Y = (H Zw) U^T for the block's two output projections,
        # and the head-stage input with the factored embedding, at the benchmark's token count
        d, k, n = 4096, 40, 65536
        U = to_device(synth.to_storage(synth.subspace_basis(d, k, 1), dt), dt)
        codec = Codec(dt, U)
        Y = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
        for name, m in (("out_proj", 4096), ("down_proj", 14336)):
            H = torch.randn((n, m), device="cuda", generator=gen).bfloat16()
            Zw = (torch.randn((m, k), device="cuda", generator=gen) / m ** 0.5).bfloat16()
            us = timed_us(lambda: codec.reparam_project(H, Zw, out=Y), 5)
            algo = n * m * 2 + n * d * 2 + (m + d) * k * 2
            print(json.dumps({"sweep": "reparam", "op": "reparam_project", "weight": name, "tokens": n, "m": m,
                              "d": d, "k": k, "us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                              "frac_of_measured": round(algo / us / 1e3 / peak, 3)}), flush=True)
            dY = (torch.randn((n, d), device="cuda", generator=gen) * 0.01).bfloat16()
            us = timed_us(lambda: codec.reparam_grad_factor(H, dY), 5)
            algo = n * m * 2 + n * d * 2 + m * k * 4 + d * k * 2
            print(json.dumps({"sweep": "reparam", "op": "reparam_grad_factor", "weight": name, "tokens": n, "m": m,
                              "d": d, "k": k, "us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                              "frac_of_measured": round(algo / us / 1e3 / peak, 3)}), flush=True)
            del H, Zw, dY
        E = (torch.randn((vocab, d), device="cuda", generator=gen) * 0.02).bfloat16()
        P = to_device(synth.to_storage(synth.sinusoidal_positions(seq, d), dt), dt)
        Elow = torch.randn((vocab, k), device="cuda", generator=gen).bfloat16()
        head = Codec(dt, U, E, P)
        wl = synth.STAGE_8B
        ids_np = synth.token_ids(wl, 3)
        ids = torch.from_numpy(ids_np).cuda()
        us = timed_us(lambda: head.head_embed(Elow, ids, seq_len=seq, out=Y), 5)
        uniq = int(np.unique(ids_np).size)
        algo = n * d * 2 + uniq * (d + k) * 2 + seq * d * 2 + n * 4 + d * k * 2
        print(json.dumps({"sweep": "reparam", "op": "head_embed", "tokens": n, "d": d, "k": k,
                          "us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                          "frac_of_measured": round(algo / us / 1e3 / peak, 3)}), flush=True)
    elif args.sweep == "dp":
        # AsyncSPARTA round steps and stage-wise clipping on one body stage of the 8B model:
        # 8.03e9 / 7 parameters in fp32, the 5 % segment of a round (229 MB, larger than L2), 4 senders
        from paper_2607_13332_b200 import dp_ops
        n_params = 8_030_261_248 // 7
        lo, hi = dp_ops.sparta_segment(n_params, 20, 7)
        seg = hi - lo
        theta = torch.randn(n_params, device="cuda", generator=gen)
        senders = 4
        chunks = [torch.randn(seg, device="cuda", generator=gen) for _ in range(senders)]
        outs = [torch.empty(seg, device="cuda") for _ in range(senders)]
        acc = torch.zeros(seg, device="cuda")
        snap = torch.empty(seg, device="cuda")
        ptr = lambda x: x.data_ptr()
        points = [
            ("sparta_snapshot", lambda: binding.sparta_snapshot(ptr(theta), lo, hi, ptr(snap)), 2 * seg * 4),
            ("sparta_accumulate", lambda: binding.sparta_accumulate(ptr(acc), ptr(chunks[0]), 0.25, seg), 3 * seg * 4),
            ("sparta_deltas, 4 senders",
             lambda: binding.sparta_deltas(ptr(acc), 1.0, [ptr(c) for c in chunks], [ptr(o) for o in outs], seg),
             (2 + 2 * senders) * seg * 4),
            ("sparta_add_delta", lambda: binding.sparta_add_delta(ptr(theta), lo, hi, ptr(outs[0])), 3 * seg * 4),
            ("sparta_apply_round", lambda: binding.sparta_apply_round(ptr(theta), lo, hi, ptr(acc), ptr(snap), 1.0),
             4 * seg * 4),
        ]
        mib = (2 << 20) // 4                                  # one 2 MiB chunk of the round's stream
        points.append(("sparta_accumulate, one 2 MiB chunk (L2-resident, launch-bound)",
                       lambda: binding.sparta_accumulate(ptr(acc), ptr(chunks[0]), 0.25, mib), 3 * mib * 4))
        for name, fn, algo in points:
            us = timed_us(fn, 10)
            print(json.dumps({"sweep": "dp", "op": name, "elements": seg if "MiB" not in name else mib,
                              "us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                              "frac_of_measured": round(algo / us / 1e3 / peak, 3)}), flush=True)
        del chunks, outs, acc, snap
        sumsq = torch.zeros(1, dtype=torch.float64, device="cuda")
        thr = binding.stage_clip_threshold(7, False)
        for tdt, code, size in ((torch.float32, binding.SSN_F32, 4), (torch.bfloat16, binding.SSN_BF16, 2)):
            grad = (theta * 1e-3).to(tdt)
            for name, fn, algo in (
                    ("stage_clip_sumsq", lambda: binding.stage_clip_sumsq(ptr(grad), n_params, code, ptr(sumsq)),
                     n_params * size),
                    ("stage_clip_scale (outside the budget: read and write)",
                     lambda: binding.stage_clip_scale(ptr(grad), n_params, code, ptr(sumsq), 1e-30),
                     2 * n_params * size),
                    ("stage_clip_scale (inside the budget: nothing to do)",
                     lambda: binding.stage_clip_scale(ptr(grad), n_params, code, ptr(sumsq), 1e30), 0)):
                sumsq.zero_()
                binding.stage_clip_sumsq(ptr(grad), n_params, code, ptr(sumsq))
                us = timed_us(fn, 5)
                print(json.dumps({"sweep": "dp", "op": name, "dtype": "f32" if size == 4 else "bf16",
                                  "elements": n_params, "us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                                  "frac_of_measured": round(algo / us / 1e3 / peak, 3)}), flush=True)
            del grad
    elif args.sweep == "wire":
        # wire rows (k fp32 coordinates + the token id) at the benchmark's stage boundary, next to the
        # storage-dtype calls of the step; ranks 24 and 40: decompress with one / two coordinate groups
        d, n = 4096, 65536
        wl = synth.STAGE_8B
        ids_np = synth.token_ids(wl, 3)
        ids = torch.from_numpy(ids_np).cuda()
        uniq = int(np.unique(ids_np).size)
        E = (torch.randn((vocab, d), device="cuda", generator=gen) * 0.02).bfloat16()
        P = to_device(synth.to_storage(synth.sinusoidal_positions(seq, d), dt), dt)
        X = torch.randn((n, d), device="cuda", generator=gen).bfloat16()
        Xh = torch.randn((n, d), device="cuda", generator=gen).bfloat16()
        Xs = torch.empty_like(X)
        for k in (24, 40):
            U = to_device(synth.to_storage(synth.subspace_basis(d, k, 1), dt), dt)
            codec, codec_t = Codec(dt, U, E, P), Codec(dt, U, E, P)
            codec_t.prepare_tables()
            wire = codec.wire_buffer(n, True)
            dZ = torch.empty((n, k), dtype=torch.float32, device="cuda")
            Z = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
            nbytes = binding.ssn_decompress_wire_workspace_bytes(codec.c, n, True)
            ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            rows_in = n * d * 2 + uniq * d * 2 + seq * d * 2 + d * k * 2 + n * 4
            points = (
                ("compress_wire", lambda: codec.compress_wire(X, ids, seq_len=seq, with_ids=True, out=wire),
                 rows_in + n * (k + 1) * 4),
                ("compress_wire, prepared tables",
                 lambda: codec_t.compress_wire(X, ids, seq_len=seq, with_ids=True, out=wire),
                 n * d * 2 + n * 4 + (uniq + seq) * k * 4 + d * k * 2 + n * (k + 1) * 4),
                ("compress (bf16 rows)", lambda: codec.compress(X, ids, seq_len=seq, out=Z), rows_in + n * k * 2),
                # the stage's last residual add fused in (X + R is never written): two reads of n x d
                ("compress_sum -> wire rows, prepared tables",
                 lambda: codec_t.compress_sum(X, Xh, ids, seq_len=seq, wire=True, with_ids=True, out=wire),
                 2 * n * d * 2 + n * 4 + (uniq + seq) * k * 4 + d * k * 2 + n * (k + 1) * 4),
                ("unfused: torch add, then compress_wire with prepared tables (same algorithmic bytes)",
                 lambda: codec_t.compress_wire(torch.add(X, Xh, out=Xs), ids, seq_len=seq, with_ids=True, out=wire),
                 2 * n * d * 2 + n * 4 + (uniq + seq) * k * 4 + d * k * 2 + n * (k + 1) * 4),
                ("grad_project_wire", lambda: codec.grad_project_wire(X, out=dZ), n * d * 2 + d * k * 2 + n * k * 4),
                ("decompress_wire",
                 lambda: codec.decompress_wire(wire, seq_len=seq, with_ids=True, out=Xh, workspace=ws),
                 n * (k + 1) * 4 + uniq * d * 2 + seq * d * 2 + d * k * 2 + n * d * 2),
                ("decompress (bf16 rows)", lambda: codec.decompress(Z, ids, seq_len=seq, out=Xh),
                 n * k * 2 + n * 4 + uniq * d * 2 + seq * d * 2 + d * k * 2 + n * d * 2),
            )
            for name, fn, algo in points:
                us = timed_us(fn, 10)
                print(json.dumps({"sweep": "wire", "op": name, "tokens": n, "d": d, "k": k, "us": round(us, 1),
                                  "GBps": round(algo / us / 1e3, 0),
                                  "frac_of_measured": round(algo / us / 1e3 / peak, 3),
                                  "status": codec.take_status() | codec_t.take_status()}), flush=True)
    else:
        d = 4096
        for k in synth.REPROJECT_RANKS:
            U = to_device(synth.to_storage(synth.subspace_basis(d, k, 1), dt), dt)
            codec = Codec(dt, U)
            for name, (rows, cols) in synth.REPROJECT_SHAPES_8B.items():
                Ws = [(torch.randn((rows, cols), device="cuda", generator=gen) * 0.02).bfloat16()
                      for _ in range(32)]
                algo = 32 * 2 * rows * cols * 2
                us = timed_us(lambda: codec.weight_reproject_rows(Ws), 5)
                out = {"sweep": "reproject", "k": k, "weight": name, "shape": [rows, cols], "layers": 32,
                       "right": {"us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                                 "frac_of_measured": round(algo / us / 1e3 / peak, 3)}}
                if rows == cols:
                    ws = codec.reproject_workspace(rows, cols, "left", 32)
                    us = timed_us(lambda: codec.weight_reproject(Ws, "left", workspace=ws), 3)
                    out["left"] = {"us": round(us, 1), "GBps": round(algo / us / 1e3, 0),
                                   "frac_of_measured": round(algo / us / 1e3 / peak, 3)}
                print(json.dumps(out), flush=True)
                del Ws


def main():
    args = parse_args()
    if args.sweep is not None:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
