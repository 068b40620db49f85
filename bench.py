"""Benchmark of the fused Ulysses QKV prologue (QK RMSNorm + 2-D RoPE + the
sequence-parallel -> head-parallel exchange, V first) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the prologue over one layer of the 21k-token workload
(P=12 virtual ranks, S=21024, H=24, D=128, bf16), through the C ABI.  N > 1
(torchrun) runs N independent replicas, one per GPU: the path has no exchange
between devices in this build.  Rank 0 prints one JSON line.

Beside the contract's keys the line carries: `repeats` (the headline loop five more
times, >= 20 ms each), `roofline` (the dominant launch timed back to back),
`e2e` (host tensors in and out through cocodiff_prologue_host), `cpu_baseline`
(the oracle on one core, on all cores, and the distance statistics between the
kernels' and the oracle's results on the sample it ran on) and `per_config`:
the other workloads (per call after an L2 flush, and back to back on rotating
buffers), the temporal workload as its eight steps (full step, selective steps,
per-token units), and the rows beyond the headline path (inverse exchange, the
two TAPA phases, the 50-step schedule, stand-alone compaction and scatter).
`--only-main`, `--only-temporal`, `--rows`, `--no-next-rows` cut the run down for
profiling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_14561_b200 import synth  # noqa: E402

METRIC = "µs/layer and achieved HBM GB/s (% of B200 peak) for fused Ulysses QKV prologue"
WORKLOAD = "qwen2304"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(cfg):
    """Every element of Q, K, V read once and written once (bf16)."""
    return 6 * cfg["S"] * cfg["H"] * cfg["D"] * 2


# ----------------------------------------------------------------- clocks ---
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------- CPU oracle ---
def oracle_sample(cfg, L, tokens, keep=False):
    """The oracle's full prologue on the first `tokens` tokens of the layer; returns the
    seconds it took (and, with keep, its three outputs)."""
    import oracle
    P, D = cfg["P"], cfg["D"]
    sl = slice(0, tokens)
    cs = oracle.rope_table_2d(L["pos"][sl], D, cfg["theta"])
    q, k, v = (np.ascontiguousarray(L[n][sl]) for n in "qkv")
    t0 = time.perf_counter()
    out = oracle.prologue(q, k, v, L["wq"], L["wk"], cfg["eps"], cs, P)
    dt = time.perf_counter() - t0
    return (dt, out) if keep else dt


def oracle_all_cores(sub, L, tokens, budget_s=5.0):
    """The same oracle source built with OpenMP, on every core this process may use."""
    import oracle
    cores = len(os.sched_getaffinity(0))
    try:
        oracle.use_all_cores(True)
        oracle_sample(sub, L, tokens)
        reps, spent = 0, 0.0
        while spent < budget_s and reps < 200:
            spent += oracle_sample(sub, L, tokens)
            reps += 1
    finally:
        oracle.use_all_cores(False)
    return {"value": algorithmic_bytes(sub) * reps / spent / 1e9, "unit": "GB/s", "cores": cores,
            "build": "the same oracle source compiled with -fopenmp", "passes": reps}


def oracle_per_config(names=("tiny", "sd3", "qwen768", "temporal")):
    """ms per layer of the oracle's full prologue on the other workloads: one core, and the
    OpenMP build on all cores (best of three)."""
    import oracle
    out = {}
    for name in names:
        cfg = synth.config(name)
        L = synth.make_layer(cfg)
        one = min(oracle_sample(cfg, L, cfg["S"]) for _ in range(2))
        try:
            oracle.use_all_cores(True)
            many = min(oracle_sample(cfg, L, cfg["S"]) for _ in range(3))
        finally:
            oracle.use_all_cores(False)
        out[name] = {"ms_one_core": 1e3 * one, "ms_all_cores": 1e3 * many}
    return out


def parity_of_sample(cfg, L, tokens, got_heads, oracle_heads):
    """Distance statistics between the kernels' Q and K and the oracle's on the sample the
    CPU baseline ran on (computed outside every timed region, with the tests' own rule)."""
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import parity_stats
    sl = slice(0, tokens)
    cs = oracle.rope_table_2d(L["pos"][sl], cfg["D"], cfg["theta"])
    out = {"tokens": tokens, "rule": "|gpu - ref| <= 2 bf16 ulp at max(|ref|, 2^-9 * magnitude of the rotated pair); "
                                    "n_strict_fail counts elements beyond 2 ulp of their own magnitude (no floor)"}
    for name, w, got, ref in (("q", L["wq"], got_heads[0], oracle_heads[0]), ("k", L["wk"], got_heads[1], oracle_heads[1])):
        _, ref_f = oracle.norm_rope(np.ascontiguousarray(L[name][sl]), w, cfg["eps"], cs, want_f32=True)
        out[name] = parity_stats(got, ref, np.ascontiguousarray(ref_f.transpose(1, 0, 2)))
    out["v_bit_exact"] = bool(np.array_equal(got_heads[2], oracle_heads[2]))
    return out


def run_reference(args):
    """The CPU oracle as it stands, on the host cores of this machine."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cfg = synth.config(WORKLOAD)
    tokens = cfg["S"] // cfg["P"]                    # one rank's shard: 1752 tokens, still P | tokens
    assert tokens % cfg["P"] == 0
    sub = dict(cfg, S=tokens)
    E = tokens * cfg["H"] * cfg["D"]
    L = {n: synth.normal_bf16(cfg["seed"], n, E).reshape(tokens, cfg["H"], cfg["D"]) for n in "qkv"}
    L["wq"] = synth.normal_bf16(cfg["seed"], "wq", cfg["D"], 1.0, 0.1)
    L["wk"] = synth.normal_bf16(cfg["seed"], "wk", cfg["D"], 1.0, 0.1)
    L["pos"] = synth.positions(*cfg["grid"], cfg["n_text"])[:tokens]
    for _ in range(args.warmup):
        oracle_sample(sub, L, tokens)
    t = [oracle_sample(sub, L, tokens) for _ in range(args.steps)]
    total = sum(t)
    bytes_per_step = algorithmic_bytes(sub)
    gbs = bytes_per_step * args.steps / total / 1e9
    sample = f"first {tokens} of {cfg['S']} tokens (one rank's shard) of the {WORKLOAD} layer per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "us_per_layer_extrapolated": 1e6 * total / args.steps * cfg["S"] / tokens,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "storage_dtype": "bf16",
        "data": "synthetic", "config": {"workload": WORKLOAD, "P": cfg["P"], "S": cfg["S"], "H": cfg["H"],
                                        "D": cfg["D"], "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line, ensure_ascii=False))


# --------------------------------------------------------------- GPU path ---
def dev(a, torch):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


def time_steps(torch, fn, stream, steps, warmup, flush=None):
    """CUDA events on `stream` around every step; returns per-step ms."""
    for _ in range(warmup):
        if flush is not None:
            flush()
        fn()
    stream.synchronize()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        if flush is not None:
            flush()
        a.record(stream)
        fn()
        b.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in ev]


def time_loop(torch, fn, stream, steps, warmup=3):
    """`steps` calls back to back between two CUDA events on `stream`; ms per call."""
    for _ in range(warmup):
        fn()
    stream.synchronize()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        fn()
    b.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


def time_graph(torch, fn, stream, steps, flush=None):
    """Capture one call of `fn` (already warmed up) into a CUDA graph on `stream`
    and time its replays; returns per-replay ms, or None if capture is refused."""
    try:
        g = torch.cuda.CUDAGraph()
        stream.synchronize()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=stream):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        with torch.cuda.stream(stream):
            for a, b in ev:
                if flush is not None:
                    flush()
                a.record(stream)
                g.replay()
                b.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]
    except Exception as exc:                      # capture not possible: report, do not fail the bench
        sys.stderr.write(f"graph capture skipped: {exc}\n")
        return None


def time_graph_loop(torch, fn, stream, calls, replays):
    """`calls` consecutive calls of `fn` captured into one CUDA graph (no host work between the
    launches), replayed `replays` times between two events; ms per call, median of 5; None if
    capture is refused."""
    try:
        for _ in range(calls):
            fn()
        stream.synchronize()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(calls):
                fn()
        torch.cuda.synchronize()
        out = []
        with torch.cuda.stream(stream):
            g.replay()
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(replays):
                    g.replay()
                b.record(stream)
                stream.synchronize()
                out.append(a.elapsed_time(b) / (replays * calls))
        torch.cuda.synchronize()
        return statistics.median(out)
    except Exception as exc:
        sys.stderr.write(f"graph capture skipped: {exc}\n")
        return None


def max_over_ranks(ms, world, device):
    """The slowest rank's time: every multi-GPU number is the max over ranks."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(step_bytes, world, ms_per_step):
    """Whole-job throughput of `world` independent replicas (weak scaling)."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2604_14561_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for this path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        from paper_2604_14561_b200 import build as cuda_build
        cuda_build.build()            # no-op when libcocodiff.so is newer than its sources
    if world > 1:
        dist.barrier()
    binding.lib()

    cfg = synth.config(WORKLOAD)
    P, S, H, D = cfg["P"], cfg["S"], cfg["H"], cfg["D"]
    E = S * H * D
    L = synth.make_layer(cfg)
    q, k, v = (dev(L[n], torch) for n in "qkv")
    wq, wk = dev(L["wq"], torch), dev(L["wk"], torch)
    cs = torch.empty((S, D // 2, 2), dtype=torch.float32, device="cuda")
    binding.rope_table_2d(cs, dev(L["pos"], torch), S, D, cfg["theta"])
    qh, kh, vh = (torch.empty(E, dtype=torch.int16, device="cuda") for _ in range(3))
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    step_bytes = algorithmic_bytes(cfg)
    peak, peak_kind = measured_peak()

    # The headline is V-first on ONE stream: V's launch, then Q/K's as its programmatic dependent; and a
    # call's first kernel is the programmatic dependent of the previous call's last one, so consecutive
    # layers overlap launch, ramp-up and drain while every kernel still waits for its predecessor
    # before it touches memory.  (The same order on two streams, joined by events, is a row of `orders`.)
    def step(order, two_streams=False):
        binding.prologue(q, k, v, qh, kh, vh, wq, wk, cfg["eps"], cs, P, S, H, D, order=order,
                         stream_qk=sq, stream_v=sv if two_streams else sq)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- headline: the V-first order, K steps back to back ------------------
    for _ in range(max(args.warmup, 3)):
        step(binding.V_FIRST)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record(sq)
    for _ in range(args.steps):
        step(binding.V_FIRST)
    stop.record(sq)
    barrier()
    total_ms = start.elapsed_time(stop)
    if rank == 0:
        # keep the sampler running a little longer so that short runs still get samples under load
        t_end = time.time() + 0.6
        while time.time() < t_end:
            step(binding.V_FIRST)
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(total_ms, world, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_gbs(step_bytes, world, ms_per_step)
    # the same back-to-back loop five more times, each at least 20 ms long whatever --steps says
    rep_steps = max(args.steps, int(np.ceil(20.0 / ms_per_step)))
    rep_ms = []
    for _ in range(5):
        barrier()
        start.record(sq)
        for _ in range(rep_steps):
            step(binding.V_FIRST)
        stop.record(sq)
        barrier()
        rep_ms.append(max_over_ranks(start.elapsed_time(stop), world, "cuda") / rep_steps)
    graph_ms = time_graph_loop(torch, lambda: step(binding.V_FIRST), sq, 10, replays=max(2, rep_steps // 10)) if (world == 1 and not args.only_main) else None
    repeats = {"n": 5, "steps_each": rep_steps, "us_per_layer_median": 1e3 * statistics.median(rep_ms),
               "us_per_layer_as_one_cuda_graph_of_10_steps": None if graph_ms is None else 1e3 * graph_ms,
               "us_per_layer_min": 1e3 * min(rep_ms), "us_per_layer_max": 1e3 * max(rep_ms),
               "gbs_median": aggregate_gbs(step_bytes, world, statistics.median(rep_ms))}

    line = None
    if rank == 0 and args.only_main:
        line = {"metric": METRIC, "value": value, "unit": "GB/s", "us_per_layer": 1e3 * ms_per_step,
                "n_gpus": world, "steps": args.steps, "note": "--only-main: headline loop only", "clocks": clocks}
    elif rank == 0:
        # ---- per-order detail, per-step events (this GPU only) --------------
        orders = {}
        for name, order, two in (("v_first", binding.V_FIRST, False), ("v_first_two_streams", binding.V_FIRST, True),
                                 ("lump", binding.LUMP, False)):
            ms = time_steps(torch, lambda: step(order, two), sq, args.steps, 3)
            loop = [time_loop(torch, lambda: step(order, two), sq, rep_steps) for _ in range(5)]
            orders[name] = {"us_median": 1e3 * statistics.median(ms), "us_min": 1e3 * min(ms),
                            "gbs_median": step_bytes / (statistics.median(ms) * 1e-3) / 1e9,
                            "us_back_to_back_median": 1e3 * statistics.median(loop), "us_back_to_back_min": 1e3 * min(loop),
                            "gbs_back_to_back": step_bytes / (statistics.median(loop) * 1e-3) / 1e9,
                            "launches_per_step": 2 if order == binding.V_FIRST else 1}
        orders["note"] = ("us_median: one call between two events; us_back_to_back: the loop of `repeats`.  v_first = V's launch, "
                          "then Q/K's as its programmatic dependent on one stream (the headline); v_first_two_streams = the same "
                          "two launches on two streams joined by events (no dependent launches across the join)")
        # V-first evidence: V's exchange and the Q/K launch issued as two calls with their own events
        ev = {n: torch.cuda.Event(enable_timing=True) for n in ("v0", "v1", "qk0", "qk1")}
        timeline = []
        for _ in range(10):
            torch.cuda.synchronize()
            ev["v0"].record(sv)
            binding.prologue(None, None, v, None, None, vh, None, None, cfg["eps"], None, P, S, H, D,
                             order=binding.LUMP, stream_qk=sv, stream_v=sv)
            ev["v1"].record(sv)
            ev["qk0"].record(sq)
            binding.prologue(q, k, None, qh, kh, None, wq, wk, cfg["eps"], cs, P, S, H, D,
                             order=binding.LUMP, stream_qk=sq, stream_v=sq)
            ev["qk1"].record(sq)
            torch.cuda.synchronize()
            timeline.append((ev["v0"].elapsed_time(ev["v1"]), ev["v0"].elapsed_time(ev["qk0"]),
                             ev["v0"].elapsed_time(ev["qk1"])))
        timeline.sort(key=lambda t: t[2])
        mid = timeline[len(timeline) // 2]
        v_first_timeline = {"v_start_us": 0.0, "v_end_us": 1e3 * mid[0], "qk_start_us": 1e3 * mid[1],
                            "qk_end_us": 1e3 * mid[2],
                            "note": "V is launched first on its own stream and completes first; Q/K (norm + RoPE) run beside it"}

        # dominant kernel of the headline loop: the norm + RoPE + exchange launch over Q and K
        # (two thirds of the bytes), timed alone on its stream
        def qk_only():
            binding.prologue(q, k, None, qh, kh, None, wq, wk, cfg["eps"], cs, P, S, H, D, order=binding.V_FIRST,
                             stream_qk=sq, stream_v=sv)
        qk_ms = time_loop(torch, qk_only, sq, args.steps)
        qk_bytes = step_bytes * 2 // 3
        achieved = qk_bytes / (qk_ms * 1e-3) / 1e9

        # context: the library's plain device copy of the same two tensors in the same back-to-back loop
        def torch_copy():
            with torch.cuda.stream(sq):
                qh.copy_(q.reshape(-1))
                kh.copy_(k.reshape(-1))
        copy_ms = time_loop(torch, torch_copy, sq, args.steps)
        roofline = {"bound": "hbm", "kernel": "move_rows_kernel<LPR=16, KIND_NORM> (Q and K: RMSNorm + RoPE + exchange, one launch)",
                    "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                    "frac": achieved / peak, "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                    "us_per_launch": 1e3 * qk_ms, "algorithmic_bytes_per_launch": qk_bytes,
                    "same_loop_torch_copy_of_the_same_bytes": {"us": 1e3 * copy_ms, "gbs": qk_bytes / (copy_ms * 1e-3) / 1e9,
                                                                "note": "two tensor.copy_ calls (no norm, no rotation, no permutation) timed like the kernel"},
                    "traffic": read_traffic_note(),
                    "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of this kernel on this "
                                      "workload, read from profiles/move_rows_kernel_qwen2304.md (not measured in this run)"}

        # ---- end to end: host buffers in, host buffers out ------------------
        hin = [torch.from_numpy(L[n].view(np.int16)).pin_memory() for n in "qkv"]
        hout = [torch.empty(E, dtype=torch.int16).pin_memory() for _ in range(3)]
        dev_in = torch.empty(3 * E, dtype=torch.int16, device="cuda")
        dev_out = torch.empty(3 * E, dtype=torch.int16, device="cuda")

        def e2e_step():
            binding.prologue_host(*hin, *hout, dev_in, dev_out, wq, wk, cfg["eps"], cs, P, S, H, D,
                                  order=binding.V_FIRST, stream_qk=sq, stream_v=sv)
        e2e_steps = max(3, min(args.steps, 10))
        e2e_ms = statistics.mean(time_steps(torch, e2e_step, sq, e2e_steps, 2))
        e2e = {"value": step_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": 3 * E * 2, "d2h_bytes_per_step": 3 * E * 2,
               "api": "cocodiff_prologue_host (pinned host tensors in and out)"}
        del hin, hout, dev_in, dev_out

        per_config = other_configs(torch, binding, args)
        per_config["temporal_steps"] = temporal_rows(torch, binding, args)
        per_config["next_rows_temporal"] = next_rows(torch, binding, args)
        # the selective step's parts as stand-alone calls (each between two events after an L2 flush, so each
        # carries the event-to-event floor): what the fused pass replaces
        nr, ts = per_config["next_rows_temporal"], per_config["temporal_steps"]
        parts = {"metric_and_selection": ts["metric_pass_context"]["us_metric_and_selection_alone"],
                 "pack_active_qkv": nr["pack_active_qkv_standalone"]["us_cold_l2"],
                 "unpack_qkv": nr["unpack_qkv_receiver_only"]["us_cold_l2"]}
        parts["sum"] = sum(parts.values())
        parts["fused_step"] = min(ts["steps_1_to_7_selective"]["us_mean"].values())
        ts["steps_1_to_7_selective"]["break_out_as_stand_alone_calls_us"] = parts

        # ---- the oracle on this machine's host cores, bounded sample ------------
        import oracle
        oracle.build()
        tokens = S // P
        sub = dict(cfg, S=tokens)
        _, oracle_heads = oracle_sample(sub, L, tokens, keep=True)     # also warms the page cache / allocator
        reps, spent = 0, 0.0
        while spent < 10.0 and reps < 40:
            spent += oracle_sample(sub, L, tokens)
            reps += 1
        cpu_gbs = algorithmic_bytes(sub) * reps / spent / 1e9
        step(binding.V_FIRST)
        torch.cuda.synchronize()
        got_heads = [t.view(H, S, D)[:, :tokens].contiguous().cpu().numpy().view(np.uint16) for t in (qh, kh, vh)]
        cpu = {"value": cpu_gbs, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "ms_per_layer_extrapolated": 1e3 * spent / reps * S / tokens,
               "sample": f"{reps} passes over the first {tokens} of {S} tokens (one rank's shard) of the same layer",
               "all_cores": oracle_all_cores(sub, L, tokens),
               "other_workloads_ms_per_layer": oracle_per_config(),
               "parity_on_sample": parity_of_sample(cfg, L, tokens, got_heads, oracle_heads)}

        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "us_per_layer": 1e3 * ms_per_step,
            "frac_of_nominal_8000": value / world / NOMINAL_HBM_GBS, "frac_of_measured_copy": value / world / peak,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "storage_dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "P": P, "S": S, "H": H, "D": D, "order": "v_first",
                       "streams": "one: V's launch, then Q/K's as its programmatic dependent; consecutive calls are chained the same way",
                       "algorithmic_bytes_per_step": step_bytes, "l2": "inputs and outputs (775 MB per step) exceed the 126 MB L2",
                       "replicas": world},
            "gpu_launches": 2 * args.steps,
            "repeats": repeats,
            "clocks": clocks, "orders": orders, "v_first_timeline": v_first_timeline, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu,
            "per_config": per_config,
        }
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line, ensure_ascii=False))


def read_traffic_note():
    """DRAM bytes per launch of the dominant kernel, from the committed ncu summary."""
    import re
    path = os.path.join(ROOT, "profiles", "move_rows_kernel_qwen2304.md")
    try:
        with open(path) as f:
            m = re.search(r"traffic_bytes_per_launch\(move_rows_norm_qwen2304\)\s*=\s*(\d+)", f.read())
        return int(m.group(1)) if m else None
    except OSError:
        return None


class Flusher:
    """Between timed iterations: write a buffer four times the L2, then read it back.  The L2
    ends up full of clean foreign lines, so the timed region neither hits in L2 nor pays for
    the write-back of the flush's own dirty lines."""

    def __init__(self, torch, stream):
        self.torch, self.stream = torch, stream
        self.scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        self.sink = torch.zeros(1, dtype=torch.int64, device="cuda")

    def __call__(self):
        with self.torch.cuda.stream(self.stream):
            self.scratch.zero_()
            self.torch.sum(self.scratch.view(self.torch.int64), dim=0, keepdim=True, out=self.sink)


def launch_floor(torch, binding, sq, flush, iters):
    """What one launch costs between two events, whatever it moves: the same prologue call on
    16 tokens of one head (8 KB), timed with the same protocol as the small workloads."""
    S, H, D = 16, 1, 128
    x = [torch.zeros(S * H * D, dtype=torch.int16, device="cuda") for _ in range(6)]
    w = torch.full((D,), 0x3F80, dtype=torch.int16, device="cuda")
    cs = torch.zeros((S, D // 2, 2), dtype=torch.float32, device="cuda")
    cs[..., 0] = 1.0

    def call():
        binding.prologue(x[0], x[1], x[2], x[3], x[4], x[5], w, w, 1e-6, cs, 1, S, H, D, order=binding.LUMP,
                         stream_qk=sq, stream_v=sq)
    return 1e3 * statistics.median(time_steps(torch, call, sq, iters, 3, flush=flush))


def other_configs(torch, binding, args, names=("tiny", "sd3", "qwen768", "temporal")):
    """µs/layer of the other synthetic workloads, L2 flushed between iterations.  They fit in
    the 126 MB L2, so part of their output is still dirty in the L2 when the timed region ends:
    the GB/s given for them is effective throughput (algorithmic bytes / time), not HBM traffic."""
    out = {}
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    flush = Flusher(torch, sq)
    iters = max(10, min(args.steps, 50))
    floor = launch_floor(torch, binding, sq, flush, iters)
    out["launch_floor"] = {"us": floor, "what": "median event-to-event time of one prologue launch that moves 8 KB, same "
                                                "flush-and-events protocol: the fixed cost inside every per_config figure"}
    # v_first: V's launch, then Q/K's as its programmatic dependent, on one stream (consecutive calls chain
    # the same way: best back to back); v_first_two_streams: the two launches start side by side on two
    # streams joined by events (best for a single call between two events); lump: one launch
    ORDERS3 = (("v_first", binding.V_FIRST, False), ("v_first_two_streams", binding.V_FIRST, True), ("lump", binding.LUMP, False))
    for name in names:
        cfg = synth.config(name)
        P, S, H, D = cfg["P"], cfg["S"], cfg["H"], cfg["D"]
        E = S * H * D
        L = synth.make_layer(cfg)
        q, k, v = (dev(L[n], torch) for n in "qkv")
        wq, wk = dev(L["wq"], torch), dev(L["wk"], torch)
        cs = torch.empty((S, D // 2, 2), dtype=torch.float32, device="cuda")
        binding.rope_table_2d(cs, dev(L["pos"], torch), S, D, cfg["theta"])
        qh, kh, vh = (torch.empty(E, dtype=torch.int16, device="cuda") for _ in range(3))

        def full(order, two=False):
            binding.prologue(q, k, v, qh, kh, vh, wq, wk, cfg["eps"], cs, P, S, H, D,
                             order=order, stream_qk=sq, stream_v=sv if two else sq)
        b = algorithmic_bytes(cfg)
        out[name] = {"bytes": b, "fits_in_l2": b < 126e6 * 2}
        for oname, order, two in ORDERS3:
            cold_all = time_steps(torch, lambda: full(order, two), sq, iters, 10, flush=flush)
            cold = statistics.median(cold_all)
            warm = statistics.median(time_steps(torch, lambda: full(order, two), sq, iters, 10))
            out[name][oname] = {"us_cold_l2": 1e3 * cold, "us_cold_l2_min": 1e3 * min(cold_all), "iterations": iters,
                                "gbs_effective_cold_l2": b / (cold * 1e-3) / 1e9, "us_warm_l2": 1e3 * warm}
            gr = time_graph(torch, lambda: full(order, two), sq, iters, flush=flush)
            if gr is not None:
                out[name][oname]["us_cold_l2_cuda_graph"] = 1e3 * statistics.median(gr)
        if name != "temporal":
            # Layers back to back on rotating buffer sets: no event or flush between the calls, and
            # the sets together exceed four times the L2 (when memory allows), so that every call
            # reads from HBM and the write-back of its output falls inside the timed region.
            n_sets = max(2, min(64, int(np.ceil(4 * 126e6 / b)) + 1))
            sets = [([t.clone() for t in (q, k, v)], [torch.empty_like(qh) for _ in range(3)]) for _ in range(n_sets)]
            for oname, order, two in ORDERS3:
                calls = [0]

                def rotating():
                    (a, c, d), (x, y, z) = sets[calls[0] % n_sets]
                    calls[0] += 1
                    binding.prologue(a, c, d, x, y, z, wq, wk, cfg["eps"], cs, P, S, H, D, order=order,
                                     stream_qk=sq, stream_v=sv if two else sq)
                rounds = max(1, -(-32 // n_sets))      # at least 32 calls per graph: a replay boundary breaks the chain of launches
                ms = time_graph_loop(torch, rotating, sq, n_sets * rounds, replays=10)
                if ms is None:
                    continue
                out[name][oname]["back_to_back_rotating_buffers"] = {
                    "us_per_layer": 1e3 * ms, "gbs": b / (ms * 1e-3) / 1e9, "buffer_sets": n_sets, "calls_per_graph": n_sets * rounds,
                    "how": "one CUDA graph of calls_per_graph consecutive calls walking the buffer sets, replayed 10 times between two events (median of 5)",
                    "working_set_bytes": n_sets * b, "exceeds_4x_l2": bool(n_sets * b >= 4 * 126e6)}
            del sets
        del q, k, v, qh, kh, vh
    return out


def temporal_rows(torch, binding, args):
    """The temporal workload as its eight denoising steps (step t+1 = step t + N(0, 1e-3)
    everywhere + N(0, 0.5) on a fifth of the 64-token tiles, re-drawn every step): step 0 is a
    full exchange that fills the caches, steps 1-7 are selective steps at r = 0.8 against
    prev_v = V of the step before.  Every step is timed on its own (cold L2, median)."""
    cfg = synth.config("temporal")
    P, S, H, D, T, r, n_groups = cfg["P"], cfg["S"], cfg["H"], cfg["D"], cfg["T"], cfg["r"], cfg["n_groups"]
    E, n = S * H * D, S // T
    seq = synth.TemporalSequence(cfg)
    steps = []
    for t in range(cfg["steps"]):
        if t:
            seq.advance()
        cur = seq.current()
        steps.append({x: dev(cur[x], torch) for x in "qkv"})
    wq, wk = dev(seq.wq, torch), dev(seq.wk, torch)
    cs = torch.empty((S, D // 2, 2), dtype=torch.float32, device="cuda")
    binding.rope_table_2d(cs, dev(seq.pos, torch), S, D, cfg["theta"])
    new = lambda: torch.empty(E, dtype=torch.int16, device="cuda")
    cache, comp = [new() for _ in range(3)], [new() for _ in range(3)]
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    metric = torch.zeros(S, dtype=torch.int64, device="cuda")
    mask = torch.zeros(S, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(S, dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    flush = Flusher(torch, sq)
    iters = max(10, min(args.steps, 30))
    tile = T * H * D * 2

    def full_step(order):
        x = steps[0]
        binding.prologue(x["q"], x["k"], x["v"], *cache, wq, wk, cfg["eps"], cs, P, S, H, D, order=order,
                         stream_qk=sq, stream_v=sv)

    def selective(t, order, T_=T, groups=n_groups, direct=False):
        x, prev = steps[t], steps[t - 1]["v"]
        binding.selective_prologue(prev, x["q"], x["k"], x["v"], wq, wk, cfg["eps"], cs, P, S, H, D, T_, r, groups,
                                   metric, mask, idx, na, *([None] * 3 if direct else comp), *cache,
                                   ws, binding.vmajor_workspace_bytes(P, S, H, D, T_), order=order,
                                   stream_qk=sq, stream_v=sv if order == binding.V_FIRST else sq)
    out = {"workload": "temporal: P=24, S=9216, H=24, D=128, T=64, r=0.8, one global group; 8 steps of the data law",
           "l2": "flushed (write + read of 512 MB) before every timed call",
           "statistic": "mean over the timed iterations of a step (event stamps are quantised to about 2 µs); medians beside it"}
    fb = 6 * E * 2
    t_full = {o: 1e3 * statistics.mean(time_steps(torch, lambda: full_step(order), sq, iters, 3, flush=flush))
              for o, order in (("v_first", binding.V_FIRST), ("lump", binding.LUMP))}
    out["step_0_full"] = {"us_cold_l2": t_full, "bytes": fb, "gbs_best": fb / (min(t_full.values()) * 1e-6) / 1e9}
    # CUDA-event stamps on this platform move in steps of about 2 µs, so a single timing is one of
    # two neighbouring values; the mean over the iterations resolves what the median cannot
    per_step = []
    for t in range(1, cfg["steps"]):
        row = {"step": t}
        for o, order in (("lump", binding.LUMP), ("v_first", binding.V_FIRST)):
            ts = time_steps(torch, lambda: selective(t, order), sq, iters, 3, flush=flush)
            row["us_" + o] = 1e3 * statistics.mean(ts)
            row["us_median_" + o] = 1e3 * statistics.median(ts)
        row["n_active"] = int(na.item())
        per_step.append(row)
    n_act = per_step[0]["n_active"]
    b_alg = 2 * E * 2 + 12 * n_act * tile          # metric pass + compaction (read, write) + scatter (read, write)
    b_moved = 2 * E * 2 + 9 * n_act * tile         # gather and scatter in one pass: one read, two writes per active row
    mean = {o: statistics.mean(row["us_" + o] for row in per_step) for o in ("lump", "v_first")}
    best = min(mean.values())
    peak, _ = measured_peak()
    out["steps_1_to_7_selective"] = {
        "per_step": per_step, "us_mean": mean, "n_units": n, "n_active": n_act,
        "algorithmic_bytes": b_alg, "bytes_moved_by_the_fused_pass": b_moved,
        "gbs_on_algorithmic_bytes": b_alg / (best * 1e-6) / 1e9, "gbs_on_bytes_moved": b_moved / (best * 1e-6) / 1e9,
        "frac_of_measured_copy_peak": {"on_algorithmic_bytes": b_alg / (best * 1e-6) / 1e9 / peak,
                                       "on_bytes_moved": b_moved / (best * 1e-6) / 1e9 / peak},
        "launches_per_step": {"lump": 2, "v_first": 3},
        "kernel_break_out": "per-kernel durations of these same launches: profiles/vmajor_selective_step_temporal.md (ncu)",
        "api": "cocodiff_selective_prologue"}
    # Direct delivery: no compact buffers, the active rows are stored straight to their slots of the
    # cached tensors (what a sender does over NVLink peer memory); one read and one write per active row.
    td = [1e3 * statistics.mean(time_steps(torch, lambda: selective(t, binding.LUMP, direct=True), sq, iters, 3, flush=flush))
          for t in range(1, cfg["steps"])]
    b_direct = 2 * E * 2 + 6 * n_act * tile
    out["steps_1_to_7_selective_direct_delivery"] = {
        "us_per_step": td, "us_mean": statistics.mean(td), "algorithmic_bytes": b_direct,
        "gbs_on_algorithmic_bytes": b_direct / (statistics.mean(td) * 1e-6) / 1e9,
        "frac_of_measured_copy_peak": b_direct / (statistics.mean(td) * 1e-6) / 1e9 / peak,
        "note": "cocodiff_selective_prologue with the three compact buffers NULL: metric pass (2 tensors read) + "
                "active rows of Q, K, V read once and written once; the caches receive the same bits as above"}
    # the metric pass and its selection alone (no compaction follows, so the selection is a launch of
    # its own), and - for context - a library read-only reduction over the same two tensors
    def metric_alone():
        binding.vmajor_select_compact(steps[0]["v"], steps[1]["v"], P, S, H, D, T, r, n_groups, metric, mask, idx, na, None,
                                      ws, binding.vmajor_workspace_bytes(P, S, H, D, T), stream=sq)
    sink = torch.zeros(2, dtype=torch.int64, device="cuda")

    def torch_read_only():
        with torch.cuda.stream(sq):
            torch.sum(steps[0]["v"].reshape(-1).view(torch.int64), dim=0, keepdim=True, out=sink[0:1])
            torch.sum(steps[1]["v"].reshape(-1).view(torch.int64), dim=0, keepdim=True, out=sink[1:2])
    out["metric_pass_context"] = {
        "bytes": 2 * E * 2,
        "us_metric_and_selection_alone": 1e3 * statistics.mean(time_steps(torch, metric_alone, sq, iters, 3, flush=flush)),
        "us_torch_sum_of_the_same_two_tensors": 1e3 * statistics.mean(time_steps(torch, torch_read_only, sq, iters, 3, flush=flush)),
        "note": "both between two events after an L2 flush; the library reduction (two launches) reads the same 113 MB"}
    gr = time_graph(torch, lambda: selective(1, binding.LUMP), sq, iters, flush=flush)
    if gr is not None:
        out["steps_1_to_7_selective"]["us_step_1_lump_cuda_graph"] = 1e3 * statistics.median(gr)
    # the paper's own granularity on the same data: per-token units (T = 1), step 1
    for groups in (1, P):
        t1 = 1e3 * statistics.mean(time_steps(torch, lambda: selective(1, binding.LUMP, 1, groups), sq, iters, 3, flush=flush))
        n_act1 = int(na.item())
        b1 = 2 * E * 2 + 12 * n_act1 * H * D * 2
        out[f"step_1_per_token_units_groups{groups}"] = {
            "us_cold_l2": t1, "n_units": S, "n_active": n_act1, "algorithmic_bytes": b1,
            "gbs_on_algorithmic_bytes": b1 / (t1 * 1e-6) / 1e9, "ratio_to_64_token_tiles": t1 / per_step[0]["us_lump"],
            "launches_per_step": 3}
    # Selective steps back to back on two rotating buffer sets (1.1 GB together, more than four times
    # the L2), captured as one CUDA graph: no event, flush or host work between the steps.  This is
    # also the only figure here that the 2 µs grain of the event stamps does not touch.
    sets = [(steps[t - 1]["v"], steps[t], [new() for _ in range(3)], [new() for _ in range(3)]) for t in (1, 2)]

    def rotating_loop(T_, groups, direct=False):
        calls = [0]

        def rotating():
            prev, x, cmp_, cch = sets[calls[0] % 2]
            calls[0] += 1
            binding.selective_prologue(prev, x["q"], x["k"], x["v"], wq, wk, cfg["eps"], cs, P, S, H, D, T_, r, groups,
                                       metric, mask, idx, na, *([None] * 3 if direct else cmp_), *cch, ws,
                                       binding.vmajor_workspace_bytes(P, S, H, D, T_),
                                       order=binding.LUMP, stream_qk=sq, stream_v=sq)
        return time_graph_loop(torch, rotating, sq, 16, replays=5)
    how = "one CUDA graph of 16 consecutive steps alternating between two buffer sets, replayed 5 times (median of 5)"
    ms = rotating_loop(T, n_groups)
    if ms is not None:
        out["steps_1_to_7_selective"]["back_to_back_rotating_buffers"] = {
            "us_per_step": 1e3 * ms, "gbs_on_algorithmic_bytes": b_alg / (ms * 1e-3) / 1e9,
            "gbs_on_bytes_moved": b_moved / (ms * 1e-3) / 1e9, "frac_of_measured_copy_peak_on_bytes_moved": b_moved / (ms * 1e-3) / 1e9 / peak,
            "how": how}
        msd = rotating_loop(T, n_groups, direct=True)
        if msd is not None:
            out["steps_1_to_7_selective_direct_delivery"]["back_to_back_rotating_buffers"] = {
                "us_per_step": 1e3 * msd, "gbs_on_algorithmic_bytes": b_direct / (msd * 1e-3) / 1e9,
                "frac_of_measured_copy_peak": b_direct / (msd * 1e-3) / 1e9 / peak, "how": how}
        for groups in (1, P):
            ms1 = rotating_loop(1, groups)
            if ms1 is not None:
                out[f"step_1_per_token_units_groups{groups}"]["back_to_back_rotating_buffers"] = {
                    "us_per_step": 1e3 * ms1, "ratio_to_64_token_tiles": ms1 / ms, "how": how}
    del sets
    return out


def next_rows(torch, binding, args, rows=("inverse", "tapa", "schedule", "moves")):
    """Rows beyond the headline path, on the temporal workload (P=24, S=9216, H=24, D=128):
    inverse exchange, the two TAPA phases, and the paper's 50-step cache schedule (5 warm-up
    steps, refresh every 10 steps, linear cache ratio)."""
    cfg = synth.config("temporal")
    P, S, H, D = cfg["P"], cfg["S"], cfg["H"], cfg["D"]
    E = S * H * D
    L = synth.make_layer(cfg)
    q, k, v = (dev(L[n], torch) for n in "qkv")
    wq, wk = dev(L["wq"], torch), dev(L["wk"], torch)
    cs = torch.empty((S, D // 2, 2), dtype=torch.float32, device="cuda")
    binding.rope_table_2d(cs, dev(L["pos"], torch), S, D, cfg["theta"])
    new = lambda n=1: torch.empty(n * E, dtype=torch.int16, device="cuda")
    qh, kh, vh = new(), new(), new()
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    flush = Flusher(torch, sq)

    iters = max(10, min(args.steps, 30))
    out = {}

    def timed(name, fn, nbytes):
        t = statistics.median(time_steps(torch, fn, sq, iters, 3, flush=flush))
        out[name] = {"us_cold_l2": 1e3 * t, "bytes": nbytes, "gbs": nbytes / (t * 1e-3) / 1e9}

    binding.prologue(q, k, v, qh, kh, vh, wq, wk, cfg["eps"], cs, P, S, H, D, order=binding.LUMP, stream_qk=sq, stream_v=sq)
    if "inverse" in rows:
        back = [new() for _ in range(3)]
        timed("inverse_a2a", lambda: binding.ulysses_a2a_inverse(qh, kh, vh, *back, P, S, H, D, stream=sq), 6 * E * 2)
        del back
    if "tapa" in rows:
        p1 = [new(2) for _ in range(3)]
        th = [new() for _ in range(3)]
        timed("tapa_phase1", lambda: binding.tapa_phase1(q, k, v, *p1, P, S, H, D, stream=sq), 9 * E * 2)
        out["tapa_phase1"]["note"] = "every shard is read once and written to both rings' holdings: 3 tensors x (1 read + 2 writes)"
        timed("tapa_phase2", lambda: binding.tapa_phase2(*p1, *th, P, S, H, D, stream=sq), 6 * E * 2)
        del p1, th

    comp = [new() for _ in range(3)]

    # the 50-step schedule on 64-token tiles, inputs fixed (timing only), back to back
    T, total, warmup, interval = cfg["T"], 50, 5, 10
    n = S // T
    ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    metric = torch.zeros(n, dtype=torch.int64, device="cuda")
    mask = torch.zeros(n, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(n, dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    if "schedule" in rows:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(total + 1)]
        full = [binding.cache_schedule(i, total, warmup, interval)[0] for i in range(total)]
        for name, bufs in (("schedule_50_steps", comp), ("schedule_50_steps_direct_delivery", [None] * 3)):
            for rep in range(2):                 # first pass warms up
                sent = []
                torch.cuda.synchronize()
                ev[0].record(sq)
                for step_i in range(total):
                    _, s_el = binding.layer_step(step_i, total, warmup, interval, v, q, k, v, wq, wk,
                                                 cfg["eps"], cs, P, S, H, D, T, 1, metric, mask, idx, na, *bufs,
                                                 qh, kh, vh, ws, ws_bytes, order=binding.LUMP, stream_qk=sq, stream_v=sq)
                    sent.append(s_el)
                    ev[step_i + 1].record(sq)
                torch.cuda.synchronize()
            per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(total)]
            out[name] = {
                "total_us": 1e3 * sum(per_step),
                "always_full_us_estimate": 1e3 * total * statistics.mean(t for t, f in zip(per_step, full) if f),
                "full_steps": sum(full), "us_full_step_mean": 1e3 * statistics.mean(t for t, f in zip(per_step, full) if f),
                "us_selective_step_mean": 1e3 * statistics.mean(t for t, f in zip(per_step, full) if not f),
                "exchanged_fraction_of_always_full": sum(sent) / (total * 3 * E), "l2": "warm (steps back to back)"}
        out["schedule_50_steps"]["note"] = (
            "on one device a selective step is sender and receiver at once: metric pass + active rows read once and "
            "written twice (send buffer and cache), so it moves fewer bytes than a full step only for r > 0.56; "
            "with direct delivery (no send buffer) for r > 0.33")
    if "moves" not in rows:
        return out
    # the stand-alone compaction and the receiver-only scatter of 29 of 144 units (the selective step
    # itself moves its rows in one fused pass; these calls launch a worst-case grid because the host
    # does not know n_active, and the blocks beyond the active units return at once)
    binding.vmajor_select_compact(v, v, P, S, H, D, T, 0.8, 1, metric, mask, idx, na, None, ws, ws_bytes, stream=sq)
    torch.cuda.synchronize()
    moved = 6 * int(na.item()) * T * H * D * 2
    timed("pack_active_qkv_standalone", lambda: binding.pack_active_qkv(q, k, v, wq, wk, cfg["eps"], cs, idx, na, *comp,
                                                                         P, S, H, D, T, stream=sq), moved)
    timed("unpack_qkv_receiver_only", lambda: binding.unpack_qkv(*comp, idx, na, qh, kh, vh, P, S, H, D, T, stream=sq), moved)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only-main", action="store_true",
                    help="run only the headline loop (short launch list for profiling)")
    ap.add_argument("--only-temporal", action="store_true",
                    help="run only the temporal workload (its eight steps, then the rows beyond the headline path), for profiling")
    ap.add_argument("--no-next-rows", action="store_true", help="with --only-temporal: the eight steps only")
    ap.add_argument("--rows", nargs="+", default=None, choices=["steps", "inverse", "tapa", "schedule", "moves"],
                    help="with --only-temporal: only these parts (short launch lists for profiling)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.only_temporal:
        import torch
        from paper_2604_14561_b200 import binding
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        pc = {}
        if args.rows is None or "steps" in args.rows:
            pc["temporal_steps"] = temporal_rows(torch, binding, args)
        if not args.no_next_rows:
            pc["next_rows_temporal"] = next_rows(torch, binding, args, *([tuple(args.rows)] if args.rows else []))
        print(json.dumps({"per_config": pc}, ensure_ascii=False))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
