#!/usr/bin/env python
"""Benchmark of the failure-aware MoE routing hot path (dispatch + combine).

A step is one pass of the whole path over one batch of synthetic tokens:
gate -> mask -> top-k -> weights -> replica pick -> count/scan -> permutation
-> scatter (dispatch), then the weighted gather-reduce (combine), on the
DeepSeek-V3-shaped workload (T=8192, H=7168, E=256, k=8, 288 slots on 32
simulated ranks, one rank failed).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.

One GPU: the timed region is K steps replayed from captured CUDA graphs,
repeated until it spans at least 0.3 s; the median repeat is reported.

N > 1 GPUs: one process per GPU over NCCL.  If the process was not started by
torchrun (no WORLD_SIZE in the environment) it starts the N ranks itself.  The
batch is sharded T/N tokens per GPU and the physical slots P/N per GPU, and a
step is the exchange between the GPUs: routing, all-gather of the per-slot
counts, scatter into the owners' receive buffers, combine from them
(`moe_ep_*`).  The total work is fixed, so scaling is strong.  The figure for
N independent replicas (no exchange) is reported beside it as an extra key.

`--impl reference` times the CPU oracle, as it stands, on the host cores.
`--dry-run` walks the multi-rank protocol on CPU (gloo) without touching a GPU.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "dispatch+combine tokens/s at DSv3 shape"
UNIT = "tokens/s"
N_INPUT_SETS = 3      # device copies of the inputs that the timed steps rotate over
E2E_STEPS_IN_FLIGHT = 2          # host-fed steps kept in flight
MIN_TIMED_SECONDS = 0.3          # the timed region is repeated until it spans at least this long

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures of
# the kernels as they stand at the DSv3 shape (summaries under profiles/); None when a kernel
# changed after its last capture.
NCU_TRAFFIC_BYTES = {"k_scatter": 998_396_160, "k_combine": 1_051_368_192}

INT_FIELDS = ("topk_ids", "topk_slot", "slot_counts", "slot_offsets", "rank_counts", "rank_offsets", "dst_row")


def env_rank():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def host_info():
    """Core count and CPU model of the machine the CPU baseline runs on."""
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"host_cores": os.cpu_count(), "cpu_model": model}


def algorithmic_bytes(wl, T):
    """Bytes the method must move per launch, by kernel: routing reads the logits and writes
    four index/weight words per assignment; scatter reads each row once and writes it k times;
    combine reads k rows and writes one (plus the small index traffic of each)."""
    row = 2 * wl.H
    route = T * (4 * wl.E + 16 * wl.k)                 # logits in; ids, weights, slots, ranks out
    scatter = T * ((1 + wl.k) * row + 20 * wl.k)       # x once, k copies out; slot/rank/offset in, rows out
    combine = T * ((wl.k + 1) * row + 16 * wl.k)       # k rows in, y out; row, weight, slot, scale in
    return {"k_route": route, "k_scatter": scatter, "k_combine": combine}


def shard_tokens(T: int, world: int, rank: int):
    """Tokens [lo, hi) of the global batch that `rank` of `world` owns (contiguous, balanced)."""
    per, extra = divmod(T, world)
    lo = rank * per + min(rank, extra)
    return lo, lo + per + (1 if rank < extra else 0)


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None
        self.period = period_s

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_cfg_for(wl):
    import oracle
    return oracle.OracleConfig(num_experts=wl.E, top_k=wl.k, num_ranks=wl.R, slots_per_rank=wl.S,
                               score_func=wl.score_func, n_group=wl.n_group, topk_group=wl.topk_group)


def oracle_step(wl, inp, failed, T):
    """One dispatch + combine of the CPU oracle on the first T tokens."""
    import oracle
    from paper_2602_21140_b200 import workloads as W
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    ref = oracle.dispatch(oracle_cfg_for(wl), inp["slot_to_expert"], failed, bias,
                          inp["logits"][:T], inp["x"][:T])
    oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                   inp["slot_scale"])


def time_oracle(wl, inp, failed, budget_s=12.0, t_probe=256):
    """Oracle throughput on a bounded sample: whole steps of T_sample tokens for about budget_s."""
    n_tok = inp["logits"].shape[0]
    t_probe = min(t_probe, n_tok)
    t0 = time.perf_counter()
    oracle_step(wl, inp, failed, t_probe)
    per_tok = (time.perf_counter() - t0) / t_probe
    T_s = int(max(min(64, n_tok), min(n_tok, budget_s / 3 / per_tok)))
    n, t_start = 0, time.perf_counter()
    while n < 3 or (time.perf_counter() - t_start < budget_s and n < 50):
        oracle_step(wl, inp, failed, T_s)
        n += 1
        if time.perf_counter() - t_start > 3 * budget_s:
            break
    dt = time.perf_counter() - t_start
    return {"value": T_s * n / dt, "unit": UNIT, "cores": 1, "kind": "oracle", **host_info(),
            "sample": f"{n} dispatch+combine steps over the first {T_s} of {n_tok} tokens, {dt:.1f} s, "
                      f"plain C oracle, one thread (not pinned) of {os.cpu_count()} host cores"}


def workload_name(wl, failed):
    return (f"{wl.name}: T={wl.T} H={wl.H} bf16, E={wl.E}, k={wl.k}, "
            f"{'sigmoid+bias' if wl.score_func else 'softmax'}"
            f"{f', {wl.n_group} groups top-{wl.topk_group}' if wl.n_group > 1 else ''}, "
            f"{wl.P} slots on {wl.R} ranks, failed ranks {list(failed)}")


def base_config(wl, failed):
    return {"workload": workload_name(wl, failed), "T": wl.T, "H": wl.H, "E": wl.E, "k": wl.k,
            "slots": wl.P, "ranks": wl.R, "failed_ranks": list(failed)}


def run_reference(args):
    rank, _, world = env_rank()
    if rank != 0:
        return
    from paper_2602_21140_b200 import workloads as W
    wl = W.WORKLOADS[args.workload]
    failed = wl.failure_sets[min(args.failure_set, len(wl.failure_sets) - 1)]
    inp = W.make_inputs(wl)
    # size the per-step sample so that warmup + steps end within about two minutes
    t0 = time.perf_counter()
    oracle_step(wl, inp, failed, min(128, wl.T))
    per_tok = (time.perf_counter() - t0) / min(128, wl.T)
    T_s = int(max(8, min(wl.T, 120.0 / (args.steps + args.warmup) / per_tok)))
    for _ in range(args.warmup):
        oracle_step(wl, inp, failed, T_s)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(wl, inp, failed, T_s)
    dt = time.perf_counter() - t0
    value = T_s * args.steps / dt
    sample = (f"each step = oracle dispatch+combine over the first {T_s} of {wl.T} tokens, plain C oracle, "
              f"one thread (not pinned) of {os.cpu_count()} host cores")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak" if args.gpus == 1 else "strong", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {**base_config(wl, failed), "sample_tokens": T_s},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", **host_info(), "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest `value` over all ranks (identity for a single process)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_seed(base_seed: int, rank: int) -> int:
    """Independent replicas: same workload recipe, different seed per rank."""
    return base_seed + 1000 * rank


def apply_tuning(router, specs):
    from paper_2602_21140_b200 import binding as B
    for spec in specs or []:
        name, value = spec.split("=")
        router.set_tuning(getattr(B, "MOE_TUNE_" + name.strip().upper()), int(value))


def timed_blocks(replay_block, K, stream, sampler=None, min_seconds=MIN_TIMED_SECONDS, max_repeats=400):
    """Time `replay_block()` (which enqueues exactly K steps on `stream`) with CUDA events, again
    and again until the timed blocks span min_seconds; returns the per-block milliseconds."""
    import torch
    times = []
    if sampler is not None:
        sampler.start()
    t_wall = time.perf_counter()
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        replay_block()
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
        if len(times) >= max_repeats or (len(times) >= 3 and time.perf_counter() - t_wall >= min_seconds):
            break
    return times


def oracle_reference_outputs(wl, inp, failed, with_bias):
    """Integer outputs of the oracle for one failure set (routing and permutation)."""
    import oracle
    cfg = oracle_cfg_for(wl)
    ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"] if with_bias else None, inp["logits"])
    ref = oracle.permutation(cfg, slot)
    ref.update(topk_ids=ids, topk_slot=slot)
    return ref


def matches_oracle(out, ref_dev) -> bool:
    import torch
    return all(bool(torch.equal(getattr(out, f).reshape(-1), ref_dev[f])) for f in INT_FIELDS)


def remap_leg(router, graph, out, wl, inp, sets, restore, n_iter=30):
    """Remap -> first step on one captured single-step graph, never recaptured.  Every first step
    after a remap is compared with the oracle (ids, slots, counts, offsets, rows)."""
    import torch
    from paper_2602_21140_b200 import workloads as W
    dev = out.topk_ids.device
    with_bias = wl.score_func == W.SIGMOID
    refs = {}
    for fs in set(sets):
        ref = oracle_reference_outputs(wl, inp, fs, with_bias)
        refs[fs] = {f: torch.from_numpy(np.ascontiguousarray(ref[f]).reshape(-1)).to(dev) for f in INT_FIELDS}
    steady, added, host_us, ok = [], [], [], True
    for i in range(n_iter):
        # a plain replay and a remap + replay back to back, so that slow drift of the step time
        # cancels in their difference
        fs = sets[i % len(sets)]
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        graph.replay()
        torch.cuda.synchronize()
        t_plain = time.perf_counter() - t0
        t0 = time.perf_counter()
        router.set_failed_ranks(fs)
        t1 = time.perf_counter()
        graph.replay()
        torch.cuda.synchronize()
        t_remap = time.perf_counter() - t0
        steady.append(t_plain)
        added.append(t_remap - t_plain)
        host_us.append((t1 - t0) * 1e6)
        ok = ok and matches_oracle(out, refs[fs])     # outside the timed part
    router.set_failed_ranks(restore)
    return {"host_call_us_median": statistics.median(host_us),
            "added_latency_us_median": statistics.median(added) * 1e6,
            "step_us_median": statistics.median(steady) * 1e6,
            "first_step_matches_oracle": bool(ok),
            "checked": "every first step after a remap: " + ", ".join(INT_FIELDS),
            "added_latency": "median over pairs of (remap + replay + sync) - (replay + sync), wall clock",
            "failure_sets_cycled": [list(s) for s in sets], "launches": 3 * 2 * n_iter + n_iter}


def kimi_remap_sweep(dev, steps=20):
    """The Kimi-K2-shaped sweep: failed-rank counts 0..8 applied mid-stream to ONE captured graph."""
    import torch
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import workloads as W
    wl = W.WORKLOADS["kimi"]
    T = wl.T
    inp = W.make_inputs(wl)
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp["slot_to_expert"], inp["bias"],
                         inp["slot_scale"], device=dev)
    logits = torch.from_numpy(inp["logits"]).to(dev)
    x = torch.from_numpy(inp["x"]).view(torch.int16).view(torch.bfloat16).to(dev)
    out = router.alloc_outputs(T)
    y = torch.empty((T, wl.H), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.Stream(device=dev)
    stream.wait_stream(torch.cuda.current_stream())
    rows, launches, captures = [], 0, 0
    with torch.cuda.stream(stream):
        for _ in range(3):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
        captures += 1
        launches += 9
        for n, fs in enumerate(wl.failure_sets):
            ref = oracle_reference_outputs(wl, inp, fs, True)
            ref_dev = {f: torch.from_numpy(np.ascontiguousarray(ref[f]).reshape(-1)).to(dev) for f in INT_FIELDS}
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            router.set_failed_ranks(fs)                   # mid-stream: the same graph is replayed next
            graph.replay()
            torch.cuda.synchronize()
            first = time.perf_counter() - t0
            ok = matches_oracle(out, ref_dev)
            no_failed_rows = bool((out.rank_counts[list(fs)] == 0).all()) if fs else True
            added = []
            for _ in range(9):                           # plain replay, then remap + replay: the difference
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                graph.replay()
                torch.cuda.synchronize()
                t_plain = time.perf_counter() - t0
                t0 = time.perf_counter()
                router.set_failed_ranks(fs)
                graph.replay()
                torch.cuda.synchronize()
                added.append(time.perf_counter() - t0 - t_plain)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            launches += 3 * (19 + steps) + 10
            rows.append({"failed_ranks": n, "first_step_matches_oracle": bool(ok),
                         "failed_ranks_own_no_rows": no_failed_rows,
                         "added_latency_us": statistics.median(added) * 1e6,
                         "first_step_us_wall": first * 1e6,
                         "steady_tokens_per_s": T * steps / (e0.elapsed_time(e1) * 1e-3),
                         "steady_us_per_step": e0.elapsed_time(e1) * 1e3 / steps})
    assert router.device_status() == 0
    router.close()
    return {"workload": workload_name(wl, ()), "tokens": T, "graph_captures": captures,
            "graph_recaptured": captures != 1, "rows": rows,
            "what": "full Kimi-K2 shape; per failed-rank count: remap + first replay of the one captured graph "
                    "checked against the oracle (" + ", ".join(INT_FIELDS) + "), added latency = median over 9 pairs "
                    "of (wall time of remap + replay) - (wall time of the replay before it), steady throughput over "
                    f"{steps} replays (CUDA events)", "launches": launches}


def run_single(args):
    """One GPU: the whole path on one device (simulated EP ranks are regions of the send buffer)."""
    import torch
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl = W.WORKLOADS[args.workload]
    failed = wl.failure_sets[min(args.failure_set, len(wl.failure_sets) - 1)]
    T, K, Wm = (args.tokens or wl.T), args.steps, args.warmup
    inp = W.make_inputs(wl, T=T)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None

    def new_router(inputs=inp):
        r = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inputs["slot_to_expert"],
                        inputs["bias"] if wl.score_func == W.SIGMOID else None, inputs["slot_scale"], device=dev)
        apply_tuning(r, args.tune)
        r.set_failed_ranks(failed)
        return r

    router = new_router()
    lg_h = torch.from_numpy(inp["logits"]).pin_memory()
    x_h = torch.from_numpy(inp["x"]).view(torch.int16).view(torch.bfloat16).pin_memory()
    y_h = torch.empty((T, wl.H), dtype=torch.bfloat16).pin_memory()
    logits, x = lg_h.to(dev), x_h.to(dev)
    # the timed steps rotate over three copies of the inputs, so that no step can find its x rows
    # or logits in L2 from an earlier step (one copy is about as large as the 126 MB L2)
    in_sets = [(logits, x)] + [(logits.clone(), x.clone()) for _ in range(N_INPUT_SETS - 1)]
    out = router.alloc_outputs(T)
    y = torch.empty((T, wl.H), dtype=torch.bfloat16, device=dev)

    stream = torch.cuda.Stream(device=dev)
    stream.wait_stream(torch.cuda.current_stream())
    launches, captures = 2, 0                      # the two state-derivation kernels of init and remap
    if args.quick:
        # profiling aid: a few eager steps and nothing else, so that a profiler capture stays short
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for i in range(Wm + K):
                if i == Wm:
                    e0.record(stream)
                router.dispatch(logits, x, out)
                router.combine(out.send_buf, T, y)
            e1.record(stream)
            torch.cuda.synchronize()
            assert router.device_status() == 0
        print(json.dumps({"quick": True, "workload": workload_name(wl, failed), "tokens": T, "steps": K,
                          "ms_per_step": e0.elapsed_time(e1) / max(K, 1)}))
        router.close()
        return
    with torch.cuda.stream(stream):
        n_warm = max(Wm, 3)
        for _ in range(n_warm):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
        stream.synchronize()
        launches += 3 * n_warm
        assert router.device_status() == 0
        assert int(out.slot_offsets[-1]) == T * wl.k
        graphs = []
        for lg_i, x_i in in_sets:                      # one captured step per input set, same outputs
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                router.dispatch(lg_i, x_i, out)
                router.combine(out.send_buf, T, y)
            graphs.append(g)
            captures += 1
        graph = graphs[0]
        # ... and one graph holding a step on every input set back to back, as the layers of a model
        # sit in one graph: inside it the routing kernel of a step is scheduled while the combine
        # of the step before drains (programmatic dependent launch needs both in the same graph)
        cycle = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cycle, stream=stream):
            for lg_i, x_i in in_sets:
                router.dispatch(lg_i, x_i, out)
                router.combine(out.send_buf, T, y)
        captures += 1
        captures_before_timing = captures
        for i in range(n_warm):
            graphs[i % N_INPUT_SETS].replay()
        cycle.replay()
        stream.synchronize()
        launches += 3 * (n_warm + N_INPUT_SETS)

        # ---- timed region: blocks of K replayed steps, repeated until they span 0.3 s ---------
        def replay_block():
            for _ in range(K // N_INPUT_SETS):
                cycle.replay()                           # N_INPUT_SETS steps each
            for i in range(K % N_INPUT_SETS):
                graphs[i].replay()

        sampler = ClockSampler(0)
        torch.cuda.synchronize()
        block_ms = timed_blocks(replay_block, K, stream, sampler)
        clocks = sampler.stop()
        ms_total = statistics.median(block_ms)
        launches += 3 * K * len(block_ms)
        value = T * K / (ms_total * 1e-3)

        # ---- per-kernel durations: eager launches with events between the kernels
        K2 = 200
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K2)]
        for i in range(K2):
            router.set_timing_event(ev[i][1])
            ev[i][0].record(stream)
            router.dispatch(*in_sets[i % N_INPUT_SETS], out)
            ev[i][2].record(stream)
            router.combine(out.send_buf, T, y)
            ev[i][3].record(stream)
        router.set_timing_event(None)
        torch.cuda.synchronize()
        launches += 3 * K2
        dur_ms = {"k_route": statistics.mean(e[0].elapsed_time(e[1]) for e in ev),
                  "k_scatter": statistics.mean(e[1].elapsed_time(e[2]) for e in ev),
                  "k_combine": statistics.mean(e[2].elapsed_time(e[3]) for e in ev)}

        # ---- end to end through the C ABI with host buffers ----------------
        # Every step uploads its logits and x from pinned host memory and downloads its y.  A few
        # steps are kept in flight (one context, stream, staging and output set each), so
        # that one step's upload overlaps the other's download; the one-at-a-time figure is
        # reported beside it.
        K3 = min(K, 20)
        lg_d, x_d = torch.empty_like(logits), torch.empty_like(x)
        for _ in range(2):
            router.step_host(lg_h, x_h, out, lg_d, x_d, y, y_h)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(K3):
            router.step_host(lg_h, x_h, out, lg_d, x_d, y, y_h)     # returns after the D2H copy
        e2e_serial_s = time.perf_counter() - t0
        launches += 3 * (K3 + 2)

        lanes = [dict(r=router, st=stream, out=out, lg_d=lg_d, x_d=x_d, y=y, y_h=y_h)]
        for _ in range(E2E_STEPS_IN_FLIGHT - 1):
            r_extra = new_router()
            launches += 2
            lanes.append(dict(r=r_extra, st=torch.cuda.Stream(device=dev), out=r_extra.alloc_outputs(T),
                              lg_d=torch.empty_like(logits), x_d=torch.empty_like(x), y=torch.empty_like(y),
                              y_h=torch.empty((T, wl.H), dtype=torch.bfloat16).pin_memory()))

        def host_step(i):
            ln = lanes[i % E2E_STEPS_IN_FLIGHT]
            ln["st"].synchronize()                       # the lane's previous step has delivered its y
            with torch.cuda.stream(ln["st"]):
                ln["r"].step_host_async(lg_h, x_h, ln["out"], ln["lg_d"], ln["x_d"], ln["y"], ln["y_h"])

        for i in range(2 * E2E_STEPS_IN_FLIGHT):
            host_step(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(K3):
            host_step(i)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        launches += 3 * (K3 + 2 * E2E_STEPS_IN_FLIGHT)
        for ln in lanes[1:]:
            assert ln["r"].device_status() == 0
            assert torch.equal(lanes[0]["y_h"], ln["y_h"])            # every lane computed the same batch
            ln["r"].close()
        e2e = {"value": T * K3 / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": T * wl.E * 4 + T * wl.H * 2, "d2h_bytes_per_step": T * wl.H * 2,
               "steps": K3, "ms_per_step": 1e3 * e2e_s / K3, "steps_in_flight": E2E_STEPS_IN_FLIGHT,
               "one_step_at_a_time": {"value": T * K3 / e2e_serial_s,
                                      "ms_per_step": 1e3 * e2e_serial_s / K3}}
        del lanes

        # ---- two independent batches in flight (microbatching): context B on a second stream,
        # so that batch B's routing overlaps batch A's memory-bound kernels.  Reported beside the
        # single-stream number, never instead of it.
        overlap = None
        if not args.no_overlap:
            inp_b = W.make_inputs(wl, T=T, seed=shard_seed(wl.seed, 1))
            router_b = new_router(inp_b)
            launches += 2
            lg_b = torch.from_numpy(inp_b["logits"]).to(dev)
            x_b = torch.from_numpy(inp_b["x"]).view(torch.int16).view(torch.bfloat16).to(dev)
            out_b, y_b = router_b.alloc_outputs(T), torch.empty_like(y)
            side = torch.cuda.Stream(device=dev)
            for _ in range(3):
                router_b.dispatch(lg_b, x_b, out_b)
                router_b.combine(out_b.send_buf, T, y_b)
            stream.synchronize()
            pair = torch.cuda.CUDAGraph()
            with torch.cuda.graph(pair, stream=stream):
                side.wait_stream(stream)
                router.dispatch(logits, x, out)
                router.combine(out.send_buf, T, y)
                with torch.cuda.stream(side):
                    router_b.dispatch(lg_b, x_b, out_b)
                    router_b.combine(out_b.send_buf, T, y_b)
                stream.wait_stream(side)
            for _ in range(3):
                pair.replay()
            torch.cuda.synchronize()
            n_pairs = max(1, min(K, 400) // 2)
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record(stream)
            for _ in range(n_pairs):
                pair.replay()
            p1.record(stream)
            torch.cuda.synchronize()
            launches += 6 * (n_pairs + 6)
            ms_pair = p0.elapsed_time(p1) / n_pairs
            overlap = {"value": 2 * T / (ms_pair * 1e-3), "unit": UNIT, "ms_per_step": ms_pair / 2,
                       "what": "two batches in flight on two streams (two contexts), one graph per pair"}
            assert router_b.device_status() == 0
            router_b.close()
            del lg_b, x_b, out_b, y_b

        # ---- the multi-GPU exchange path, emulated on this one device: 4 virtual GPUs, each with a
        # quarter of the batch, store their rows straight into each other's receive buffers
        # (moe_ep_*); "peer" memory is local HBM here, so this times the kernels, not NVLink.
        ep_leg = None
        if not args.no_overlap and wl.R % 4 == 0 and T % 4 == 0:
            Gv, Tq = 4, T // 4
            cfg_q = B.config_for_workload(wl, max_tokens=Tq)
            vr = [B.MoeRouter(cfg_q, inp["slot_to_expert"], bias, inp["slot_scale"], device=dev) for _ in range(Gv)]
            recv = [torch.empty((T * wl.k // 2, wl.H), dtype=torch.bfloat16, device=dev) for _ in range(Gv)]
            counts_all = torch.zeros((Gv, wl.P), dtype=torch.int32, device=dev)
            offs = [torch.zeros(wl.P // Gv + 1, dtype=torch.int32, device=dev) for _ in range(Gv)]
            outs_q, ys_q = [], []
            for g, r in enumerate(vr):
                apply_tuning(r, args.tune)
                r.set_failed_ranks(failed)
                r.ep_attach(Gv, g, [b.data_ptr() for b in recv], recv[0].shape[0])
                o = r.alloc_outputs(Tq)
                o.slot_counts = counts_all[g]          # the all-gather of the counts is a no-op on one device
                o.send_buf = o.send_buf[:1]
                outs_q.append(o)
                ys_q.append(torch.empty((Tq, wl.H), dtype=torch.bfloat16, device=dev))
            launches += 2 * Gv

            vstreams = [torch.cuda.Stream(device=dev) for _ in range(Gv)]

            def on_every_virtual_gpu(fn):
                # each virtual GPU works on its own stream, as separate devices would; all of them
                # are joined before the next phase (the ordering a collective provides between GPUs)
                for g, r in enumerate(vr):
                    vstreams[g].wait_stream(stream)
                    with torch.cuda.stream(vstreams[g]):
                        fn(g, r)
                for g in range(Gv):
                    stream.wait_stream(vstreams[g])

            def ep_step():
                on_every_virtual_gpu(lambda g, r: r.ep_route(logits[g * Tq:(g + 1) * Tq], outs_q[g]))
                on_every_virtual_gpu(lambda g, r: r.ep_scatter(x[g * Tq:(g + 1) * Tq], counts_all, offs[g]))
                on_every_virtual_gpu(lambda g, r: r.ep_combine(Tq, ys_q[g]))

            for _ in range(3):
                ep_step()
            stream.synchronize()
            assert all(r.device_status() == 0 for r in vr)
            ep_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(ep_graph, stream=stream):
                ep_step()
            for _ in range(3):
                ep_graph.replay()
            n_ep = max(1, min(K, 200))
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record(stream)
            for _ in range(n_ep):
                ep_graph.replay()
            q1.record(stream)
            torch.cuda.synchronize()
            launches += 4 * Gv * (n_ep + 6)
            ms_ep = q0.elapsed_time(q1) / n_ep
            same = all(torch.equal(ys_q[g], y[g * Tq:(g + 1) * Tq]) for g in range(Gv)) if wl.n_redundant == 0 else None
            ep_leg = {"value": T / (ms_ep * 1e-3), "unit": UNIT, "ms_per_step": ms_ep, "virtual_gpus": Gv,
                      "tokens_per_virtual_gpu": Tq, "y_equals_single_gpu_step": same,
                      "what": "4 virtual GPUs on one device, one stream each, joined between the phases: "
                              "route, count table, scatter into the owners' receive buffers, combine from "
                              "them; 16 kernels per step in one graph"}
            for r in vr:
                r.close()
            del recv, outs_q, ys_q

        # ---- remap -> first step: same graph, no recapture ------------------
        sets = [fs for fs in wl.failure_sets] or [()]
        remap = remap_leg(router, graph, out, wl, inp, sets, failed)
        launches += remap.pop("launches")
        remap["graph_captures_during_remaps"] = captures - captures_before_timing
        remap["graph_recaptured"] = captures != captures_before_timing
        assert router.device_status() == 0

    # ---- roofline of the dominant kernel -----------------------------------
    peak, peak_kind = measured_peaks()
    alg = algorithmic_bytes(wl, T)
    dom = max(("k_scatter", "k_combine"), key=lambda n: dur_ms[n])
    achieved = alg[dom] / (dur_ms[dom] * 1e-3) / 1e9
    step_gbs = sum(alg.values()) * K / (ms_total * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": NCU_TRAFFIC_BYTES[dom] if (wl.name == "dsv3" and T == wl.T) else None,
                "algorithmic_bytes": alg[dom], "kernel_ms": dur_ms[dom],
                "per_kernel_source": "a separate eager leg with CUDA events between the launches; the kernels "
                                     "overlap less there than in the graph replays of the timed region, so the "
                                     "three durations add up to more than ms_per_step",
                "per_kernel": {n: {"ms": dur_ms[n], "algorithmic_bytes": alg[n],
                                   "GB/s": alg[n] / (dur_ms[n] * 1e-3) / 1e9,
                                   "frac": alg[n] / (dur_ms[n] * 1e-3) / 1e9 / peak} for n in dur_ms},
                "step": {"algorithmic_bytes": sum(alg.values()), "GB/s": step_gbs, "frac": step_gbs / peak,
                         "frac_of_8TBs_nominal": step_gbs / 8000.0}}

    cpu_baseline = time_oracle(wl, inp, failed)
    router.close()
    del out, y, in_sets, logits, x
    torch.cuda.empty_cache()

    kimi = None
    if wl.name == "dsv3" and T == wl.T and not args.no_kimi_sweep:
        kimi = kimi_remap_sweep(dev)
        launches += kimi.pop("launches")

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "ms_per_step_min": min(block_ms) / K, "ms_per_step_max": max(block_ms) / K,
        "timed_repeats": len(block_ms), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {**base_config(wl, failed), "T_per_gpu": T,
                   "parallelism": "one GPU; the EP ranks are regions of its send buffer",
                   "l2": f"inputs rotate over {N_INPUT_SETS} device copies ({N_INPUT_SETS} x "
                         f"{(T * wl.E * 4 + T * wl.H * 2) / 1e6:.0f} MB) and a step moves "
                         f"{sum(algorithmic_bytes(wl, T).values()) / 1e9:.2f} GB, both beyond the 126 MB L2; no flush",
                   "timed": f"blocks of {K} steps replayed from CUDA graphs ({N_INPUT_SETS} consecutive steps per graph), "
                            f"CUDA events per block, repeated until the blocks span {MIN_TIMED_SECONDS} s; the median block is reported"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
        "cpu_baseline": cpu_baseline, "remap": remap, "kimi_remap_sweep": kimi, "two_batches_in_flight": overlap,
        "expert_parallel_emulated": ep_leg}))


def run_group(args):
    """N > 1 GPUs: one rank per GPU; a step is the exchange between the GPUs (moe_ep_*)."""
    import torch
    import torch.distributed as dist
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import ep
    from paper_2602_21140_b200 import workloads as W

    rank, local_rank, world = env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world == 1:                                      # --exchange on one GPU: a group of one
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if "MASTER_PORT" not in os.environ:
            with socket.socket() as s:
                s.bind(("127.0.0.1", 0))
                os.environ["MASTER_PORT"] = str(s.getsockname()[1])
        dist.init_process_group("nccl", device_id=dev, rank=0, world_size=1)
    else:
        dist.init_process_group("nccl", device_id=dev)

    wl = W.WORKLOADS[args.workload]
    failed = wl.failure_sets[min(args.failure_set, len(wl.failure_sets) - 1)]
    T, K, Wm = (args.tokens or wl.T), args.steps, args.warmup
    if wl.R % world != 0:
        raise SystemExit(f"{wl.R} simulated ranks do not split over {world} GPUs")
    lo, hi = shard_tokens(T, world, rank)
    Tl = hi - lo
    inp = W.make_inputs(wl, T=T)                        # the same global batch on every rank; each keeps its shard
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    cfg = B.config_for_workload(wl, max_tokens=max(Tl, 1))
    recv_rows = T * wl.k                                # always suffices: every row of the step could land here
    # The exchange needs symmetric memory between the GPUs of the group.  Where that cannot be set
    # up, every rank learns of it here (one all-reduce) and the run reports the independent
    # replicas alone instead of failing half-way through a collective.
    exch_error, group = None, None
    try:
        group = ep.DistributedEp(cfg, inp["slot_to_expert"], bias, inp["slot_scale"], recv_rows, dev)
    except Exception as exc:                            # noqa: BLE001 - reported in the JSON line
        exch_error = f"{type(exc).__name__}: {exc}"[:300]
    if max_over_ranks(1.0 if exch_error else 0.0, world, dev) > 0:
        if group is not None:
            group.close()
        group = None
        exch_error = exch_error or "another rank could not set up the exchange"
    launches = 0
    if group is not None:
        apply_tuning(group.router, args.tune)
        group.router.set_failed_ranks(failed)

        lg_h = torch.from_numpy(inp["logits"][lo:hi]).pin_memory()
        x_h = torch.from_numpy(inp["x"][lo:hi]).view(torch.int16).view(torch.bfloat16).pin_memory()
        y_h = torch.empty((Tl, wl.H), dtype=torch.bfloat16).pin_memory()
        logits, x = lg_h.to(dev), x_h.to(dev)
        out = group.router.alloc_outputs(Tl)
        out.send_buf = out.send_buf[:1]                    # no send buffer in this mode
        y = torch.empty((Tl, wl.H), dtype=torch.bfloat16, device=dev)

        def step():
            group.dispatch(logits, x, out)
            group.combine(Tl, y)

        launches = 2
        for _ in range(max(Wm, 3)):
            step()
        torch.cuda.synchronize()
        launches += 4 * max(Wm, 3)
        assert group.router.device_status() == 0
        # a captured step (NCCL calls included) removes the host from the loop; plain launches otherwise
        replay, timed_how = step, "eager launches"
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step()
            g.replay()
            torch.cuda.synchronize()
            replay, timed_how = g.replay, "CUDA-graph replays of one step"
        except Exception:
            torch.cuda.synchronize()
        def timed_block():
            dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(K):
                replay()
            e1.record()
            torch.cuda.synchronize()
            return max_over_ranks(e0.elapsed_time(e1), world, dev)     # the same figure on every rank

        sampler = ClockSampler(local_rank)
        sampler.start()
        block_ms = [timed_block()]
        # every rank derives the same number of repeats from the same (max over ranks) first block
        repeats = max(3, min(100, int(np.ceil(MIN_TIMED_SECONDS * 1e3 / block_ms[0]))))
        while len(block_ms) < repeats:
            block_ms.append(timed_block())
        clocks = sampler.stop()
        dist.barrier()
        ms_total = statistics.median(block_ms)
        launches += 4 * K * len(block_ms)
        value = T * K / (ms_total * 1e-3)

        # end to end: every step uploads this rank's shard from pinned host memory and downloads its y
        K3 = min(K, 20)
        lg_d, x_d = torch.empty_like(logits), torch.empty_like(x)

        def host_step():
            lg_d.copy_(lg_h, non_blocking=True)
            x_d.copy_(x_h, non_blocking=True)
            group.dispatch(lg_d, x_d, out)
            group.combine(Tl, y)
            y_h.copy_(y, non_blocking=True)
            torch.cuda.synchronize()

        for _ in range(2):
            host_step()
        dist.barrier()
        t0 = time.perf_counter()
        for _ in range(K3):
            host_step()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world, dev)
        launches += 4 * (K3 + 2)
        e2e = {"value": T * K3 / e2e_s, "unit": UNIT, "h2d_bytes_per_step": T * wl.E * 4 + T * wl.H * 2,
               "d2h_bytes_per_step": T * wl.H * 2, "steps": K3, "ms_per_step": 1e3 * e2e_s / K3,
               "what": "bytes are whole-job totals over all ranks; each rank moves its T/N shard"}
        assert group.router.device_status() == 0
        group.close()

    # extra: N independent replicas, every rank a whole batch of its own and no exchange (weak scaling)
    inp_r = W.make_inputs(wl, T=T, seed=shard_seed(wl.seed, rank))
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp_r["slot_to_expert"],
                         inp_r["bias"] if wl.score_func == W.SIGMOID else None, inp_r["slot_scale"], device=dev)
    apply_tuning(router, args.tune)
    router.set_failed_ranks(failed)
    lg_r = torch.from_numpy(inp_r["logits"]).to(dev)
    x_r = torch.from_numpy(inp_r["x"]).view(torch.int16).view(torch.bfloat16).to(dev)
    out_r = router.alloc_outputs(T)
    y_r = torch.empty((T, wl.H), dtype=torch.bfloat16, device=dev)
    for _ in range(3):
        router.dispatch(lg_r, x_r, out_r)
        router.combine(out_r.send_buf, T, y_r)
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        router.dispatch(lg_r, x_r, out_r)
        router.combine(out_r.send_buf, T, y_r)
    gr.replay()
    dist.barrier()
    torch.cuda.synchronize()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for _ in range(K):
        gr.replay()
    r1.record()
    torch.cuda.synchronize()
    ms_rep = max_over_ranks(r0.elapsed_time(r1), world, dev)
    launches += 3 * (K + 5) + 2
    replicas = {"value": world * T * K / (ms_rep * 1e-3), "unit": UNIT, "ms_per_step": ms_rep / K, "scaling": "weak",
                "what": f"{world} independent replicas, one whole batch of {T} tokens per GPU, no exchange"}
    assert router.device_status() == 0
    router.close()

    if rank == 0 and group is None:
        # no exchange on this machine: the replicas are all there is to report
        print(json.dumps({
            "metric": METRIC, "value": replicas["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": replicas["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {**base_config(wl, failed), "T_per_gpu": T,
                       "parallelism": f"{world} independent replicas, no data-path collective",
                       "timed": "CUDA-graph replays of one step, CUDA events, max over ranks"},
            "exchange_unavailable": exch_error, "clocks": None, "e2e": None, "gpu_launches": launches,
            "roofline": None, "cpu_baseline": None, "independent_replicas": replicas}))
    elif rank == 0:
        alg = algorithmic_bytes(wl, T)
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_total / K, "ms_per_step_min": min(block_ms) / K, "ms_per_step_max": max(block_ms) / K,
            "timed_repeats": len(block_ms), "higher_is_better": True, "scaling": "strong" if world > 1 else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {**base_config(wl, failed), "T_per_gpu": Tl, "slots_per_gpu": wl.P // world,
                       "parallelism": f"ep{world}: tokens sharded T/{world} per GPU, slots P/{world} per GPU; per step "
                                      "route, all-gather of per-slot counts (NCCL), scatter into the owners' receive "
                                      "buffers over peer memory, combine from them; two one-word all-reduces order the GPUs",
                       "l2": f"a step moves {sum(alg.values()) / 1e9:.2f} GB over all GPUs; inputs are not rotated",
                       "timed": f"blocks of {K} steps, {timed_how}, CUDA events around each block, max over ranks per "
                                f"block, blocks repeated until they span {MIN_TIMED_SECONDS} s, the median block is reported"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "step", "achieved": sum(alg.values()) * K / (ms_total * 1e-3) / 1e9,
                         "peak": measured_peaks()[0] * world, "unit": "GB/s",
                         "frac": sum(alg.values()) * K / (ms_total * 1e-3) / 1e9 / (measured_peaks()[0] * world),
                         "peak_source": f"of {measured_peaks()[1]} (per-GPU copy bandwidth x {world})", "traffic": None},
            "cpu_baseline": None, "independent_replicas": replicas}))
    dist.destroy_process_group()


def run_dry(args):
    """The multi-rank protocol on CPU (gloo), without a GPU: sharding, the exchange of the per-slot
    counts, the layout arithmetic of the library (host entry point) and the one JSON line."""
    import torch
    import torch.distributed as dist
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import ep
    from paper_2602_21140_b200 import workloads as W

    rank, _, world = env_rank()
    if world > 1:
        dist.init_process_group("gloo")
    wl = W.WORKLOADS[args.workload]
    failed = wl.failure_sets[min(args.failure_set, len(wl.failure_sets) - 1)]
    T = args.tokens or wl.T
    lo, hi = shard_tokens(T, world, rank)
    # stand-in for the routing result of this rank's shard: a seeded slot for every assignment
    # that avoids the failed ranks (drawing inputs only; no arithmetic of the method)
    rng = np.random.Generator(np.random.Philox(key=[wl.seed, 99 + rank]))
    live = np.array([p for p in range(wl.P) if p // wl.S not in failed], dtype=np.int64)
    slots = live[rng.integers(0, live.size, size=(hi - lo) * wl.k)]
    counts = torch.from_numpy(np.bincount(slots, minlength=wl.P).astype(np.int32))
    counts_all = ep.gather_counts(counts) if world > 1 else counts[None]
    st, src_base, recv_off = B.moe_ep_plan_host(counts_all.numpy(), rank)
    assert st == B.MOE_OK
    rows_here = int(recv_off[-1])
    total = torch.tensor([rows_here], dtype=torch.int64)
    if world > 1:
        dist.all_reduce(total)
    assert int(total) == T * wl.k, (int(total), T * wl.k)          # every row has exactly one owner
    ms = max_over_ranks(1.0 + rank, world)                          # the max-over-ranks plumbing
    if rank == 0:
        print(json.dumps({
            "dry_run": True, "metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": None, "higher_is_better": True,
            "scaling": "strong" if world > 1 else "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {**base_config(wl, failed), "T_per_gpu": hi - lo, "slots_per_gpu": wl.P // world,
                       "parallelism": f"ep{world}" if world > 1 else "one GPU"},
            "rows_received_rank0": rows_here, "rows_total": int(total), "max_over_ranks_check": ms}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def spawn_ranks(args) -> int:
    """Start N ranks of this script with torchrun's launcher (one per GPU) and pass their output through."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_expert_failure_sweep(args):
    """Sec. 4.2's lost-expert sweep as a throughput experiment: for the two selection policies
    ("every nth", "most activated") and r in 1/64 .. 1/2, fail the experts, replay the captured
    step and report tokens/s and the load imbalance over the physical slots that still receive
    tokens (largest slot count / mean slot count).  One JSON line, separate from the default run."""
    import torch
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import workloads as W

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = W.WORKLOADS[args.workload]
    T, K = (args.tokens or wl.T), min(args.steps, 200)
    inp = W.make_inputs(wl, T=T)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp["slot_to_expert"], bias,
                         inp["slot_scale"], device=dev)
    logits = torch.from_numpy(inp["logits"]).to(dev)
    x = torch.from_numpy(inp["x"]).view(torch.int16).view(torch.bfloat16).to(dev)
    out = router.alloc_outputs(T)
    y = torch.empty((T, wl.H), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.Stream(device=dev)
    rows = []
    with torch.cuda.stream(stream):
        for _ in range(3):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)

        def measure(label, r, mask):
            try:
                router.set_failed_experts(mask)
            except B.MoeError as e:
                rows.append({"policy": label, "r": r, "rejected": str(e)})
                return
            for _ in range(3):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(K):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            counts = out.slot_counts.cpu().numpy().astype(np.int64)
            used = counts[counts > 0]
            rows.append({"policy": label, "r": r, "experts_lost": int(np.asarray(mask).sum()) if mask is not None else 0,
                         "tokens_per_s": T * K / (e0.elapsed_time(e1) * 1e-3),
                         "us_per_step": e0.elapsed_time(e1) * 1e3 / K,
                         "slots_used": int(used.size), "imbalance_max_over_mean": float(used.max() / used.mean())})

        measure("none", 0.0, None)
        # activation counts per logical expert with nothing failed, for the worst-case policy
        activations = np.bincount(out.topk_ids.cpu().numpy().reshape(-1), minlength=wl.E)
        for r in (1 / 64, 1 / 32, 1 / 16, 1 / 8, 1 / 4, 1 / 2):
            measure("every_nth", r, W.every_nth_mask(wl.E, r))
            measure("most_activated", r, W.most_activated_mask(activations, r))
        router.set_failed_experts(None)
    assert router.device_status() == 0
    router.close()
    print(json.dumps({"experiment": "lost experts: throughput and load imbalance against the lost fraction r",
                      "workload": workload_name(wl, ()), "tokens": T, "steps_per_point": K, "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="dsv3")
    ap.add_argument("--failure-set", type=int, default=1, help="index into the workload's failure sets")
    ap.add_argument("--tokens", type=int, default=0, help="override T (profiling captures on a smaller case)")
    ap.add_argument("--quick", action="store_true", help="a few eager steps only (for profiler captures)")
    ap.add_argument("--no-overlap", action="store_true", help="skip the two extra legs (two batches in flight, emulated multi-GPU exchange)")
    ap.add_argument("--no-kimi-sweep", action="store_true", help="skip the Kimi-K2-shaped remap sweep of the default run")
    ap.add_argument("--tune", action="append", metavar="OPTION=VALUE",
                    help="override a launch choice through moe_set_tuning, e.g. combine_stages=4 (repeatable)")
    ap.add_argument("--exchange", action="store_true",
                    help="time the multi-GPU exchange path (moe_ep_*, NCCL) even with one GPU: a group of one")
    ap.add_argument("--dry-run", action="store_true", help="walk the multi-rank protocol on CPU (gloo); no GPU is touched")
    ap.add_argument("--expert-failure-sweep", action="store_true",
                    help="run the lost-expert sweep (throughput and load imbalance against r) instead of the benchmark")
    args = ap.parse_args()
    _, _, world = env_rank()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        if args.impl == "reference":
            return run_reference(args)                   # one process: rank 0 alone runs the oracle arm
        raise SystemExit(spawn_ranks(args))
    if args.dry_run:
        return run_dry(args)
    if args.expert_failure_sweep:
        return run_expert_failure_sweep(args)
    if args.impl == "reference":
        return run_reference(args)
    if world > 1 or args.exchange:
        return run_group(args)
    return run_single(args)


if __name__ == "__main__":
    main()
