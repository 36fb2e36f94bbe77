#!/usr/bin/env python
"""Benchmark of the failure-aware MoE routing hot path (dispatch + combine).

A step is one pass of the whole path over one batch of synthetic tokens:
gate -> mask -> top-k -> weights -> replica pick -> count/scan -> permutation
-> scatter (dispatch), then the weighted gather-reduce (combine), on the
DeepSeek-V3-shaped workload (T=8192, H=7168, E=256, k=8, 288 slots on 32
simulated ranks, one rank failed).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  N > 1 is launched with torchrun, one rank per GPU; the
path shards by tokens (every rank routes its own batch, no collective on the
data path), so scaling is weak.  `--impl reference` times the CPU oracle, as it
stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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
E2E_STEPS_IN_FLIGHT = int(os.environ.get("MOE_BENCH_E2E_IN_FLIGHT", "2"))   # host-fed steps kept in flight

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures of
# the kernels as they stand at the DSv3 shape (summaries under profiles/); None when a kernel
# changed after its last capture.
NCU_TRAFFIC_BYTES = {"k_scatter": 998_612_992, "k_combine": 1_051_182_336}


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


def algorithmic_bytes(wl, T):
    """Bytes the method must move per launch, by kernel: routing reads the logits and writes
    four index/weight words per assignment; scatter reads each row once and writes it k times;
    combine reads k rows and writes one (plus the small index traffic of each)."""
    row = 2 * wl.H
    route = T * (4 * wl.E + 16 * wl.k)                 # logits in; ids, weights, slots, ranks out
    scatter = T * ((1 + wl.k) * row + 20 * wl.k)       # x once, k copies out; slot/rank/offset in, rows out
    combine = T * ((wl.k + 1) * row + 16 * wl.k)       # k rows in, y out; row, weight, slot, scale in
    return {"k_route": route, "k_scatter": scatter, "k_combine": combine}


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
    t0 = time.perf_counter()
    oracle_step(wl, inp, failed, t_probe)
    per_tok = (time.perf_counter() - t0) / t_probe
    n_tok = inp["logits"].shape[0]
    t_probe = min(t_probe, n_tok)
    T_s = int(max(min(64, n_tok), min(n_tok, budget_s / 3 / per_tok)))
    n, t_start = 0, time.perf_counter()
    while n < 3 or (time.perf_counter() - t_start < budget_s and n < 50):
        oracle_step(wl, inp, failed, T_s)
        n += 1
        if time.perf_counter() - t_start > 3 * budget_s:
            break
    dt = time.perf_counter() - t_start
    return {"value": T_s * n / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n} dispatch+combine steps over the first {T_s} of {n_tok} tokens, {dt:.1f} s, single thread"}


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
    oracle_step(wl, inp, failed, 128)
    per_tok = (time.perf_counter() - t0) / 128
    T_s = int(max(8, min(wl.T, 120.0 / (args.steps + args.warmup) / per_tok)))
    for _ in range(args.warmup):
        oracle_step(wl, inp, failed, T_s)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(wl, inp, failed, T_s)
    dt = time.perf_counter() - t0
    value = T_s * args.steps / dt
    sample = f"each step = oracle dispatch+combine over the first {T_s} of {wl.T} tokens, single thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": workload_name(wl, failed), "T": wl.T, "H": wl.H, "E": wl.E, "k": wl.k,
                   "slots": wl.P, "ranks": wl.R, "failed_ranks": list(failed), "sample_tokens": T_s},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def workload_name(wl, failed):
    return (f"{wl.name}: T={wl.T} H={wl.H} bf16, E={wl.E}, k={wl.k}, "
            f"{'sigmoid+bias' if wl.score_func else 'softmax'}"
            f"{f', {wl.n_group} groups top-{wl.topk_group}' if wl.n_group > 1 else ''}, "
            f"{wl.P} slots on {wl.R} ranks, failed ranks {list(failed)}")


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
    """Every rank routes its own batch: same workload recipe, different seed."""
    return base_seed + 1000 * rank


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2602_21140_b200 import binding as B
    from paper_2602_21140_b200 import workloads as W

    rank, local_rank, world = env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = W.WORKLOADS[args.workload]
    failed = wl.failure_sets[min(args.failure_set, len(wl.failure_sets) - 1)]
    T, K, Wm = (args.tokens or wl.T), args.steps, args.warmup
    inp = W.make_inputs(wl, T=T, seed=shard_seed(wl.seed, rank))
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp["slot_to_expert"], bias,
                         inp["slot_scale"], device=dev)
    router.set_failed_ranks(failed)

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
    launches = 0
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
        for _ in range(max(Wm, 3)):
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
        stream.synchronize()
        assert router.device_status() == 0
        assert int(out.slot_offsets[-1]) == T * wl.k
        graphs = []
        for lg_i, x_i in in_sets:                      # one captured step per input set, same outputs
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                router.dispatch(lg_i, x_i, out)
                router.combine(out.send_buf, T, y)
            graphs.append(g)
        graph = graphs[0]
        # ... and one graph holding a step on every input set back to back, as the layers of a model
        # sit in one graph: inside it the routing kernel of a step is scheduled while the combine
        # of the step before drains (programmatic dependent launch needs both in the same graph)
        cycle = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cycle, stream=stream):
            for lg_i, x_i in in_sets:
                router.dispatch(lg_i, x_i, out)
                router.combine(out.send_buf, T, y)
        for i in range(max(Wm, 3)):
            graphs[i % N_INPUT_SETS].replay()
        cycle.replay()
        stream.synchronize()

        # ---- timed region: K replays of the captured step -----------------
        sampler = ClockSampler(local_rank)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.start()
        e0.record(stream)
        for _ in range(K // N_INPUT_SETS):
            cycle.replay()                               # N_INPUT_SETS steps each
        for i in range(K % N_INPUT_SETS):
            graphs[i].replay()
        e1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        if world > 1:
            dist.barrier()
        ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
        launches += 3 * K
        value = world * T * K / (ms_total * 1e-3)

        # ---- per-kernel durations: eager launches with events between the kernels
        K2 = min(K, 200)
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
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(K3):
            router.step_host(lg_h, x_h, out, lg_d, x_d, y, y_h)     # returns after the D2H copy
        e2e_serial_s = max_over_ranks(time.perf_counter() - t0, world, dev)
        launches += 3 * (K3 + 2)

        lanes = [dict(r=router, st=stream, out=out, lg_d=lg_d, x_d=x_d, y=y, y_h=y_h)]
        for _ in range(E2E_STEPS_IN_FLIGHT - 1):
            r_extra = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp["slot_to_expert"], bias,
                                  inp["slot_scale"], device=dev)
            r_extra.set_failed_ranks(failed)
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
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(K3):
            host_step(i)
        torch.cuda.synchronize()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world, dev)
        launches += 3 * (K3 + 2 * E2E_STEPS_IN_FLIGHT)
        for ln in lanes[1:]:
            assert ln["r"].device_status() == 0
            assert torch.equal(lanes[0]["y_h"], ln["y_h"])            # every lane computed the same batch
            ln["r"].close()
        e2e = {"value": world * T * K3 / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": T * wl.E * 4 + T * wl.H * 2, "d2h_bytes_per_step": T * wl.H * 2,
               "steps": K3, "ms_per_step": 1e3 * e2e_s / K3, "steps_in_flight": E2E_STEPS_IN_FLIGHT,
               "one_step_at_a_time": {"value": world * T * K3 / e2e_serial_s,
                                      "ms_per_step": 1e3 * e2e_serial_s / K3}}
        del lanes

        # ---- two independent batches in flight (microbatching): context B on a second stream,
        # so that batch B's routing overlaps batch A's memory-bound kernels.  Reported beside the
        # single-stream number, never instead of it.
        overlap = None
        if rank == 0 and world == 1 and not args.no_overlap:
            inp_b = W.make_inputs(wl, T=T, seed=shard_seed(wl.seed, 1))
            router_b = B.MoeRouter(B.config_for_workload(wl, max_tokens=T), inp_b["slot_to_expert"],
                                   inp_b["bias"] if wl.score_func == W.SIGMOID else None,
                                   inp_b["slot_scale"], device=dev)
            router_b.set_failed_ranks(failed)
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
        if rank == 0 and world == 1 and not args.no_overlap and wl.R % 4 == 0 and T % 4 == 0:
            Gv, Tq = 4, T // 4
            cfg_q = B.config_for_workload(wl, max_tokens=Tq)
            vr = [B.MoeRouter(cfg_q, inp["slot_to_expert"], bias, inp["slot_scale"], device=dev) for _ in range(Gv)]
            recv = [torch.empty((T * wl.k // 2, wl.H), dtype=torch.bfloat16, device=dev) for _ in range(Gv)]
            counts_all = torch.zeros((Gv, wl.P), dtype=torch.int32, device=dev)
            offs = [torch.zeros(wl.P // Gv + 1, dtype=torch.int32, device=dev) for _ in range(Gv)]
            outs_q, ys_q = [], []
            for g, r in enumerate(vr):
                r.set_failed_ranks(failed)
                r.ep_attach(Gv, g, [b.data_ptr() for b in recv], recv[0].shape[0])
                o = r.alloc_outputs(Tq)
                o.slot_counts = counts_all[g]          # the all-gather of the counts is a no-op on one device
                o.send_buf = o.send_buf[:1]
                outs_q.append(o)
                ys_q.append(torch.empty((Tq, wl.H), dtype=torch.bfloat16, device=dev))

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
        remap = None
        if rank == 0:
            import oracle
            sets = [fs for fs in wl.failure_sets] or [()]
            steady, with_remap, host_us = [], [], []
            for i in range(30):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                graph.replay()
                torch.cuda.synchronize()
                steady.append(time.perf_counter() - t0)
            for i in range(30):
                fs = sets[i % len(sets)]
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                router.set_failed_ranks(fs)
                t1 = time.perf_counter()
                graph.replay()
                torch.cuda.synchronize()
                with_remap.append(time.perf_counter() - t0)
                host_us.append((t1 - t0) * 1e6)
            launches += 60 * 3
            # the step after the last remap is correct for the new failure set
            ids, w, slot = oracle.route(oracle_cfg_for(wl), inp["slot_to_expert"], fs, bias, inp["logits"])
            ok = (np.array_equal(out.topk_ids.cpu().numpy(), ids) and
                  np.array_equal(out.topk_slot.cpu().numpy(), slot))
            router.set_failed_ranks(failed)
            remap = {"host_call_us_median": statistics.median(host_us),
                     "added_latency_us_median": (statistics.median(with_remap) - statistics.median(steady)) * 1e6,
                     "step_us_median": statistics.median(steady) * 1e6,
                     "first_step_matches_oracle": bool(ok), "graph_recaptured": False,
                     "failure_sets_cycled": [list(s) for s in sets]}
        assert router.device_status() == 0

    # ---- roofline of the dominant kernel -----------------------------------
    peak, peak_kind = measured_peaks()
    alg = algorithmic_bytes(wl, T)
    dom = max(("k_scatter", "k_combine"), key=lambda n: dur_ms[n])
    achieved = alg[dom] / (dur_ms[dom] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": NCU_TRAFFIC_BYTES[dom] if (wl.name == "dsv3" and T == wl.T) else None,
                "algorithmic_bytes": alg[dom], "kernel_ms": dur_ms[dom],
                "per_kernel": {n: {"ms": dur_ms[n], "algorithmic_bytes": alg[n],
                                   "GB/s": alg[n] / (dur_ms[n] * 1e-3) / 1e9,
                                   "frac": alg[n] / (dur_ms[n] * 1e-3) / 1e9 / peak} for n in dur_ms},
                "step": {"algorithmic_bytes": sum(alg.values()),
                         "GB/s": sum(alg.values()) * K / (ms_total * 1e-3) / 1e9,
                         "frac": sum(alg.values()) * K / (ms_total * 1e-3) / 1e9 / peak,
                         "frac_of_8TBs_nominal": sum(alg.values()) * K / (ms_total * 1e-3) / 1e9 / 8000.0}}

    cpu_baseline = None
    if rank == 0 and world == 1:
        cpu_baseline = time_oracle(wl, inp, failed)

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(wl, failed), "T_per_gpu": T, "H": wl.H, "E": wl.E,
                       "k": wl.k, "slots": wl.P, "ranks": wl.R, "failed_ranks": list(failed),
                       "parallelism": f"token-sharded x{world}, no data-path collective",
                       "l2": f"inputs rotate over {N_INPUT_SETS} device copies ({N_INPUT_SETS} x "
                             f"{(T * wl.E * 4 + T * wl.H * 2) / 1e6:.0f} MB) and a step moves "
                             f"{sum(algorithmic_bytes(wl, T).values()) / 1e9:.2f} GB, both beyond the 126 MB L2; no flush",
                       "timed": f"CUDA-graph replays ({N_INPUT_SETS} consecutive steps per graph), CUDA events, max over ranks"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "remap": remap, "two_batches_in_flight": overlap,
            "expert_parallel_emulated": ep_leg}))
    router.close()
    if world > 1:
        dist.destroy_process_group()


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
    ap.add_argument("--expert-failure-sweep", action="store_true",
                    help="run the lost-expert sweep (throughput and load imbalance against r) instead of the benchmark")
    args = ap.parse_args()
    if args.expert_failure_sweep:
        return run_expert_failure_sweep(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
