"""Expert parallelism over several GPUs (Sec. 2.3: dispatch and combine as exchanges between devices).

CPU part: the plain multi-GPU oracle is pinned against the single-GPU oracle, a library
sort and a closed form; the library's host-side layout arithmetic and a two-process gloo
run of the count exchange are checked against it.  GPU part: a whole group emulated on
one device (peers = buffers of the same device) against the oracle, bit for bit.
"""
import dataclasses
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2602_21140_b200 import workloads as W
from util import bf16_to_f64, oracle_cfg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def small(name, H=64):
    return dataclasses.replace(W.WORKLOADS[name], H=H)


def batches(wl, world, T_list):
    """One seeded batch per sender; placement, bias and scales are shared."""
    inps = [W.make_inputs(wl, T=max(T, 1), seed=wl.seed + 1000 * g) for g, T in enumerate(T_list)]
    for inp, T in zip(inps, T_list):
        inp["logits"], inp["x"] = inp["logits"][:T], inp["x"][:T]
    return inps


def run_oracle(wl, world, inps, failed):
    cfg = oracle_cfg(wl)
    bias = inps[0]["bias"] if wl.score_func == W.SIGMOID else None
    return cfg, oracle.ep_dispatch(cfg, world, inps[0]["slot_to_expert"], failed, bias,
                                   [i["logits"] for i in inps], [i["x"] for i in inps])


# ------------------------------------------------------------------ oracle pins (CPU)

def test_world_one_is_the_single_gpu_dispatch():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    cfg, (snd, own) = run_oracle(wl, 1, [inp], wl.failure_sets[0])
    ref = oracle.dispatch(cfg, inp["slot_to_expert"], wl.failure_sets[0], None, inp["logits"], inp["x"])
    assert np.array_equal(own[0]["recv_buf"], ref["send_buf"])
    assert np.array_equal(snd[0]["dst_row"], ref["dst_row"])
    assert np.array_equal(own[0]["recv_slot_offsets"], ref["slot_offsets"])


@pytest.mark.parametrize("world", [2, 4, 8])
def test_layout_is_a_sort_by_slot_sender_assignment(world):
    wl = small("dsv3")
    inps = batches(wl, world, [37, 5, 64, 1, 0, 23, 48, 9][:world])
    _, (snd, own) = run_oracle(wl, world, inps, (7,))
    spg = wl.P // world
    # every assignment of every sender, sorted by (slot, sender, i) with a library sort
    slot = np.concatenate([s["topk_slot"].reshape(-1) for s in snd])
    sender = np.concatenate([np.full(s["topk_slot"].size, g) for g, s in enumerate(snd)])
    idx = np.concatenate([np.arange(s["topk_slot"].size) for s in snd])
    order = np.lexsort((idx, sender, slot))
    for d in range(world):
        mine = order[(slot[order] // spg) == d]
        assert np.array_equal(own[d]["recv_src"], np.stack([sender[mine], idx[mine]], axis=1))
        rows = np.stack([inps[g]["x"][i // wl.k] for g, i in own[d]["recv_src"]]) if len(mine) else \
            np.zeros((0, wl.H), np.uint16)
        assert np.array_equal(own[d]["recv_buf"], rows)
        counts = np.bincount(slot[mine] - d * spg, minlength=spg)
        assert np.array_equal(np.diff(own[d]["recv_slot_offsets"]), counts)
    total = sum(o["recv_buf"].shape[0] for o in own)
    assert total == sum(i["logits"].shape[0] for i in inps) * wl.k
    # no slot of a failed rank receives anything
    d7, q0 = (7 * wl.S) // spg, (7 * wl.S) % spg
    off = own[d7]["recv_slot_offsets"]
    assert off[q0 + wl.S] == off[q0]


def test_without_redundancy_the_group_equals_one_big_batch():
    # no replicas: the slot of (t, e) does not depend on t, so the buffers of the group, one after
    # the other, are the send buffer of a single dispatch over the concatenated batches
    wl = small("qwen3")
    world = 4
    inps = batches(wl, world, [19, 40, 3, 26])
    cfg, (snd, own) = run_oracle(wl, world, inps, (5,))
    logits = np.concatenate([i["logits"] for i in inps])
    x = np.concatenate([i["x"] for i in inps])
    ref = oracle.dispatch(cfg, inps[0]["slot_to_expert"], (5,), None, logits, x)
    assert np.array_equal(np.concatenate([o["recv_buf"] for o in own]), ref["send_buf"])


def test_combine_closed_form():
    wl = small("dsv3")
    world = 4
    inps = batches(wl, world, [16, 33, 8, 21])
    cfg, (snd, own) = run_oracle(wl, world, inps, (7, 20))
    scale = inps[0]["slot_scale"]
    for g in range(world):
        y = bf16_to_f64(oracle.ep_combine(cfg, world, g, snd[g], own, scale))
        c = (snd[g]["topk_weights"] * scale[snd[g]["topk_slot"]]).astype(np.float64).sum(axis=1)
        want = c[:, None] * bf16_to_f64(inps[g]["x"])
        assert np.all(np.abs(y - want) <= 2.0 ** -7 * np.abs(want) + 1e-30)


# ------------------------------------------------------------------ host logic of the library (CPU)

def test_plan_host_matches_the_oracle_layout():
    from paper_2602_21140_b200 import binding as B
    wl = small("kimi")
    world = 8
    inps = batches(wl, world, [11, 0, 25, 7, 30, 2, 18, 13])
    _, (snd, own) = run_oracle(wl, world, inps, wl.failure_sets[3])
    counts_all = np.stack([s["slot_counts"] for s in snd])
    spg = wl.P // world
    covered = [np.zeros(o["recv_buf"].shape[0], np.int32) for o in own]
    for g in range(world):
        st, src_base, recv_off = B.moe_ep_plan_host(counts_all, g)
        assert st == B.MOE_OK
        assert np.array_equal(recv_off, own[g]["recv_slot_offsets"])
        flat = snd[g]["topk_slot"].reshape(-1)
        for p in range(wl.P):
            mine = np.nonzero(flat == p)[0]
            if mine.size:
                assert src_base[p] == snd[g]["dst_row"][mine].min()
                covered[p // spg][src_base[p]: src_base[p] + mine.size] += 1
    for c in covered:                      # the senders' row ranges tile every buffer exactly once
        assert np.all(c == 1)


def test_plan_host_rejects_bad_arguments():
    from paper_2602_21140_b200 import binding as B
    counts = np.zeros((2, 9), np.int32)                     # 9 slots do not split over 2 GPUs
    assert B.moe_ep_plan_host(counts, 0)[0] == B.MOE_ERR_INVALID_ARG
    counts = np.zeros((2, 8), np.int32)
    assert B.moe_ep_plan_host(counts, 2)[0] == B.MOE_ERR_INVALID_ARG
    assert B.moe_ep_plan_host(counts, -1)[0] == B.MOE_ERR_INVALID_ARG
    counts[:] = 2 ** 30                                     # offsets beyond 31 bits
    assert B.moe_ep_plan_host(counts, 1)[0] == B.MOE_ERR_CAPACITY


WORKER = r"""
import dataclasses, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"]); sys.path.insert(0, os.path.join(os.environ["REPO_ROOT"], "tests"))
import numpy as np
import torch
import torch.distributed as dist
import oracle
from paper_2602_21140_b200 import binding as B, ep, workloads as W
from util import oracle_cfg

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
wl = dataclasses.replace(W.WORKLOADS["mixtral"], H=32)
T = [29, 14][rank]
inp = W.make_inputs(wl, T=T, seed=wl.seed + 1000 * rank)
cfg = oracle_cfg(wl)
ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], (3,), None, inp["logits"])
counts = torch.from_numpy(np.bincount(slot.reshape(-1), minlength=wl.P).astype(np.int32))
counts_all = ep.gather_counts(counts)                      # the exchange every rank performs
assert counts_all.shape == (world, wl.P) and torch.equal(counts_all[rank], counts)
st, src_base, recv_off = B.moe_ep_plan_host(counts_all.numpy(), rank)
assert st == B.MOE_OK
everything = [None] * world
dist.all_gather_object(everything, dict(logits=inp["logits"], x=inp["x"], src_base=src_base, recv_off=recv_off,
                                        slot=slot))
if rank == 0:
    snd, own = oracle.ep_dispatch(cfg, world, inp["slot_to_expert"], (3,), None,
                                  [e["logits"] for e in everything], [e["x"] for e in everything])
    for g, e in enumerate(everything):
        assert np.array_equal(e["slot"], snd[g]["topk_slot"])
        assert np.array_equal(e["recv_off"], own[g]["recv_slot_offsets"])
        flat = e["slot"].reshape(-1)
        for i in range(flat.size):                         # first row + rank inside the sender's run
            pos = int(np.count_nonzero(flat[:i] == flat[i]))
            assert e["src_base"][flat[i]] + pos == snd[g]["dst_row"][i]
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_count_exchange_and_layout_two_ranks_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=300)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0 and f"rank {r} ok" in o, o


# ------------------------------------------------------------------ emulated group on one GPU

def _check_group(wl, world, T_list, failed, recv_rows=None):
    import torch
    from gpu_util import WEIGHT_RTOL, assert_y_close, bf16_bits, to_dev
    from paper_2602_21140_b200 import binding as B, ep

    inps = batches(wl, world, T_list)
    cfg, (snd, own) = run_oracle(wl, world, inps, failed)
    bias = inps[0]["bias"] if wl.score_func == W.SIGMOID else None
    rows = recv_rows if recv_rows is not None else max(1, sum(T_list) * wl.k)
    group = ep.EmulatedEpGroup(world, B.config_for_workload(wl, max_tokens=max(max(T_list), 1)),
                               inps[0]["slot_to_expert"], bias, inps[0]["slot_scale"], rows)
    group.set_failed_ranks(failed)
    logits = [to_dev(i["logits"]) for i in inps]
    x = [to_dev(i["x"], torch.bfloat16) for i in inps]
    for _ in range(2):                                       # twice: the second step overwrites the first
        outs = group.dispatch(logits, x)
        ys = group.combine(T_list)
    torch.cuda.synchronize()
    assert group.device_status() == [0] * world
    for g in range(world):
        if T_list[g] == 0:
            assert int(outs[g].slot_counts.sum()) == 0
            continue
        for f in ("topk_ids", "topk_slot", "slot_counts", "dst_row"):
            assert np.array_equal(getattr(outs[g], f).cpu().numpy().reshape(-1), snd[g][f].reshape(-1)), (g, f)
        w = outs[g].topk_weights.cpu().numpy().astype(np.float64)
        rw = snd[g]["topk_weights"].astype(np.float64)
        assert np.all(np.abs(w - rw) <= WEIGHT_RTOL * np.abs(rw))
        assert_y_close(bf16_bits(ys[g]), oracle.ep_combine(cfg, world, g, snd[g], own, inps[0]["slot_scale"]))
    for d in range(world):
        n = own[d]["recv_buf"].shape[0]
        assert np.array_equal(group.recv_slot_offsets[d].cpu().numpy(), own[d]["recv_slot_offsets"])
        assert np.array_equal(bf16_bits(group.recv_bufs[d][:n]), own[d]["recv_buf"]), d
    group.close()


@pytest.mark.gpu
@pytest.mark.parametrize("name,world,T_list,failed", [
    ("mixtral", 1, [200], (3,)),
    ("mixtral", 2, [129, 64], (3,)),
    ("qwen3", 4, [77, 300, 1, 150], (5,)),
    ("dsv3", 4, [260, 31, 0, 512], (7, 20)),
    ("dsv3", 8, [64, 3, 100, 0, 257, 19, 88, 40], ()),
    ("kimi", 8, [50, 120, 7, 33, 256, 0, 91, 12], None),
])
def test_emulated_group_matches_oracle(name, world, T_list, failed):
    wl = small(name, H=256)
    _check_group(wl, world, T_list, wl.failure_sets[4] if failed is None else failed)


@pytest.mark.gpu
def test_emulated_group_full_width_rows():
    # the real row width of the DeepSeek-V3 shape (one warp moves a whole 14 KB row)
    _check_group(W.WORKLOADS["dsv3"], 4, [96, 130, 57, 200], (7,))


@pytest.mark.gpu
def test_receive_buffer_overflow_is_reported_and_nothing_is_written_outside():
    import torch
    from gpu_util import to_dev
    from paper_2602_21140_b200 import binding as B, ep

    wl = small("mixtral", H=64)
    world, T_list, rows = 2, [128, 128], 40                  # far too few rows
    inps = batches(wl, world, T_list)
    group = ep.EmulatedEpGroup(world, B.config_for_workload(wl, max_tokens=128), inps[0]["slot_to_expert"],
                               None, inps[0]["slot_scale"], rows)
    # put each receive buffer in front of a guard zone
    guarded = [torch.full((rows + 64, wl.H), 7.0, dtype=torch.bfloat16, device="cuda") for _ in range(world)]
    for g, r in enumerate(group.routers):
        r.ep_attach(world, g, [b.data_ptr() for b in guarded], rows)
    group.dispatch([to_dev(i["logits"]) for i in inps], [to_dev(i["x"], torch.bfloat16) for i in inps])
    torch.cuda.synchronize()
    assert all(code == B.MOE_ERR_CAPACITY for code in group.device_status())
    for b in guarded:
        assert bool((b[rows:] == 7.0).all())
    # The combine that follows (in a captured group step the host cannot step in between) must
    # not follow the rows that did not fit: they are recorded as dst_row = -1 and contribute
    # zero, so y is the closed form c_t * x restricted to the rows that were placed.
    ys = group.combine(T_list)
    torch.cuda.synchronize()
    for g, (inp, out, y) in enumerate(zip(inps, group.outs, ys)):
        dst = out.dst_row.cpu().numpy().reshape(-1, wl.k)
        assert ((dst >= -1) & (dst < rows)).all() and (dst == -1).any()
        w = out.topk_weights.cpu().numpy().astype(np.float64)
        scale = inps[0]["slot_scale"].astype(np.float64)[out.topk_slot.cpu().numpy()]   # the group's scales
        c = w * scale * (dst >= 0)
        want = c.sum(1)[:, None] * W.bf16_bits_to_f32(inp["x"]).astype(np.float64)
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        assert ((err <= 1e-2 * np.abs(want)) | (err <= 1e-3)).all()
    for b in guarded:
        assert bool((b[rows:] == 7.0).all())
    group.close()


@pytest.mark.gpu
def test_ep_argument_checks():
    import torch
    from paper_2602_21140_b200 import binding as B

    wl = small("mixtral", H=64)
    inp = W.make_inputs(wl, T=8)
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=8), inp["slot_to_expert"], None, inp["slot_scale"])
    buf = torch.zeros((64, wl.H), dtype=torch.bfloat16, device="cuda")
    out = router.alloc_outputs(8)
    # not attached yet
    assert B.moe_ep_route(router._ctx, 0, 0, out.as_struct()) == B.MOE_ERR_INVALID_ARG
    # 8 ranks do not split over 3 GPUs; bad rank; misaligned buffer
    assert B.moe_ep_attach(router._ctx, 3, 0, [buf.data_ptr()] * 3, 64) == B.MOE_ERR_INVALID_ARG
    assert B.moe_ep_attach(router._ctx, 2, 2, [buf.data_ptr()] * 2, 64) == B.MOE_ERR_INVALID_ARG
    assert B.moe_ep_attach(router._ctx, 2, 0, [buf.data_ptr() + 2] * 2, 64) == B.MOE_ERR_INVALID_ARG
    assert B.moe_ep_attach(router._ctx, 2, 0, [buf.data_ptr()] * 2, 64) == B.MOE_OK
    # scatter and combine need a preceding moe_ep_route with the same T
    cnt = torch.zeros((2, wl.P), dtype=torch.int32, device="cuda")
    off = torch.zeros(wl.P // 2 + 1, dtype=torch.int32, device="cuda")
    x = torch.zeros((8, wl.H), dtype=torch.bfloat16, device="cuda")
    assert B.moe_ep_scatter(router._ctx, x.data_ptr(), 8, cnt.data_ptr(), off.data_ptr()) == B.MOE_ERR_INVALID_ARG
    assert B.moe_ep_combine(router._ctx, 8, x.data_ptr()) == B.MOE_ERR_INVALID_ARG
    # a single-GPU combine must not follow a multi-GPU routing
    lg = torch.zeros((8, wl.E), dtype=torch.float32, device="cuda")
    assert B.moe_ep_route(router._ctx, lg.data_ptr(), 8, out.as_struct()) == B.MOE_OK
    assert B.moe_combine(router._ctx, buf.data_ptr(), 8, x.data_ptr()) == B.MOE_ERR_INVALID_ARG
    torch.cuda.synchronize()
    router.close()


DIST_WORKER = r"""
import dataclasses, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"]); sys.path.insert(0, os.path.join(os.environ["REPO_ROOT"], "tests"))
import numpy as np
import torch
import torch.distributed as dist
import oracle
from paper_2602_21140_b200 import binding as B, ep, workloads as W
from gpu_util import assert_y_close, bf16_bits, to_dev
from util import oracle_cfg

torch.cuda.set_device(0)
dist.init_process_group("nccl", device_id=torch.device("cuda", 0))
wl = dataclasses.replace(W.WORKLOADS["mixtral"], H=256)
T = 300
inp = W.make_inputs(wl, T=T)
group = ep.DistributedEp(B.config_for_workload(wl, max_tokens=T), inp["slot_to_expert"], None,
                         inp["slot_scale"], T * wl.k, "cuda:0")
group.router.set_failed_ranks((3,))
out = group.router.alloc_outputs(T)
group.dispatch(to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16), out)
y = group.combine(T)
torch.cuda.synchronize()
assert group.router.device_status() == 0
cfg = oracle_cfg(wl)
ref = oracle.dispatch(cfg, inp["slot_to_expert"], (3,), None, inp["logits"], inp["x"])
assert np.array_equal(bf16_bits(group.recv_buf), ref["send_buf"])
assert np.array_equal(out.dst_row.cpu().numpy(), ref["dst_row"])
assert_y_close(bf16_bits(y), oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"],
                                            ref["topk_slot"], inp["slot_scale"]))
group.close()
dist.destroy_process_group()
print("distributed ok")
"""


@pytest.mark.gpu
def test_distributed_form_with_a_group_of_one():
    # the one-process-per-GPU orchestration (NCCL all-gather of the counts, symmetric-memory
    # receive buffer, peer pointer table) on the only group this machine can form
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port), REPO_ROOT=ROOT, TORCH_SYMM_MEM_DISABLE_MULTICAST="1",
               NCCL_NVLS_ENABLE="0")
    p = subprocess.run([sys.executable, "-c", DIST_WORKER], env=env, stdout=subprocess.PIPE,
                       stderr=subprocess.STDOUT, text=True, timeout=600)
    assert p.returncode == 0 and "distributed ok" in p.stdout, p.stdout[-3000:]


@pytest.mark.gpu
def test_captured_group_step_survives_remaps():
    # the exchange entry points allocate nothing: a whole group step captured once in a CUDA graph
    # stays correct when the failure set changes between replays (no recapture)
    import torch
    from gpu_util import assert_y_close, bf16_bits, to_dev
    from paper_2602_21140_b200 import binding as B

    wl = small("dsv3", H=256)
    world, T_list = 4, [96, 160, 33, 128]
    inps = batches(wl, world, T_list)
    bias = inps[0]["bias"]
    routers = [B.MoeRouter(B.config_for_workload(wl, max_tokens=max(T_list)), inps[0]["slot_to_expert"], bias,
                           inps[0]["slot_scale"]) for _ in range(world)]
    rows = sum(T_list) * wl.k
    recv = [torch.zeros((rows, wl.H), dtype=torch.bfloat16, device="cuda") for _ in range(world)]
    counts_all = torch.zeros((world, wl.P), dtype=torch.int32, device="cuda")
    offs = [torch.zeros(wl.P // world + 1, dtype=torch.int32, device="cuda") for _ in range(world)]
    logits = [to_dev(i["logits"]) for i in inps]
    x = [to_dev(i["x"], torch.bfloat16) for i in inps]
    outs, ys = [], []
    for g, r in enumerate(routers):
        r.ep_attach(world, g, [b.data_ptr() for b in recv], rows)
        o = r.alloc_outputs(T_list[g])
        o.slot_counts = counts_all[g]                       # on one device the all-gather is a view
        outs.append(o)
        ys.append(torch.empty((T_list[g], wl.H), dtype=torch.bfloat16, device="cuda"))

    def step():
        for g, r in enumerate(routers):
            r.ep_route(logits[g], outs[g])
        for g, r in enumerate(routers):
            r.ep_scatter(x[g], counts_all, offs[g])
        for g, r in enumerate(routers):
            r.ep_combine(T_list[g], ys[g])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for failed in [(), (7,), (7, 20), ()]:
        for r in routers:
            r.set_failed_ranks(failed)
        graph.replay()
        torch.cuda.synchronize()
        cfg, (snd, own) = run_oracle(wl, world, inps, failed)
        for g in range(world):
            assert np.array_equal(outs[g].dst_row.cpu().numpy(), snd[g]["dst_row"]), (failed, g)
            assert_y_close(bf16_bits(ys[g]), oracle.ep_combine(cfg, world, g, snd[g], own, inps[0]["slot_scale"]))
        for d in range(world):
            n = own[d]["recv_buf"].shape[0]
            assert np.array_equal(bf16_bits(recv[d][:n]), own[d]["recv_buf"]), (failed, d)
    for r in routers:
        assert r.device_status() == 0
        r.close()
