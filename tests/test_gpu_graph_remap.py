"""Recovery on the GPU: a remap rewrites only the rank bitmap / replica table in
device memory, so one captured CUDA graph of dispatch + combine stays valid
across failures (the paper recompiles its graph instead, Sec. 3.6)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import assert_y_close, bf16_bits, check_dispatch, make_router, to_dev
from util import oracle_cfg

pytestmark = pytest.mark.gpu


def _capture(router, logits, x, T):
    out = router.alloc_outputs(T)
    y = torch.empty((T, router.cfg.hidden), dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):                                   # warm-up outside capture
            router.dispatch(logits, x, out)
            router.combine(out.send_buf, T, y)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        router.dispatch(logits, x, out)
        router.combine(out.send_buf, T, y)
    return graph, out, y


def _oracle_step(wl, inp, failed, s2e=None):
    s2e = inp["slot_to_expert"] if s2e is None else s2e
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    ref = oracle.dispatch(oracle_cfg(wl), s2e, failed, bias, inp["logits"], inp["x"])
    ref["y"] = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                              inp["slot_scale"])
    return ref


@pytest.mark.parametrize("name", ["tiny", "dsv3", "kimi"])
def test_one_graph_survives_a_sweep_of_failures(name):
    wl = W.WORKLOADS[name]
    T, H = min(wl.T, 600), min(wl.H, 512)
    inp = W.make_inputs(wl, T=T, H=H)
    router = make_router(wl, inp, max_tokens=T, hidden=H)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    graph, out, y = _capture(router, logits, x, T)
    sets = list(wl.failure_sets) + [()]
    for failed in sets:
        router.set_failed_ranks(failed)          # between replays, on the replay stream
        graph.replay()                           # the same executable graph every time
        torch.cuda.synchronize()
        ref = _oracle_step(wl, inp, failed)
        check_dispatch(out, ref)
        assert_y_close(bf16_bits(y), ref["y"])
        if failed:
            assert not np.isin(out.topk_slot.cpu().numpy() // wl.S, list(failed)).any()
            assert int(out.rank_counts.cpu()[list(failed)].sum()) == 0
    assert router.device_status() == 0
    router.close()


def test_replays_are_bit_identical():
    wl = W.WORKLOADS["dsv3"]
    T = 2048
    inp = W.make_inputs(wl, T=T, H=1024)
    router = make_router(wl, inp, max_tokens=T, hidden=1024)
    router.set_failed_ranks((7,))
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    graph, out, y = _capture(router, logits, x, T)
    graph.replay()
    torch.cuda.synchronize()
    first = {f: getattr(out, f).clone() for f in out.__dataclass_fields__}
    y0 = y.clone()
    for _ in range(20):
        graph.replay()
    torch.cuda.synchronize()
    for f, v in first.items():
        assert torch.equal(getattr(out, f).view(torch.int32) if v.dtype == torch.float32 else getattr(out, f),
                           v.view(torch.int32) if v.dtype == torch.float32 else v), f
    assert torch.equal(y.view(torch.int16), y0.view(torch.int16))
    router.close()


def test_rejected_remap_leaves_device_state_untouched():
    wl = W.WORKLOADS["mixtral"]
    inp = W.make_inputs(wl, T=200, H=128)
    router = make_router(wl, inp, max_tokens=200, hidden=128)
    router.set_failed_ranks((3,))
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    with pytest.raises(B.MoeError) as e:
        router.set_failed_ranks((0, 1, 2, 3, 4, 5, 6))     # one expert left < k = 2
    assert e.value.status == B.MOE_ERR_INSUFFICIENT_EXPERTS
    with pytest.raises(B.MoeError) as e:
        router.set_failed_ranks((8,))
    assert e.value.status == B.MOE_ERR_INVALID_ARG
    out = router.dispatch(logits, x)
    torch.cuda.synchronize()
    check_dispatch(out, _oracle_step(wl, inp, (3,)))
    router.close()


def test_failed_ranks_equal_emptied_slots_in_the_map():
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=300, H=128)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    failed = (7, 20)
    a = make_router(wl, inp, max_tokens=300, hidden=128)
    a.set_failed_ranks(failed)
    out_a = a.dispatch(logits, x)
    b = make_router(wl, inp, max_tokens=300, hidden=128)
    s2e = inp["slot_to_expert"].copy()
    for r in failed:
        s2e[r * wl.S:(r + 1) * wl.S] = -1
    b.update_replica_map(s2e)
    out_b = b.dispatch(logits, x)
    torch.cuda.synchronize()
    for f in out_a.__dataclass_fields__:
        assert torch.equal(getattr(out_a, f), getattr(out_b, f)), f
    check_dispatch(out_b, _oracle_step(wl, inp, (), s2e))
    # moving a replica: expert 0 gains a copy on the last rank's spare slot if it is empty
    a.close(); b.close()


def test_many_back_to_back_remaps_keep_order():
    wl = W.WORKLOADS["kimi"]
    inp = W.make_inputs(wl, T=128, H=64)
    router = make_router(wl, inp, max_tokens=128, hidden=64)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    rng = np.random.default_rng(2)
    last = ()
    for i in range(50):                          # more than the staging ring holds
        last = tuple(int(r) for r in rng.choice(wl.R, int(rng.integers(0, 6)), replace=False))
        router.set_failed_ranks(last)
    out = router.dispatch(logits, x)
    torch.cuda.synchronize()
    check_dispatch(out, _oracle_step(wl, inp, last))
    router.close()


def test_remap_while_capturing_is_refused():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    router = make_router(wl, inp, max_tokens=wl.T)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        st = B.moe_set_failed_ranks(router._ctx, [2], torch.cuda.current_stream().cuda_stream)
        torch.zeros(1, device="cuda").add_(1)
    assert st == B.MOE_ERR_INVALID_ARG
    router.close()


@pytest.mark.parametrize("name,T,replays", [("tiny", 128, 6000), ("dsv3", 2048, 1500)])
def test_long_run_of_replays_with_remaps_stays_exact(name, T, replays):
    # thousands of back-to-back replays of one graph, a remap every 37 steps: the look-back
    # descriptors are recycled by their epoch tag and the ticket resets every step, so a rare
    # ordering slip would show up as a changed result, a wrong total or a device status
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=T)
    router = make_router(wl, inp, max_tokens=T)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)      # the graph reads these: keep them
    graph, out, y = _capture(router, logits, x, T)
    sets = list(wl.failure_sets)
    seen = {}
    for i in range(replays):
        if i % 37 == 0:
            failed = sets[(i // 37) % len(sets)]
            router.set_failed_ranks(failed)
        graph.replay()
        if i % 211 == 0 or i == replays - 1:
            torch.cuda.synchronize()
            assert int(out.slot_offsets[-1]) == T * wl.k
            sig = (out.dst_row.clone(), y.clone())
            if tuple(failed) in seen:
                assert torch.equal(seen[tuple(failed)][0], sig[0]) and torch.equal(seen[tuple(failed)][1], sig[1])
            seen.setdefault(tuple(failed), sig)
    assert router.device_status() == 0
    # and the result is the right one, not just a stable one
    ref = _oracle_step(wl, inp, failed)
    check_dispatch(out, ref)
    assert_y_close(bf16_bits(y), ref["y"])
    router.close()


@pytest.mark.parametrize("name", ["dsv3", "qwen3"])
def test_random_sequence_of_remaps_under_one_graph(name):
    # every kind of remap (failed ranks, lost experts, rank order, replica map), drawn at random and
    # applied between replays of one captured graph; a rejected remap must leave the state as it was
    import dataclasses
    wl = dataclasses.replace(W.WORKLOADS[name], H=64)
    T = 300
    inp = W.make_inputs(wl, T=T)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = make_router(wl, inp, max_tokens=T)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    graph, out, y = _capture(router, logits, x, T)
    rng = np.random.default_rng(5)
    failed, lost, order, s2e = (), np.zeros(wl.E, np.uint8), None, inp["slot_to_expert"].copy()
    applied = rejected = 0
    for _ in range(120):
        op = int(rng.integers(0, 4))
        nf, nl, no, ns = failed, lost, order, s2e
        try:
            if op == 0:
                nf = tuple(int(r) for r in rng.choice(wl.R, int(rng.integers(0, max(2, wl.R // 3))), replace=False))
                router.set_failed_ranks(nf)
            elif op == 1:
                nl = (rng.random(wl.E) < rng.choice([0.0, 0.05, 0.3])).astype(np.uint8)
                router.set_failed_experts(nl)
            elif op == 2:
                alive = [r for r in range(wl.R) if r not in failed]
                no = [int(r) for r in rng.permutation(alive)] if rng.random() < 0.7 else None
                router.set_rank_order(no if no is not None else [])
            else:
                ns = s2e.copy()
                i, j = rng.integers(0, wl.P, 2)
                ns[i], ns[j] = ns[j], ns[i]
                router.update_replica_map(ns)
            failed, lost, order, s2e = nf, nl, no, ns
            applied += 1
        except B.MoeError:
            rejected += 1
        graph.replay()
        torch.cuda.synchronize()
        assert router.device_status() == 0
        ref = oracle.dispatch(oracle_cfg(wl), s2e, failed, bias, inp["logits"], inp["x"], lost, order)
        check_dispatch(out, ref)
        assert_y_close(bf16_bits(y), oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"],
                                                    ref["topk_slot"], inp["slot_scale"]))
    assert applied > 60 and rejected > 0
    router.close()
