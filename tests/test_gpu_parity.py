"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle,
element by element, on the same seeded inputs.  Integer outputs bit-exact,
weights within 1e-6 relative, combined output within 1e-2 relative or 1e-3
absolute."""
import dataclasses
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import (assert_y_close, bf16_bits, check_dispatch, make_router, run_and_check, to_dev)
from util import oracle_cfg, small_grouped_workload

pytestmark = pytest.mark.gpu

CASES = [(name, fi) for name, wl in W.WORKLOADS.items() for fi in range(len(wl.failure_sets))]


@pytest.mark.parametrize("name,fi", CASES)
def test_parity_reduced_tokens_ragged_tail(name, fi):
    # several routing tiles (32 tokens each) plus a ragged tail; full hidden width
    wl = W.WORKLOADS[name]
    T = wl.T if wl.T <= 128 else 1000 + 37
    inp = W.make_inputs(wl, T=T)
    run_and_check(wl, inp, wl.failure_sets[fi])


@pytest.mark.parametrize("name", ["mixtral", "dsv3", "qwen3"])
def test_parity_full_size(name):
    # the full workload in the launch configuration the benchmark times
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl)
    run_and_check(wl, inp, wl.failure_sets[-1])


def test_parity_full_size_kimi():
    # 32768 x 7168 with 448 slots, every output compared in full.  The 3.7 GB send buffer is
    # compared on the device against the rows the oracle's permutation names (a bit copy of
    # x[src_index // k]); the combined output y of all 32768 tokens is compared with the oracle,
    # which computes it chunk by chunk from those same rows.
    wl = W.WORKLOADS["kimi"]
    inp = W.make_inputs(wl)
    failed = wl.failure_sets[3]
    router = make_router(wl, inp, max_tokens=wl.T)
    router.set_failed_ranks(failed)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    out = router.dispatch(logits, x)
    y = router.combine(out.send_buf, wl.T)
    torch.cuda.synchronize()
    assert router.device_status() == 0
    cfg = oracle_cfg(wl)
    ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"])
    ref = oracle.permutation(cfg, slot)
    ref.update(topk_ids=ids, topk_weights=w, topk_slot=slot)
    check_dispatch(out, ref, check_send=False)
    # send buffer: row r is the bit copy of token ref.src_index[r] // k
    src_tok = torch.from_numpy(ref["src_index"].astype(np.int64) // wl.k).cuda()
    for lo in range(0, wl.T * wl.k, 1 << 16):
        hi = min(lo + (1 << 16), wl.T * wl.k)
        assert torch.equal(out.send_buf[lo:hi].view(torch.int16), x[src_tok[lo:hi]].view(torch.int16))
    # y: the oracle's combine on every token, 2048 tokens at a time (the rows of a chunk are its
    # tokens' x rows repeated k times, in assignment order)
    y_bits = bf16_bits(y)
    step = 2048
    for lo in range(0, wl.T, step):
        hi = min(lo + step, wl.T)
        rows = np.repeat(inp["x"][lo:hi], wl.k, axis=0)
        ref_y = oracle.combine(rows, np.arange(rows.shape[0], dtype=np.int32), w[lo:hi], slot[lo:hi],
                               inp["slot_scale"])
        assert_y_close(y_bits[lo:hi], ref_y)
    router.close()


@pytest.mark.parametrize("T", [0, 1, 31, 32, 33, 64, 65])
def test_token_counts_around_tile_edges(T):
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=max(T, 1), H=512)
    if T == 0:
        router = make_router(wl, inp, max_tokens=8, hidden=512)
        out = router.alloc_outputs(0)
        st = B.moe_dispatch(router._ctx, 0, 0, 0, out.as_struct(), 0)
        assert st == B.MOE_OK
        assert B.moe_combine(router._ctx, 0, 0, 0, 0) == B.MOE_OK
        router.close()
        return
    run_and_check(wl, inp, (7, 20))


@pytest.mark.parametrize("H", [8, 24, 264, 1000, 1032])
def test_odd_hidden_widths(H):
    wl = W.WORKLOADS["qwen3"]
    inp = W.make_inputs(wl, T=77, H=H)
    run_and_check(wl, inp, (5,))


def test_all_tokens_choose_the_same_experts():
    # identical logits for every token: k slots receive T rows each, the rest none
    wl = W.WORKLOADS["kimi"]
    inp = W.make_inputs(wl, T=700, H=256)
    inp["logits"][:] = inp["logits"][0]
    out, _, ref = run_and_check(wl, inp, ())
    assert (ref["slot_counts"] > 0).sum() <= 2 * wl.k


def test_ties_and_signed_zeros_follow_lower_id():
    wl = W.Workload("ties", T=64, H=64, E=64, k=4, R=8, S=8, seed=9, max_replicas=1)
    inp = W.make_inputs(wl)
    lg = np.round(inp["logits"] * 2) / 2          # many exact ties
    lg[lg == 0] = np.where(np.arange((lg == 0).sum()) % 2 == 0, 0.0, -0.0)
    inp["logits"] = lg.astype(np.float32)
    out, _, ref = run_and_check(wl, inp, (3,))
    srt = np.sort(lg, axis=1)
    assert (srt[:, -4] == srt[:, -5]).any(), "the case must contain ties at the selection boundary"


def test_minus_inf_logits_act_as_mask():
    for name in ("qwen3", "dsv3"):
        wl = W.WORKLOADS[name]
        inp = W.make_inputs(wl, T=200, H=128)
        rng = np.random.default_rng(1)
        inp["logits"][rng.random(inp["logits"].shape) < 0.2] = -np.inf
        run_and_check(wl, inp, wl.failure_sets[-1])


@pytest.mark.parametrize("E,k,n_group,topk_group", [(8, 2, 4, 2), (16, 4, 4, 2), (24, 6, 6, 3), (160, 6, 8, 3)])
def test_grouped_selection_small_shapes(E, k, n_group, topk_group):
    R = 8 if E % 8 == 0 else 4
    for score in (W.SOFTMAX, W.SIGMOID):
        wl = small_grouped_workload(E=E, k=k, n_group=n_group, topk_group=topk_group, R=R, S=E // R,
                                    score_func=score)
        wl = dataclasses.replace(wl, max_replicas=1)
        inp = W.make_inputs(wl, T=300, H=64)
        run_and_check(wl, inp, ())
        run_and_check(wl, inp, (1,))


def test_group_with_fewer_than_m_finite_keys():
    wl = W.Workload("thin-group", T=1, H=8, E=12, k=4, R=12, S=1, n_group=3, topk_group=2, max_replicas=1)
    inp = W.make_inputs(wl)
    inp["logits"] = np.array([[9.0, 8.0, 7.0, 6.0, 3.0, 2.5, 1.0, 0.0, 2.0, 2.0, 1.5, 0.1]], np.float32)
    out, _, _ = run_and_check(wl, inp, (1, 2, 3))
    assert out.topk_ids.cpu().tolist() == [[0, 4, 5, 6]]


def test_route_scale():
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=100, H=64)
    out, _, _ = run_and_check(wl, inp, (7,), route_scale=2.5)
    assert torch.allclose(out.topk_weights.sum(1), torch.full((100,), 2.5, device="cuda"), rtol=1e-5)


def test_bulk_copy_scatter_matches_oracle():
    bulk = {B.MOE_TUNE_SCATTER_IMPL: 1}
    for name, T in (("dsv3", 1037), ("tiny", 128), ("qwen3", 300)):
        wl = W.WORKLOADS[name]
        inp = W.make_inputs(wl, T=T)
        run_and_check(wl, inp, wl.failure_sets[-1], tuning=bulk)
    for stages in (1, 2, 8):
        wl = W.WORKLOADS["dsv3"]
        run_and_check(wl, W.make_inputs(wl, T=2048 + 5, H=1024), (7,),
                      tuning={**bulk, B.MOE_TUNE_SCATTER_BULK_STAGES: stages})


def test_combine_variants_match_oracle():
    # the register (vector-load) combine and other shapes of the bulk-copy ring
    settings = [{B.MOE_TUNE_COMBINE_IMPL: 0},
                {B.MOE_TUNE_COMBINE_IMPL: 1, B.MOE_TUNE_COMBINE_CHUNK: 2, B.MOE_TUNE_COMBINE_STAGES: 2},
                {B.MOE_TUNE_COMBINE_IMPL: 1, B.MOE_TUNE_COMBINE_CHUNK: 2, B.MOE_TUNE_COMBINE_STAGES: 6},
                {B.MOE_TUNE_COMBINE_IMPL: 1, B.MOE_TUNE_COMBINE_CHUNK: 4, B.MOE_TUNE_COMBINE_STAGES: 2}]
    for tuning in settings:
        for name, T, H in (("dsv3", 1037, None), ("mixtral", 300, 1000), ("tiny", 128, None), ("qwen3", 5, 8)):
            wl = W.WORKLOADS[name]
            run_and_check(wl, W.make_inputs(wl, T=T, H=H), wl.failure_sets[-1], tuning=tuning)


def test_routing_tile_and_lane_overrides_match_oracle():
    # other tile sizes (several tiles per SM count, one big tile) and 8 lanes per token
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=1037, H=256)
    for tuning in ({B.MOE_TUNE_ROUTE_TOKENS_PER_TILE: 8}, {B.MOE_TUNE_ROUTE_TOKENS_PER_TILE: 500},
                   {B.MOE_TUNE_ROUTE_LANES_PER_TOKEN: 8}, {B.MOE_TUNE_PDL: 0}):
        run_and_check(wl, inp, (7, 20), tuning=tuning)


def test_two_contexts_of_different_top_k_share_the_ring_kernel():
    # both shapes use the generic-k instantiation of the ring combine with different ring sizes;
    # creating the second context must not shrink what the first may launch with
    wl16 = W.Workload("k16", T=64, H=512, E=64, k=16, R=8, S=8, seed=5, max_replicas=1)
    wl6 = W.Workload("k6", T=64, H=512, E=64, k=6, R=8, S=8, seed=6, max_replicas=1)
    inp16, inp6 = W.make_inputs(wl16), W.make_inputs(wl6)
    r16 = make_router(wl16, inp16, max_tokens=64)
    r6 = make_router(wl6, inp6, max_tokens=64)
    for _ in range(2):
        run_and_check(wl16, inp16, (), router=r16)
        run_and_check(wl6, inp6, (), router=r6)
    r16.close(); r6.close()


def test_step_from_host_memory():
    wl = W.WORKLOADS["dsv3"]
    T = 500
    inp = W.make_inputs(wl, T=T)
    router = make_router(wl, inp, max_tokens=T)
    router.set_failed_ranks((7, 20))
    lg_h = torch.from_numpy(inp["logits"]).pin_memory()
    x_h = torch.from_numpy(inp["x"]).view(torch.int16).view(torch.bfloat16).pin_memory()
    y_h = torch.empty((T, wl.H), dtype=torch.bfloat16).pin_memory()
    lg_d, x_d = torch.empty_like(lg_h, device="cuda"), torch.empty_like(x_h, device="cuda")
    y_d = torch.empty((T, wl.H), dtype=torch.bfloat16, device="cuda")
    out = router.alloc_outputs(T)
    router.step_host(lg_h, x_h, out, lg_d, x_d, y_d, y_h)
    ref = oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], (7, 20), inp["bias"], inp["logits"], inp["x"])
    check_dispatch(out, ref)
    ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"], inp["slot_scale"])
    assert_y_close(y_h.view(torch.int16).numpy().view(np.uint16), ref_y)
    router.close()


def test_two_host_fed_steps_in_flight():
    # two contexts on two streams, nothing waited for until both steps are enqueued
    wl = W.WORKLOADS["qwen3"]
    T = 700
    parts = []
    for seed in (3, 4):
        inp = W.make_inputs(wl, T=T, seed=seed)
        router = make_router(wl, inp, max_tokens=T)
        router.set_failed_ranks((5,))
        parts.append(dict(
            inp=inp, router=router, stream=torch.cuda.Stream(), out=router.alloc_outputs(T),
            lg_h=torch.from_numpy(inp["logits"]).pin_memory(),
            x_h=torch.from_numpy(inp["x"]).view(torch.int16).view(torch.bfloat16).pin_memory(),
            y_h=torch.zeros((T, wl.H), dtype=torch.bfloat16).pin_memory(),
            lg_d=torch.empty((T, wl.E), dtype=torch.float32, device="cuda"),
            x_d=torch.empty((T, wl.H), dtype=torch.bfloat16, device="cuda"),
            y_d=torch.empty((T, wl.H), dtype=torch.bfloat16, device="cuda")))
    torch.cuda.synchronize()
    for _ in range(3):
        for p in parts:
            with torch.cuda.stream(p["stream"]):
                p["router"].step_host_async(p["lg_h"], p["x_h"], p["out"], p["lg_d"], p["x_d"], p["y_d"], p["y_h"])
    for p in parts:
        p["stream"].synchronize()
        inp = p["inp"]
        ref = oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], (5,), None, inp["logits"], inp["x"])
        check_dispatch(p["out"], ref)
        ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                               inp["slot_scale"])
        assert_y_close(p["y_h"].view(torch.int16).numpy().view(np.uint16), ref_y)
        assert p["router"].device_status() == 0
        p["router"].close()


def test_argument_validation_on_device():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    router = make_router(wl, inp, max_tokens=wl.T)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    out = router.alloc_outputs(wl.T)
    ctx = router._ctx
    assert B.moe_combine(ctx, out.send_buf.data_ptr(), wl.T, x.data_ptr(), 0) == B.MOE_ERR_INVALID_ARG  # no dispatch yet
    assert B.moe_dispatch(ctx, logits.data_ptr(), x.data_ptr(), wl.T + 1, out.as_struct(), 0) == B.MOE_ERR_CAPACITY
    assert B.moe_dispatch(ctx, logits.data_ptr(), x.data_ptr() + 2, wl.T, out.as_struct(), 0) == B.MOE_ERR_INVALID_ARG
    s = out.as_struct(); s.dst_row = None
    assert B.moe_dispatch(ctx, logits.data_ptr(), x.data_ptr(), wl.T, s, 0) == B.MOE_ERR_INVALID_ARG
    assert B.moe_dispatch(ctx, logits.data_ptr(), x.data_ptr(), wl.T, out.as_struct(), 0) == B.MOE_OK
    assert B.moe_combine(ctx, out.send_buf.data_ptr(), wl.T - 1, x.data_ptr(), 0) == B.MOE_ERR_INVALID_ARG
    torch.cuda.synchronize()
    router.close()


def test_device_status_reports_unroutable_token_and_recovers():
    wl = W.WORKLOADS["qwen3"]
    inp = W.make_inputs(wl, T=64, H=64)
    router = make_router(wl, inp, max_tokens=64, hidden=64)
    bad = inp["logits"].copy()
    bad[5, 3:] = -np.inf                      # token 5 has 3 < k selectable experts
    x = to_dev(inp["x"], torch.bfloat16)
    out = router.dispatch(to_dev(bad), x)
    torch.cuda.synchronize()
    assert router.device_status() == B.MOE_ERR_INSUFFICIENT_EXPERTS
    assert router.device_status() == 0        # reading clears it
    # outputs stay in range, so nothing was written out of bounds
    assert int(out.topk_slot.min()) >= 0 and int(out.topk_slot.max()) < wl.P
    assert int(out.slot_offsets[-1]) == 64 * wl.k
    router.close()
    run_and_check(wl, inp, (5,))
