"""GPU parity at the edges of the supported shapes: most experts, largest k,
most replicas per expert, many slots, large routing tiles, tokens far below
max_tokens."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import assert_y_close, bf16_bits, check_dispatch, run_and_check, to_dev
from util import oracle_cfg

pytestmark = pytest.mark.gpu


def _replicated_layout(E, R, S, copies):
    """Copy c of expert e lives on rank (e + c * R / copies) mod R: `copies` distinct ranks each."""
    assert E * copies == R * S and R % copies == 0
    s2e = np.full(R * S, -1, np.int32)
    used = [0] * R
    for e in range(E):
        for c in range(copies):
            r = (e + c * (R // copies)) % R
            s2e[r * S + used[r]] = e
            used[r] += 1
    return s2e


@pytest.mark.parametrize("score", [W.SOFTMAX, W.SIGMOID])
def test_most_experts_largest_k(score):
    wl = W.Workload("wide", T=300, H=64, E=512, k=16, R=64, S=8, score_func=score, seed=41, max_replicas=1)
    run_and_check(wl, W.make_inputs(wl), (3, 17))


def test_grouped_at_512_experts():
    wl = W.Workload("wide-grouped", T=200, H=64, E=512, k=8, R=64, S=8, score_func=W.SIGMOID,
                    n_group=8, topk_group=4, seed=42, max_replicas=1)
    run_and_check(wl, W.make_inputs(wl), (0, 63))


def test_eight_replicas_per_expert_and_many_failures():
    E, R, S = 32, 32, 8
    wl = W.Workload("replicated", T=500, H=64, E=E, k=4, R=R, S=S, seed=43, max_replicas=8)
    inp = W.make_inputs(dataclasses.replace(wl, max_replicas=1, R=4, S=8))     # logits / x / bias only
    inp["slot_to_expert"] = _replicated_layout(E, R, S, 8)
    inp["slot_scale"] = np.random.default_rng(2).uniform(0.5, 1.5, R * S).astype(np.float32)
    for failed in [(), (1,), tuple(range(0, 32, 2)), tuple(range(1, 29))]:
        if not oracle.failure_set_ok(oracle_cfg(wl), inp["slot_to_expert"], failed):
            continue
        out, _, ref = run_and_check(wl, inp, failed)
        assert len(np.unique(ref["topk_slot"])) > wl.k       # replicas are actually spread over


def test_many_slots():
    wl = W.Workload("slots", T=400, H=64, E=256, k=8, R=128, S=8, seed=44, max_replicas=1)   # 1024 slots
    inp = W.make_inputs(dataclasses.replace(wl, R=32, S=8))
    s2e = np.full(wl.P, -1, np.int32)
    s2e[::4] = np.arange(256)                                  # experts on every fourth slot
    inp["slot_to_expert"] = s2e
    inp["slot_scale"] = np.random.default_rng(3).uniform(0.5, 1.5, wl.P).astype(np.float32)
    run_and_check(wl, inp, (5, 77))


@pytest.mark.parametrize("E,k,R,S", [(512, 8, 368, 8), (512, 8, 256, 4), (8, 2, 2900, 1)])
def test_shapes_whose_routing_tables_share_shared_memory(E, k, R, S):
    # so many slots or experts that the histogram's count matrix reuses the token phase's tables
    P = R * S
    assert B.moe_workspace_bytes(B.make_config(E, k, 64, 300, R, S, 1)) > 0
    wl = W.Workload("edge", T=300, H=64, E=E, k=k, R=R, S=S, seed=51, max_replicas=1)
    inp = W.make_inputs(dataclasses.replace(wl, R=max(E // 8, 1), S=8))     # logits / x / bias only
    s2e = np.full(P, -1, np.int32)
    s2e[np.linspace(0, P - 1, E).astype(int)] = np.arange(E)
    inp["slot_to_expert"] = s2e
    inp["slot_scale"] = np.random.default_rng(3).uniform(0.5, 1.5, P).astype(np.float32)
    run_and_check(wl, inp, (1, 5))


@pytest.mark.parametrize("max_tokens", [5000, 40000, 131072])
def test_large_routing_tiles_and_partial_batches(max_tokens):
    # the routing tile grows with max_tokens (64 ... 1024 tokens); batches far below it still work
    wl = W.WORKLOADS["dsv3"]
    for T in (1, 777, 4500):
        inp = W.make_inputs(wl, T=T, H=64)
        cfg = B.config_for_workload(wl, max_tokens=max_tokens, hidden=64)
        router = B.MoeRouter(cfg, inp["slot_to_expert"], inp["bias"], inp["slot_scale"])
        router.set_failed_ranks((7, 20))
        run_and_check(wl, inp, (7, 20), router=router)
        router.close()


def test_config_limits_are_enforced():
    wl = W.WORKLOADS["dsv3"]
    for field, value in (("max_tokens", 262145), ("num_experts", 513), ("top_k", 17), ("max_replicas", 9)):
        cfg = B.config_for_workload(wl)
        setattr(cfg, field, value)
        assert B.moe_workspace_bytes(cfg) == 0, field
    cfg = B.config_for_workload(wl, max_tokens=262144)
    assert B.moe_workspace_bytes(cfg) > 0


@pytest.mark.parametrize("H,k", [(16384, 8), (8200, 4), (32768, 2), (12288, 16)])
def test_rows_wider_than_one_warp_pass(H, k):
    # rows above 16 KB are moved in several pieces per warp by the scatter and in many column
    # chunks by the combine; widths that are not a multiple of a chunk leave a ragged last chunk
    wl = W.Workload("widerows", T=150, H=H, E=32, k=k, R=8, S=4, score_func=W.SOFTMAX, seed=43, max_replicas=1)
    run_and_check(wl, W.make_inputs(wl), (5,))


@pytest.mark.parametrize("R", [83, 84, 85, 86, 87, 88])
def test_routing_tables_around_the_default_shared_memory_limit(R):
    # slot counts that put the routing kernel's shared-memory tables just below, at and just
    # above the 48 KB a kernel gets without opting in to more
    E, S, copies = 192, 7, 3
    wl = W.Workload("smem-edge", T=244, H=584, E=E, k=3, R=R, S=S, score_func=W.SOFTMAX, seed=47,
                    max_replicas=copies)
    inp = W.make_inputs(dataclasses.replace(wl, max_replicas=1, R=24, S=8))   # logits / x only
    s2e = np.full(R * S, -1, np.int32)
    s2e[: E * copies] = np.repeat(np.arange(E), copies)      # three copies of every expert, the rest empty
    inp["slot_to_expert"] = s2e
    inp["slot_scale"] = np.random.default_rng(4).uniform(0.5, 1.5, R * S).astype(np.float32)
    run_and_check(wl, inp, (1, 40))


def test_tuning_call_validates_and_restores():
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=300, H=128)
    router = B.MoeRouter(B.config_for_workload(wl, max_tokens=300, hidden=128), inp["slot_to_expert"],
                         inp["bias"], inp["slot_scale"])
    ctx = router._ctx
    assert B.moe_set_tuning(ctx, -1, 0) == B.MOE_ERR_INVALID_ARG
    assert B.moe_set_tuning(ctx, 99, 0) == B.MOE_ERR_INVALID_ARG
    assert B.moe_set_tuning(ctx, B.MOE_TUNE_PDL, -2) == B.MOE_ERR_INVALID_ARG
    assert B.moe_set_tuning(None, B.MOE_TUNE_PDL, 0) == B.MOE_ERR_INVALID_ARG
    # a tile the shape cannot have (not enough shared memory for it) is refused and nothing changes
    assert B.moe_set_tuning(ctx, B.MOE_TUNE_ROUTE_TOKENS_PER_TILE, 10 ** 6) in (B.MOE_OK, B.MOE_ERR_INVALID_ARG)
    run_and_check(wl, inp, (), router=router)
    # overrides, then back to the automatic choices: results never change
    for option, value in ((B.MOE_TUNE_ROUTE_TOKENS_PER_TILE, 16), (B.MOE_TUNE_COMBINE_IMPL, 0),
                          (B.MOE_TUNE_SCATTER_IMPL, 1), (B.MOE_TUNE_ROUTE_PREFETCH, 0),
                          (B.MOE_TUNE_SCATTER_STORE_POLICY, 3)):
        assert B.moe_set_tuning(ctx, option, value) == B.MOE_OK
        run_and_check(wl, inp, (), router=router)
    for option in range(16):
        assert B.moe_set_tuning(ctx, option, -1) == B.MOE_OK
    run_and_check(wl, inp, (), router=router)
    router.close()
