"""Dense-FFN TP-group rebalancing (Sec. 3.4): the first layers of some models are
dense FFNs run tensor-parallel (TP = 4) and replicated over several FFN groups;
a group that lost any shard is compromised and attention spreads its tokens
evenly over the healthy groups.  Here that is a routing mode of the same
dispatch/combine path (score_func 2)."""
import numpy as np
import pytest

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import build as build_mod
from paper_2602_21140_b200 import workloads as W
from util import bf16_to_f64, oracle_cfg

DENSE = 2
TP, GROUPS = 4, 8
WL = W.Workload("dense-ffn", T=1037, H=256, E=GROUPS * TP, k=TP, R=16, S=2, score_func=DENSE,
                seed=31, failure_sets=((), (5,), (5, 9), (0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13)),
                max_replicas=1)


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build_library()


def _compromised(failed):
    return sorted({(r * WL.S + s) // TP for r in failed for s in range(WL.S)})


def test_oracle_spreads_tokens_evenly_over_healthy_groups():
    inp = W.make_inputs(WL, with_x=False)
    cfg = oracle_cfg(WL)
    for failed in WL.failure_sets:
        ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], failed, None, inp["logits"])
        groups = ids[:, 0] // TP
        assert np.array_equal(ids, groups[:, None] * TP + np.arange(TP)[None, :]), "all shards of one group"
        bad = _compromised(failed)
        assert not np.isin(groups, bad).any(), "compromised groups get nothing"
        healthy = [g for g in range(GROUPS) if g not in bad]
        loads = np.bincount(groups, minlength=GROUPS)[healthy]
        assert loads.max() - loads.min() <= 1, "even rebalance"
        assert np.array_equal(groups, np.array(healthy)[np.arange(WL.T) % len(healthy)])
        assert np.all(w == 1.0) and np.array_equal(slot, ids)
        assert not np.isin(slot // WL.S, list(failed)).any()


def test_oracle_partials_add_up_in_combine():
    inp = W.make_inputs(WL, T=64, H=32)
    cfg = oracle_cfg(WL)
    out = oracle.dispatch(cfg, inp["slot_to_expert"], (5,), None, inp["logits"], inp["x"])
    scale = np.full(WL.P, 1.0 / TP, np.float32)          # each shard contributes a quarter
    y = oracle.combine(out["send_buf"], out["dst_row"], out["topk_weights"], out["topk_slot"], scale)
    assert np.array_equal(y, inp["x"])                   # 4 * (x / 4) is exact in bf16
    y2 = oracle.combine(out["send_buf"], out["dst_row"], out["topk_weights"], out["topk_slot"],
                        np.ones(WL.P, np.float32))
    assert np.array_equal(bf16_to_f64(y2), TP * bf16_to_f64(inp["x"]))


def test_admission_needs_one_healthy_group():
    cfg = B.config_for_workload(WL)
    cfg_o = oracle_cfg(WL)
    s2e = W.slot_to_expert(WL)
    assert B.moe_plan_routing_state(cfg, s2e, (5, 9))[0] == B.MOE_OK
    assert B.moe_plan_routing_state(cfg, s2e, WL.failure_sets[3])[3] == 1      # one healthy group left
    every_group_hit = [0, 2, 4, 6, 8, 10, 12, 14]
    assert B.moe_plan_routing_state(cfg, s2e, every_group_hit)[0] == B.MOE_ERR_INSUFFICIENT_EXPERTS
    assert not oracle.failure_set_ok(cfg_o, s2e, every_group_hit)
    assert oracle.failure_set_ok(cfg_o, s2e, WL.failure_sets[3])
    bad = B.config_for_workload(WL); bad.num_experts = 30                       # not a multiple of TP
    assert B.moe_workspace_bytes(bad) == 0


@pytest.mark.gpu
def test_gpu_dense_mode_matches_oracle():
    import torch
    from gpu_util import assert_y_close, bf16_bits, check_dispatch, to_dev
    inp = W.make_inputs(WL)
    router = B.MoeRouter(B.config_for_workload(WL), inp["slot_to_expert"], None, inp["slot_scale"])
    x = to_dev(inp["x"], torch.bfloat16)
    logits = to_dev(inp["logits"])
    out = router.alloc_outputs(WL.T)
    y = torch.empty_like(x)
    for failed in WL.failure_sets:
        router.set_failed_ranks(failed)
        st = B.moe_dispatch(router._ctx, 0, x.data_ptr(), WL.T, out.as_struct(),      # logits not needed
                            torch.cuda.current_stream().cuda_stream)
        assert st == B.MOE_OK
        router.combine(out.send_buf, WL.T, y)
        torch.cuda.synchronize()
        ref = oracle.dispatch(oracle_cfg(WL), inp["slot_to_expert"], failed, None, inp["logits"], inp["x"])
        check_dispatch(out, ref)
        ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                               inp["slot_scale"])
        assert_y_close(bf16_bits(y), ref_y)
    with pytest.raises(B.MoeError) as e:
        router.set_failed_ranks([0, 2, 4, 6, 8, 10, 12, 14])
    assert e.value.status == B.MOE_ERR_INSUFFICIENT_EXPERTS
    out2 = router.dispatch(logits, x)                     # passing logits is allowed, they are ignored
    torch.cuda.synchronize()
    check_dispatch(out2, oracle.dispatch(oracle_cfg(WL), inp["slot_to_expert"], WL.failure_sets[-1], None,
                                         inp["logits"], inp["x"]))
    assert router.device_status() == 0
    router.close()
