"""Expert-level failures (the paper's lost-expert experiment, Sec. 4.2): experts
are failed one by one under two policies, "every nth" and "most activated",
and routing must use the next-best experts.  CPU part: pins of the oracle and
of the two generators.  GPU part: parity of moe_set_failed_experts."""
import numpy as np
import pytest

import oracle
from paper_2602_21140_b200 import workloads as W
from util import oracle_cfg

RATES = [1 / 64, 1 / 32, 1 / 16, 1 / 8, 1 / 4, 1 / 2]


def test_every_nth_generator():
    for r in RATES:
        m = W.every_nth_mask(256, r)
        assert m.sum() == round(256 * r)
    assert W.every_nth_mask(8, 0.5).tolist() == [1, 0, 1, 0, 1, 0, 1, 0]   # every even-indexed expert


def test_most_activated_generator():
    counts = np.array([5, 9, 9, 1, 0, 7, 3, 2])
    assert W.most_activated_mask(counts, 0.25).tolist() == [0, 1, 1, 0, 0, 0, 0, 0]
    assert W.most_activated_mask(counts, 0.5).tolist() == [1, 1, 1, 0, 0, 1, 0, 0]
    assert W.most_activated_mask(counts, 1 / 64).sum() == 0


@pytest.mark.parametrize("name", ["qwen3", "dsv3", "kimi"])
def test_oracle_expert_mask_equals_minus_inf_columns(name):
    # Sec. 4.2: a failed expert's routing logit is masked to -inf right before top-k
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=256, with_x=False)
    cfg = oracle_cfg(wl)
    for r in (1 / 32, 1 / 2):
        mask = W.every_nth_mask(wl.E, r)
        ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], (), inp["bias"], inp["logits"], mask)
        lg = inp["logits"].copy()
        lg[:, mask != 0] = -np.inf
        ids2, w2, slot2 = oracle.route(cfg, inp["slot_to_expert"], (), inp["bias"], lg)
        assert np.array_equal(ids, ids2) and np.array_equal(w, w2) and np.array_equal(slot, slot2)
        assert not mask[ids].any()
        # the survivors are the next best: ids equal the unmasked top-k wherever that avoided the mask
        ids0, _, _ = oracle.route(cfg, inp["slot_to_expert"], (), inp["bias"], inp["logits"])
        untouched = ~mask[ids0].any(axis=1)
        if wl.n_group == 1:
            assert np.array_equal(ids[untouched], ids0[untouched])


def test_oracle_expert_mask_combines_with_failed_ranks_and_replicas():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    cfg = oracle_cfg(wl)
    mask = np.zeros(wl.E, np.uint8); mask[0] = 1            # expert 0 lost although it has two replicas
    ids, _, slot = oracle.route(cfg, inp["slot_to_expert"], (2,), None, inp["logits"], mask)
    assert not np.isin(ids, [0, 4, 5]).any()
    assert not np.isin(slot, [0, 8, 4, 5]).any()
    assert oracle.failure_set_ok(cfg, inp["slot_to_expert"], (2,), mask)
    everything = np.ones(wl.E, np.uint8); everything[3] = 0
    assert not oracle.failure_set_ok(cfg, inp["slot_to_expert"], (), everything)


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["dsv3", "kimi", "qwen3"])
def test_gpu_parity_under_both_policies(name):
    import torch
    from paper_2602_21140_b200 import binding as B
    from gpu_util import assert_y_close, bf16_bits, check_dispatch, make_router, to_dev
    wl = W.WORKLOADS[name]
    T, H = 1037, 256
    inp = W.make_inputs(wl, T=T, H=H)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = make_router(wl, inp, max_tokens=T, hidden=H)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    out = router.dispatch(logits, x)
    torch.cuda.synchronize()
    counts = np.bincount(out.topk_ids.cpu().numpy().ravel(), minlength=wl.E)   # our own activation counts
    failed_ranks = wl.failure_sets[1] if len(wl.failure_sets) > 1 else ()
    router.set_failed_ranks(failed_ranks)
    for r in (1 / 64, 1 / 8, 1 / 2):
        for mask in (W.every_nth_mask(wl.E, r), W.most_activated_mask(counts, r)):
            if not oracle.failure_set_ok(oracle_cfg(wl), inp["slot_to_expert"], failed_ranks, mask):
                with pytest.raises(B.MoeError) as e:
                    router.set_failed_experts(mask)
                assert e.value.status == B.MOE_ERR_INSUFFICIENT_EXPERTS
                continue
            router.set_failed_experts(mask)
            out = router.dispatch(logits, x, out)
            y = router.combine(out.send_buf, T)
            torch.cuda.synchronize()
            ref = oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], failed_ranks, bias, inp["logits"],
                                  inp["x"], mask)
            check_dispatch(out, ref)
            assert not mask[out.topk_ids.cpu().numpy()].any()
            ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                                   inp["slot_scale"])
            assert_y_close(bf16_bits(y), ref_y)
    router.set_failed_experts(None)               # clearing restores rank-only routing
    out = router.dispatch(logits, x, out)
    torch.cuda.synchronize()
    check_dispatch(out, oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], failed_ranks, bias,
                                        inp["logits"], inp["x"]))
    assert router.device_status() == 0
    router.close()
