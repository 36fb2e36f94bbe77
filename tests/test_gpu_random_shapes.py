"""Seeded sweep over random shapes: experts, k, groups, ranks, slots, replicas,
failed ranks, lost experts, rank order, tokens and width are all drawn at random
(from a fixed seed); every configuration the library accepts must match the
oracle in every output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import assert_y_close, bf16_bits, check_dispatch, to_dev

pytestmark = pytest.mark.gpu


def _draw(rng):
    k = int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16]))
    n_group, topk_group = 1, 1
    if rng.random() < 0.4 and k % 2 == 0:
        topk_group = k // int(rng.choice([1, 2])) if k > 1 else 1
        n_group = int(rng.choice([g for g in (2, 4, 8, 16) if g >= topk_group] or [topk_group]))
    per_group = int(rng.choice([1, 2, 3, 4, 8, 16, 32]))
    E = n_group * per_group if n_group > 1 else int(rng.integers(max(k, 2), 400))
    E = min(E, 512)
    copies = int(rng.choice([1, 1, 2, 3]))
    S = int(rng.integers(1, 9))
    R = max(2, -(-E * copies // S) + int(rng.integers(0, 3)))
    if R * S > 4096:
        return None
    s2e = np.full(R * S, -1, np.int32)
    slots = rng.permutation(R * S)[: E * copies] if rng.random() < 0.5 else np.arange(E * copies)
    s2e[slots] = np.repeat(np.arange(E), copies)
    return dict(E=E, k=k, n_group=n_group, topk_group=topk_group, R=R, S=S, max_rep=copies, s2e=s2e,
                score=int(rng.integers(0, 2)), T=int(rng.integers(1, 400)), H=8 * int(rng.integers(1, 80)),
                scale=float(rng.choice([1.0, 2.5])))


@pytest.mark.parametrize("seed", [20261128, 3, 11])
def test_random_configurations_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    accepted = 0
    for trial in range(400):
        c = _draw(rng)
        if c is None:
            continue
        cfg = B.make_config(c["E"], c["k"], c["H"], max(c["T"], 1), c["R"], c["S"], c["max_rep"], c["score"],
                            c["n_group"], c["topk_group"], c["scale"])
        if B.moe_workspace_bytes(cfg) == 0:
            continue
        ocfg = oracle.OracleConfig(c["E"], c["k"], c["R"], c["S"], c["score"], c["n_group"], c["topk_group"], c["scale"])
        failed = tuple(int(r) for r in rng.choice(c["R"], int(rng.integers(0, max(1, c["R"] // 3))), replace=False))
        lost = (rng.random(c["E"]) < rng.choice([0.0, 0.1])).astype(np.uint8)
        if not oracle.failure_set_ok(ocfg, c["s2e"], failed, lost):
            st, *_ = B.moe_plan_routing_state(cfg, c["s2e"], failed)
            if not lost.any():
                assert st == B.MOE_ERR_INSUFFICIENT_EXPERTS
            continue
        logits = rng.standard_normal((c["T"], c["E"])).astype(np.float32)
        if rng.random() < 0.3:
            logits = np.round(logits * 4) / 4                         # ties
        x = W.f32_to_bf16_bits(rng.standard_normal((c["T"], c["H"])).astype(np.float32))
        bias = (0.05 * rng.standard_normal(c["E"])).astype(np.float32) if c["score"] else None
        sscale = rng.uniform(0.5, 1.5, c["R"] * c["S"]).astype(np.float32)
        alive = [r for r in range(c["R"]) if r not in failed]
        order = [int(r) for r in rng.permutation(alive)] if rng.random() < 0.5 else None

        router = B.MoeRouter(cfg, c["s2e"], bias, sscale)
        router.set_failed_ranks(failed)
        router.set_failed_experts(lost)
        if order is not None:
            router.set_rank_order(order)
        out = router.dispatch(to_dev(logits), to_dev(x, torch.bfloat16))
        y = router.combine(out.send_buf, c["T"])
        torch.cuda.synchronize()
        assert router.device_status() == 0, c
        ref = oracle.dispatch(ocfg, c["s2e"], failed, bias, logits, x, lost, order)
        try:
            check_dispatch(out, ref)
            ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"], sscale)
            assert_y_close(bf16_bits(y), ref_y)
        except AssertionError as e:
            raise AssertionError(f"trial {trial}: { {k: v for k, v in c.items() if k != 's2e'} } failed={failed}: {e}")
        router.close()
        accepted += 1
    assert accepted >= 150, accepted
