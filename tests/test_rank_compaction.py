"""Logical-rank compaction (Sec. 3.5) and the send-buffer layout in logical-rank
order.  CPU: the paper's worked relation for both the oracle and the library's
host helper, and the oracle's ordered permutation against numpy.  GPU: parity of
moe_set_rank_order."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import build as build_mod
from paper_2602_21140_b200 import workloads as W
from util import oracle_cfg


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build_library()


def _by_the_text(R, failed, switched=-1, replaced=-1):
    """Sec. 3.5 step by step on a dict rank -> logical rank."""
    logical = {r: r for r in range(R)}
    gaps = []
    if switched >= 0:
        gaps.append(logical[switched])          # the switched device leaves its place ...
        logical[switched] = logical[replaced]   # ... and takes the failed device's logical rank
        del logical[replaced]
    for a in sorted(failed):
        if a in logical:
            gaps.append(logical.pop(a))
    for g in sorted(gaps, reverse=True):        # close every gap: later ranks move down by one
        for r in logical:
            if logical[r] > g:
                logical[r] -= 1
    return [r for r, _ in sorted(logical.items(), key=lambda kv: kv[1])]


def test_worked_relation_single_failure():
    # device A with logical rank 2 fails: B = 3 takes 2, later ranks decrement
    assert oracle.compact_ranks(6, [2]) == [0, 1, 3, 4, 5]
    st, order = B.moe_compact_ranks(6, [2])
    assert st == B.MOE_OK and order == [0, 1, 3, 4, 5]


def test_worked_relation_role_switch():
    # switched device C = 5 takes the logical rank of failed A = 2; nothing else moves
    assert oracle.compact_ranks(6, [2], 5, 2) == [0, 1, 5, 3, 4]
    st, order = B.moe_compact_ranks(6, [2], 5, 2)
    assert st == B.MOE_OK and order == [0, 1, 5, 3, 4]
    # C = 0 in front of A = 3: C's old place closes first, then C sits where A was
    assert oracle.compact_ranks(6, [3], 0, 3) == [1, 2, 0, 4, 5]


def test_compaction_exhaustive_small():
    R = 6
    for n in range(0, 4):
        for failed in itertools.combinations(range(R), n):
            want = _by_the_text(R, failed)
            assert oracle.compact_ranks(R, failed) == want
            assert B.moe_compact_ranks(R, failed) == (B.MOE_OK, want)
            for a in failed:
                for c in range(R):
                    if c in failed:
                        continue
                    want = _by_the_text(R, failed, c, a)
                    assert oracle.compact_ranks(R, failed, c, a) == want, (failed, c, a)
                    assert B.moe_compact_ranks(R, failed, c, a) == (B.MOE_OK, want)


def test_compaction_rejects_bad_arguments():
    assert B.moe_compact_ranks(4, [4])[0] == B.MOE_ERR_INVALID_ARG
    assert B.moe_compact_ranks(4, [1], 1, 1)[0] == B.MOE_ERR_INVALID_ARG     # switched rank is itself failed
    assert B.moe_compact_ranks(4, [1], 2, 3)[0] == B.MOE_ERR_INVALID_ARG     # replaced rank is not failed
    assert B.moe_compact_ranks(4, [1], 2, -1)[0] == B.MOE_ERR_INVALID_ARG


@pytest.mark.parametrize("name", ["tiny", "dsv3"])
def test_oracle_ordered_permutation_matches_numpy(name):
    wl = W.WORKLOADS[name]
    T = min(wl.T, 512)
    inp = W.make_inputs(wl, T=T, with_x=False)
    cfg = oracle_cfg(wl)
    failed = wl.failure_sets[-1]
    order = oracle.compact_ranks(wl.R, failed)
    if len(order) > 2:
        order[0], order[-1] = order[-1], order[0]           # any order of the alive ranks is allowed
    _, _, slot = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"])
    out = oracle.permutation(cfg, slot, order)
    full = order + [r for r in range(wl.R) if r not in order]
    pos_of_rank = np.empty(wl.R, np.int64); pos_of_rank[full] = np.arange(wl.R)
    flat = slot.ravel().astype(np.int64)
    key = pos_of_rank[flat // wl.S] * wl.S + flat % wl.S      # position of the slot in the layout
    src = np.argsort(key, kind="stable")
    assert np.array_equal(out["src_index"], src)
    counts = np.bincount(flat, minlength=wl.P)
    assert np.array_equal(out["slot_counts"], counts)
    by_pos = counts.reshape(wl.R, wl.S)[full]
    assert np.array_equal(out["rank_counts"], by_pos.sum(1))
    assert np.array_equal(out["rank_offsets"], np.concatenate([[0], np.cumsum(by_pos.sum(1))]))
    start = np.concatenate([[0], np.cumsum(by_pos.ravel())])[:-1].reshape(wl.R, wl.S)
    want_off = np.empty(wl.P, np.int64); want_off.reshape(wl.R, wl.S)[full] = start
    assert np.array_equal(out["slot_offsets"][:-1], want_off)
    # the rows of the alive ranks are contiguous and in logical order: no holes
    assert out["rank_counts"][len(order):].sum() == 0


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["tiny", "dsv3", "kimi"])
def test_gpu_layout_follows_rank_order(name):
    import torch
    from gpu_util import assert_y_close, bf16_bits, check_dispatch, make_router, to_dev
    wl = W.WORKLOADS[name]
    T, H = min(wl.T, 1037), min(wl.H, 256)
    inp = W.make_inputs(wl, T=T, H=H)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = make_router(wl, inp, max_tokens=T, hidden=H)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    failed = wl.failure_sets[-1]
    router.set_failed_ranks(failed)
    alive = [r for r in range(wl.R) if r not in failed]
    orders = [B.moe_compact_ranks(wl.R, failed)[1], list(reversed(alive))]
    if failed:
        orders.append(B.moe_compact_ranks(wl.R, failed, alive[-1], failed[0])[1])      # role switch
    for order in orders:
        router.set_rank_order(order)
        out = router.dispatch(logits, x)
        y = router.combine(out.send_buf, T)
        torch.cuda.synchronize()
        ref = oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], failed, bias, inp["logits"], inp["x"],
                              rank_order=order)
        check_dispatch(out, ref)
        ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                               inp["slot_scale"])
        assert_y_close(bf16_bits(y), ref_y)
    # an order that leaves out an alive rank is refused and changes nothing
    with pytest.raises(B.MoeError) as e:
        router.set_rank_order(alive[:-1])
    assert e.value.status == B.MOE_ERR_INVALID_ARG
    with pytest.raises(B.MoeError):
        router.set_rank_order([alive[0], alive[0]])
    if failed:
        with pytest.raises(B.MoeError):            # reviving a rank that the order does not list
            router.set_failed_ranks(())
    out = router.dispatch(logits, x)
    torch.cuda.synchronize()
    check_dispatch(out, oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], failed, bias, inp["logits"],
                                        inp["x"], rank_order=orders[-1]))
    router.set_rank_order([])                      # back to the physical numbering
    out = router.dispatch(logits, x)
    torch.cuda.synchronize()
    check_dispatch(out, oracle.dispatch(oracle_cfg(wl), inp["slot_to_expert"], failed, bias, inp["logits"], inp["x"]))
    assert router.device_status() == 0
    router.close()
