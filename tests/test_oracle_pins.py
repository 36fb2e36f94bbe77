"""Pins for the CPU oracle: each test checks the oracle against something that
is not the oracle (brute force, a library routine, a closed form, libm, a
hand-worked example), so that a slip anywhere in it fails here before any
CUDA result is compared with it."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import workloads as W
from util import bf16_to_f64, oracle_cfg, small_grouped_workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# exp / sigmoid built from fp32 ops: error bound against libm, monotonicity
# --------------------------------------------------------------------------

def test_exp_spec_within_2ulp_of_libm():
    z = np.concatenate([np.linspace(-87, 88, 3_000_001), np.linspace(-1, 1, 1_000_001),
                        np.array([0.0, -0.0, 1e-30, -1e-30])]).astype(np.float32)
    got = oracle.exp_spec(z).astype(np.float64)
    ref = np.exp(z.astype(np.float64))
    ulp = np.spacing(ref.astype(np.float32)).astype(np.float64)
    assert np.max(np.abs(got - ref) / ulp) <= 2.0
    assert oracle.exp_spec(np.float32(0.0)) == np.float32(1.0)


def test_exp_spec_clamps():
    e = oracle.exp_spec(np.array([-1000.0, -np.inf, 1000.0, np.inf], np.float32)).astype(np.float64)
    assert np.allclose(e[:2], math.exp(-87), rtol=1e-6)
    assert np.allclose(e[2:], math.exp(88), rtol=1e-6)


def test_sigmoid_spec_accuracy_symmetry_monotone():
    x = np.linspace(-40, 40, 4_000_001).astype(np.float32)
    s = oracle.sigmoid_spec(x)
    ref = 1.0 / (1.0 + np.exp(-x.astype(np.float64)))
    assert np.max(np.abs(s - ref) / ref) < 3e-7
    assert np.all(np.diff(s) >= 0), "selection order must follow the logits"
    assert oracle.sigmoid_spec(np.float32(0.0)) == np.float32(0.5)
    assert np.all((s > 0) & (s <= 1))


# --------------------------------------------------------------------------
# bf16 rounding of the combine result: one rounding, ties to even
# --------------------------------------------------------------------------

def test_double_to_bf16_matches_torch_on_fp32_values():
    rng = np.random.default_rng(0)
    f = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-30, 30, 20000),
                        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, 1e-40, -1e-40, 9.2e-41, 4.6e-41],
                                 np.float32)]).astype(np.float32)
    want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.double_to_bf16(f.astype(np.float64))
    assert np.array_equal(got, want)


def test_double_to_bf16_ties_and_single_rounding():
    one = 0x3F80
    cases = {
        1.0 + 2.0 ** -8: one,                       # tie -> even (down)
        1.0 + 3 * 2.0 ** -8: one + 2,               # tie -> even (up)
        1.0 + 2.0 ** -8 + 2.0 ** -40: one + 1,      # above the tie; via fp32 it would round twice to 1.0
        1.0 + 2.0 ** -8 - 2.0 ** -40: one,
        -(1.0 + 2.0 ** -8 + 2.0 ** -40): 0x8000 | (one + 1),
        2.0 ** -133: 0x0001,                         # smallest subnormal
        2.0 ** -134: 0x0000,                         # tie with zero -> even
        2.0 ** -134 * 1.5: 0x0001,
        1e39: 0x7F80,
    }
    for d, bits in cases.items():
        assert int(oracle.double_to_bf16(np.float64(d)).item()) == bits, d


# --------------------------------------------------------------------------
# hand-worked example (tests/golden/hand_worked_routing.json)
# --------------------------------------------------------------------------

def _load_hand_worked():
    with open(os.path.join(GOLDEN, "hand_worked_routing.json")) as f:
        g = json.load(f)
    cfg = oracle.OracleConfig(**g["config"])
    logits = np.log(np.array(g["logits_exp"], np.float64)).astype(np.float32)
    x = W.f32_to_bf16_bits(np.array(g["x"], np.float32))
    return g, cfg, logits, x


def test_hand_worked_example():
    g, cfg, logits, x = _load_hand_worked()
    e = g["expect"]
    out = oracle.dispatch(cfg, g["slot_to_expert"], g["failed_ranks"], None, logits, x)
    assert out["topk_ids"].tolist() == e["topk_ids"]
    assert out["topk_slot"].tolist() == e["topk_slot"]
    np.testing.assert_allclose(out["topk_weights"], np.array(e["topk_weights"]), rtol=1e-6)
    for name in ("slot_counts", "slot_offsets", "rank_counts", "rank_offsets", "dst_row", "src_index"):
        assert out[name].tolist() == e[name], name
    assert W.bf16_bits_to_f32(out["send_buf"]).tolist() == e["send_buf"]
    y = oracle.combine(out["send_buf"], out["dst_row"], out["topk_weights"], out["topk_slot"],
                       np.array(g["slot_scale"], np.float32))
    assert W.bf16_bits_to_f32(y).tolist() == e["y"]
    ids0, w0, _ = oracle.route(cfg, g["slot_to_expert"], [], None, logits)
    assert ids0.tolist() == e["topk_ids_no_failure"]
    np.testing.assert_allclose(w0, np.array(e["topk_weights_no_failure"]), rtol=1e-6)


# --------------------------------------------------------------------------
# P1: top-k against brute-force enumeration of subsets
# --------------------------------------------------------------------------

def _avail(wl, s2e, failed):
    avail = np.zeros(wl.E, bool)
    for p, e in enumerate(s2e):
        if e >= 0 and (p // wl.S) not in failed:
            avail[e] = True
    return avail


def _dominates(keys, i, j):
    """(key_i, -i) > (key_j, -j)"""
    return keys[i] > keys[j] or (keys[i] == keys[j] and i < j)


def _brute_topk(keys, allowed, k):
    cand = [e for e in range(len(keys)) if allowed[e]]
    hits = []
    for S in itertools.combinations(cand, k):
        rest = [e for e in cand if e not in S]
        if all(_dominates(keys, i, j) for i in S for j in rest):
            hits.append(S)
    assert len(hits) == 1
    S = list(hits[0])
    S.sort(key=lambda e: (-keys[e], e))
    return S


def test_topk_tiny_bruteforce_all_subsets():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    failed = wl.failure_sets[0]
    ids, _, _ = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], failed, None, inp["logits"])
    avail = _avail(wl, inp["slot_to_expert"], failed)
    assert avail.tolist() == [True, True, True, True, False, False, True, True]
    for t in range(wl.T):
        assert ids[t].tolist() == _brute_topk(inp["logits"][t], avail, wl.k)


def _brute_grouped(keys, allowed, k, n_group, topk_group):
    """Group-limited selection by enumeration of group subsets; keys fp32."""
    E = len(keys)
    per = E // n_group
    m = k // topk_group
    gs = []
    for g in range(n_group):
        fin = sorted((np.float32(keys[e]) for e in range(g * per, (g + 1) * per)
                      if allowed[e] and keys[e] != -np.inf), reverse=True)[:m]
        if not fin:
            gs.append(-np.inf)
        else:
            s = fin[0]
            for v in fin[1:]:
                s = np.float32(s + v)
            gs.append(float(s))
    hits = []
    for G in itertools.combinations(range(n_group), topk_group):
        rest = [g for g in range(n_group) if g not in G]
        if all(_dominates(gs, a, b) for a in G for b in rest):
            hits.append(G)
    assert len(hits) == 1
    allowed2 = [allowed[e] and (e // per) in hits[0] and keys[e] != -np.inf for e in range(E)]
    return _brute_topk(keys, allowed2, k)


@pytest.mark.parametrize("E,k,n_group,topk_group", [(8, 2, 4, 2), (16, 4, 4, 2), (24, 6, 6, 3)])
def test_grouped_selection_bruteforce_softmax_keys(E, k, n_group, topk_group):
    # softmax mode: the keys are the raw logits, so brute force needs no exp at all
    wl = small_grouped_workload(E=E, k=k, n_group=n_group, topk_group=topk_group, R=E // 4, S=4,
                                score_func=W.SOFTMAX)
    inp = W.make_inputs(wl)
    for failed in [(), (1,)]:
        avail = _avail(wl, inp["slot_to_expert"], failed)
        ids, _, _ = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], failed, None, inp["logits"])
        for t in range(wl.T):
            assert ids[t].tolist() == _brute_grouped(inp["logits"][t], avail, k, n_group, topk_group)


def test_grouped_selection_bruteforce_sigmoid_keys_with_margin():
    # sigmoid keys recomputed in float64; tokens whose decision margins are below 1e-5 are skipped
    wl = small_grouped_workload()
    inp = W.make_inputs(wl)
    keys64 = 1.0 / (1.0 + np.exp(-inp["logits"].astype(np.float64))) + inp["bias"].astype(np.float64)
    ids, _, _ = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (), inp["bias"], inp["logits"])
    checked = 0
    for t in range(wl.T):
        kk = keys64[t]
        per = wl.E // wl.n_group
        gs = np.array([np.sort(kk[g * per:(g + 1) * per])[-2:].sum() for g in range(wl.n_group)])
        gsort = np.sort(gs)
        if np.min(np.diff(gsort)) < 1e-5 or np.min(np.diff(np.sort(kk))) < 1e-5:
            continue
        checked += 1
        assert ids[t].tolist() == _brute_grouped(kk.astype(np.float32), np.ones(wl.E, bool),
                                                 wl.k, wl.n_group, wl.topk_group)
    assert checked > wl.T // 2


def test_group_with_fewer_than_m_finite_keys():
    # 3 groups of 4, keep 2, k = 4 so m = 2.  Group 0 keeps a single available expert with a
    # large key: its score is that key alone (9), not 9 + (-inf), so it is kept with group 1
    # (3 + 2.5 = 5.5) ahead of group 2 (2 + 2 = 4).
    cfg = oracle.OracleConfig(num_experts=12, top_k=4, num_ranks=12, slots_per_rank=1,
                              n_group=3, topk_group=2)
    logits = np.array([[9.0, 8.0, 7.0, 6.0, 3.0, 2.5, 1.0, 0.0, 2.0, 2.0, 1.5, 0.1]], np.float32)
    ids, w, _ = oracle.route(cfg, np.arange(12), (1, 2, 3), None, logits)
    assert ids[0].tolist() == [0, 4, 5, 6]
    u = np.exp(np.array([0.0, -6.0, -6.5, -8.0]))
    np.testing.assert_allclose(w[0], u / u.sum(), rtol=1e-6)
    # a group with no finite key scores -inf and loses to any group with one
    ids, _, _ = oracle.route(cfg, np.arange(12), (0, 1, 2, 3), None, logits)
    assert ids[0].tolist() == [4, 5, 8, 9]


# --------------------------------------------------------------------------
# P2: counts / offsets / permutation reduce to numpy routines
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "dsv3", "kimi"])
def test_permutation_matches_numpy(name):
    wl = W.WORKLOADS[name]
    T = min(wl.T, 1024)
    inp = W.make_inputs(wl, T=T, with_x=False)
    cfg = oracle_cfg(wl)
    for failed in wl.failure_sets[:3]:
        _, _, slot = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"])
        out = oracle.permutation(cfg, slot)
        flat = slot.ravel()
        counts = np.bincount(flat, minlength=wl.P)
        assert np.array_equal(out["slot_counts"], counts)
        assert np.array_equal(out["slot_offsets"], np.concatenate([[0], np.cumsum(counts)]))
        src = np.argsort(flat, kind="stable")
        assert np.array_equal(out["src_index"], src)
        inv = np.empty_like(src)
        inv[src] = np.arange(src.size)
        assert np.array_equal(out["dst_row"], inv)
        assert np.array_equal(out["rank_counts"], counts.reshape(wl.R, wl.S).sum(1))
        assert np.array_equal(out["rank_offsets"][:-1], out["slot_offsets"][:-1:wl.S])
        assert out["rank_offsets"][-1] == T * wl.k
        for r in failed:
            assert out["rank_counts"][r] == 0


# --------------------------------------------------------------------------
# P3 / P4: no failures, no redundancy, softmax -> textbook softmax + topk + renorm
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["mixtral", "qwen3"])
def test_softmax_special_case_matches_torch(name):
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=512, with_x=False)
    ids, w, slot = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (), None, inp["logits"])
    lg = torch.from_numpy(inp["logits"]).double()
    probs = torch.softmax(lg, dim=-1)
    tv, ti = torch.topk(probs, wl.k, dim=-1)
    assert np.array_equal(ids, ti.numpy())
    ref_w = (tv / tv.sum(-1, keepdim=True)).numpy()
    np.testing.assert_allclose(w, ref_w, rtol=1e-6)
    # softmax over the k chosen logits is the same thing
    ref2 = torch.softmax(torch.gather(lg, 1, ti), dim=-1).numpy()
    np.testing.assert_allclose(w, ref2, rtol=1e-6)
    assert np.array_equal(slot, ids), "one slot per expert, slot id == expert id"


def test_sigmoid_weights_ignore_bias_and_renormalise():
    wl = W.WORKLOADS["kimi"]
    inp = W.make_inputs(wl, T=256, with_x=False)
    ids, w, _ = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (), inp["bias"], inp["logits"])
    s = 1.0 / (1.0 + np.exp(-inp["logits"].astype(np.float64)))
    keys = s + inp["bias"].astype(np.float64)
    chosen = np.take_along_axis(s, ids.astype(np.int64), axis=1)
    np.testing.assert_allclose(w, chosen / chosen.sum(1, keepdims=True), rtol=1e-6)
    # selection follows key = score + bias: the chosen set is the top-k of the float64 keys
    # wherever the k-th / (k+1)-th keys are clearly apart
    srt = np.sort(keys, axis=1)
    clear = (srt[:, -wl.k] - srt[:, -wl.k - 1]) > 1e-5
    top = np.argsort(-keys, axis=1, kind="stable")[:, :wl.k]
    assert clear.sum() > 200
    assert np.array_equal(np.sort(ids[clear], 1), np.sort(top[clear], 1))


def test_route_scale_multiplies_weights():
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=64, with_x=False)
    _, w1, _ = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (), inp["bias"], inp["logits"])
    _, w2, _ = oracle.route(oracle_cfg(wl, 2.5), inp["slot_to_expert"], (), inp["bias"], inp["logits"])
    np.testing.assert_allclose(w2, 2.5 * w1.astype(np.float64), rtol=1e-6)
    np.testing.assert_allclose(w2.astype(np.float64).sum(1), 2.5, rtol=1e-6)


# --------------------------------------------------------------------------
# ties (lower id wins), signed zeros
# --------------------------------------------------------------------------

def test_ties_break_to_lower_expert_id():
    cfg = oracle.OracleConfig(num_experts=8, top_k=3, num_ranks=8, slots_per_rank=1)
    logits = np.array([[1, 1, 1, 1, 1, 1, 1, 1],
                       [0, 2, 2, 0, 2, 2, 0, 0],
                       [-0.0, 0.0, -1, -1, -1, -1, 0.0, -0.0],
                       [3, 1, 3, 1, 3, 1, 3, 1]], np.float32)
    ids, w, _ = oracle.route(cfg, np.arange(8), (), None, logits)
    assert ids.tolist() == [[0, 1, 2], [1, 2, 4], [0, 1, 6], [0, 2, 4]]
    np.testing.assert_allclose(w, 1.0 / 3.0, rtol=1e-6)
    ids, _, _ = oracle.route(cfg, np.arange(8), (0, 2), None, logits)
    assert ids.tolist() == [[1, 3, 4], [1, 4, 5], [1, 6, 7], [4, 6, 1]]


def test_group_ties_break_to_lower_group():
    cfg = oracle.OracleConfig(num_experts=8, top_k=2, num_ranks=8, slots_per_rank=1,
                              n_group=4, topk_group=2)
    logits = np.array([[1, 0, 1, 0, 1, 0, 1, 0]], np.float32)    # all group scores equal (m = 1)
    ids, _, _ = oracle.route(cfg, np.arange(8), (), None, logits)
    assert ids.tolist() == [[0, 2]]


# --------------------------------------------------------------------------
# P5: masking == -inf columns (Sec. 4.2), P6: redundancy preserves routing (Sec. 3.4)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "mixtral", "dsv3", "qwen3", "kimi"])
def test_mask_equals_minus_inf_columns(name):
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=256, with_x=False)
    cfg = oracle_cfg(wl)
    for failed in wl.failure_sets:
        if not failed:
            continue
        avail = _avail(wl, inp["slot_to_expert"], failed)
        ids, w, _ = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"])
        lg = inp["logits"].copy()
        lg[:, ~avail] = -np.inf
        ids2, w2, _ = oracle.route(cfg, inp["slot_to_expert"], (), inp["bias"], lg)
        assert np.array_equal(ids, ids2)
        assert np.array_equal(w, w2)
        assert avail[ids].all()


def test_redundancy_keeps_ids_and_weights():
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=512, with_x=False)
    s2e = inp["slot_to_expert"]
    cfg = oracle_cfg(wl)
    ids0, w0, slot0 = oracle.route(cfg, s2e, (), inp["bias"], inp["logits"])
    # fail a rank whose 8 base experts are all replicated elsewhere, if there is one;
    # else build such a placement by giving rank 0's experts their copies
    s2e2 = s2e.copy()
    for r in range(1, 9):
        s2e2[r * wl.S + wl.S - 1] = r - 1              # copies of experts 0..7 on ranks 1..8
    ids1, w1, slot1 = oracle.route(cfg, s2e2, (0,), inp["bias"], inp["logits"])
    ids2, w2, _ = oracle.route(cfg, s2e2, (), inp["bias"], inp["logits"])
    assert np.array_equal(ids1, ids2) and np.array_equal(w1, w2)
    assert np.all(slot1 // wl.S != 0)
    assert (slot1 != oracle.route(cfg, s2e2, (), inp["bias"], inp["logits"])[2]).any()
    assert np.array_equal(ids0.shape, ids1.shape)


# --------------------------------------------------------------------------
# P7: invariants, P11: fraction masked = 1/EP without redundancy
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "mixtral", "dsv3", "qwen3", "kimi"])
def test_invariants(name):
    wl = W.WORKLOADS[name]
    T = min(wl.T, 2048)
    inp = W.make_inputs(wl, T=T, with_x=False)
    cfg = oracle_cfg(wl)
    s2e = inp["slot_to_expert"]
    for failed in wl.failure_sets:
        ids, w, slot = oracle.route(cfg, s2e, failed, inp["bias"], inp["logits"])
        avail = _avail(wl, s2e, failed)
        assert all(len(set(row)) == wl.k for row in ids.tolist())
        assert avail[ids].all()
        assert np.array_equal(s2e[slot], ids), "the chosen slot hosts the chosen expert"
        assert not np.isin(slot // wl.S, list(failed)).any()
        np.testing.assert_allclose(w.astype(np.float64).sum(1), 1.0, rtol=1e-6)
        out = oracle.permutation(cfg, slot)
        assert out["slot_counts"].sum() == T * wl.k
        assert sorted(out["dst_row"].tolist()) == list(range(T * wl.k))


def test_replica_choice_is_token_index_mod_live_count():
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl)
    ids, _, slot = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (), None, inp["logits"])
    live = {0: [0, 8], 1: [1, 9]}
    for t in range(wl.T):
        for j in range(wl.k):
            e = int(ids[t, j])
            want = live[e][t % 2] if e in live else e
            assert slot[t, j] == want
    ids, _, slot = oracle.route(oracle_cfg(wl), inp["slot_to_expert"], (4,), None, inp["logits"])
    assert np.array_equal(slot, ids)


def test_fraction_masked_is_one_over_ep():
    for name, frac in [("mixtral", 1 / 8), ("qwen3", 8 / 128)]:
        wl = W.WORKLOADS[name]
        avail = _avail(wl, W.slot_to_expert(wl), wl.failure_sets[0])
        assert (~avail).sum() / wl.E == frac == 1 / wl.R


# --------------------------------------------------------------------------
# P8: combine closed form  y[t,:] = c_t * x[t,:]
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "dsv3"])
def test_dispatch_then_combine_closed_form(name):
    wl = W.WORKLOADS[name]
    T, H = min(wl.T, 96), min(wl.H, 320)
    inp = W.make_inputs(wl, T=T, H=H)
    cfg = oracle_cfg(wl)
    failed = wl.failure_sets[-1]
    out = oracle.dispatch(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"], inp["x"])
    # scatter: row dst_row[i] holds token i // k, bit for bit
    assert np.array_equal(out["send_buf"][out["dst_row"]], np.repeat(inp["x"], wl.k, axis=0))
    y = oracle.combine(out["send_buf"], out["dst_row"], out["topk_weights"], out["topk_slot"],
                       inp["slot_scale"])
    coef = (out["topk_weights"] * inp["slot_scale"][out["topk_slot"]]).astype(np.float64).sum(1)
    ref = coef[:, None] * bf16_to_f64(inp["x"])
    got = bf16_to_f64(y)
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)      # half a bf16 ulp
    # unit scales: weights sum to 1, y == x up to one bf16 ulp
    y1 = oracle.combine(out["send_buf"], out["dst_row"], out["topk_weights"], out["topk_slot"],
                        np.ones(wl.P, np.float32))
    assert np.all(np.abs(bf16_to_f64(y1) - bf16_to_f64(inp["x"])) <= np.abs(bf16_to_f64(inp["x"])) * 2.0 ** -7)


def test_combine_uses_weight_times_scale_per_slot():
    # two rows with different scales and weights; result checked by hand
    buf = W.f32_to_bf16_bits(np.array([[2.0, -4.0], [8.0, 16.0]], np.float32))
    y = oracle.combine(buf, [1, 0], np.array([[0.25, 0.75]], np.float32),
                       np.array([[3, 5]], np.int32), np.array([0, 0, 0, 2.0, 0, 0.5], np.float32))
    # token 0: j=0 reads row 1 with 0.25*2.0, j=1 reads row 0 with 0.75*0.5
    assert W.bf16_bits_to_f32(y).tolist() == [[0.5 * 8 + 0.375 * 2, 0.5 * 16 - 0.375 * 4]]


# --------------------------------------------------------------------------
# P9: failing ranks == emptying their slots in the replica map
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "dsv3", "kimi"])
def test_failed_ranks_equal_emptied_slots(name):
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=256, with_x=False)
    cfg = oracle_cfg(wl)
    failed = wl.failure_sets[-1]
    a = oracle.route(cfg, inp["slot_to_expert"], failed, inp["bias"], inp["logits"])
    s2e = inp["slot_to_expert"].copy()
    for r in failed:
        s2e[r * wl.S:(r + 1) * wl.S] = -1
    b = oracle.route(cfg, s2e, (), inp["bias"], inp["logits"])
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


# --------------------------------------------------------------------------
# remap admission rule
# --------------------------------------------------------------------------

def test_failure_set_admission_ungrouped():
    cfg = oracle.OracleConfig(num_experts=8, top_k=2, num_ranks=8, slots_per_rank=1)
    s2e = np.arange(8)
    assert oracle.failure_set_ok(cfg, s2e, range(6))
    assert not oracle.failure_set_ok(cfg, s2e, range(7))
    with pytest.raises(ValueError):
        oracle.route(cfg, s2e, range(7), None, np.zeros((1, 8), np.float32))


def test_failure_set_admission_grouped_is_exact():
    # 4 groups of 2, keep 2 groups, k = 4 (m = 2): every pair of non-empty groups must hold >= 4
    cfg = oracle.OracleConfig(num_experts=8, top_k=4, num_ranks=8, slots_per_rank=1,
                              n_group=4, topk_group=2)
    s2e = np.arange(8)
    rng = np.random.default_rng(3)
    for failed in [(), (0,), (0, 1), (0, 1, 2, 3), (0, 2), (0, 1, 2, 3, 4, 5)]:
        ok = oracle.failure_set_ok(cfg, s2e, failed)
        # exhaustive-ish check: random logits plus adversarial ones that push the weakest groups up
        feasible = True
        avail = np.ones(8, bool)
        avail[list(failed)] = False
        gcount = avail.reshape(4, 2).sum(1)
        for trial in range(200):
            lg = rng.standard_normal((1, 8)).astype(np.float32)
            if trial < 24:
                order = list(itertools.permutations(range(4)))[trial]
                lg += np.repeat(np.array(order, np.float32) * 10, 2)[None, :]
            try:
                oracle.route(cfg, s2e, failed, None, lg)
            except ValueError:
                feasible = False
                break
        assert ok == feasible, (failed, gcount)
