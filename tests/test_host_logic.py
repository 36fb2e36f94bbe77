"""CPU-only checks of the C-ABI library: it loads, exports every declared
symbol, validates configurations, and its host-side remap planning (bitmap,
replica table, admission rule) agrees with the oracle.  No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import build as build_mod
from paper_2602_21140_b200 import workloads as W
from util import oracle_cfg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build_library()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "moe_route.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(moe_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(B.library_path())
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings():
    assert B.moe_status_string(B.MOE_OK) == "MOE_OK"
    assert B.moe_status_string(B.MOE_ERR_INSUFFICIENT_EXPERTS) == "MOE_ERR_INSUFFICIENT_EXPERTS"
    assert B.moe_status_string(99) == "MOE_ERR_UNKNOWN"


@pytest.mark.parametrize("name", list(W.WORKLOADS))
def test_workspace_bytes_and_config_accepted(name):
    wl = W.WORKLOADS[name]
    cfg = B.config_for_workload(wl)
    n = B.moe_workspace_bytes(cfg)
    assert 0 < n < 64 << 20, "the context holds only small state"


@pytest.mark.parametrize("field,value", [
    ("num_experts", 0), ("num_experts", 513), ("top_k", 0), ("top_k", 17), ("hidden", 12),
    ("max_tokens", 0), ("num_ranks", 0), ("max_replicas", 9), ("score_func", 2),
    ("replica_policy", 1), ("route_scale", 0.0), ("n_group", 3), ("topk_group", 3)])
def test_invalid_configs_rejected(field, value):
    cfg = B.config_for_workload(W.WORKLOADS["dsv3"])
    setattr(cfg, field, value)
    assert B.moe_workspace_bytes(cfg) == 0
    st, *_ = B.moe_plan_routing_state(cfg, W.slot_to_expert(W.WORKLOADS["dsv3"]), [])
    assert st == B.MOE_ERR_INVALID_ARG


def _expected_table(wl, s2e):
    table = np.full((wl.E, wl.max_replicas), -1, np.int32)
    fill = np.zeros(wl.E, int)
    for p, e in enumerate(s2e):
        if e >= 0:
            table[e, fill[e]] = p
            fill[e] += 1
    return table


@pytest.mark.parametrize("name", list(W.WORKLOADS))
def test_plan_matches_definition(name):
    wl = W.WORKLOADS[name]
    cfg = B.config_for_workload(wl)
    s2e = W.slot_to_expert(wl)
    for failed in wl.failure_sets:
        st, alive, table, n_avail = B.moe_plan_routing_state(cfg, s2e, failed)
        assert st == B.MOE_OK
        bits = [(int(alive[r // 32]) >> (r % 32)) & 1 for r in range(wl.R)]
        assert bits == [0 if r in failed else 1 for r in range(wl.R)]
        assert np.array_equal(table, _expected_table(wl, s2e))
        avail = {int(e) for p, e in enumerate(s2e) if e >= 0 and p // wl.S not in failed}
        assert n_avail == len(avail)
        assert oracle.failure_set_ok(oracle_cfg(wl), s2e, failed)


def test_admission_rule_agrees_with_oracle_on_random_failure_sets():
    rng = np.random.default_rng(5)
    for name in ("tiny", "mixtral", "dsv3", "kimi"):
        wl = W.WORKLOADS[name]
        cfg = B.config_for_workload(wl)
        s2e = W.slot_to_expert(wl)
        seen = set()
        for _ in range(300):
            n = int(rng.integers(0, wl.R + 1))
            failed = tuple(sorted(rng.choice(wl.R, n, replace=False).tolist()))
            st, *_ = B.moe_plan_routing_state(cfg, s2e, failed)
            ok = oracle.failure_set_ok(oracle_cfg(wl), s2e, failed)
            assert (st == B.MOE_OK) == ok, (name, failed)
            assert st in (B.MOE_OK, B.MOE_ERR_INSUFFICIENT_EXPERTS)
            seen.add(st)
        assert len(seen) == 2, "the sweep must hit both outcomes"


def test_grouped_admission_counts_only_nonempty_groups():
    # 8 groups of 32: groups 0-4 entirely dead, groups 5-7 alive.  Fewer non-empty groups
    # than topk_group, so all three are kept and hold 96 >= 8 experts: accepted.
    wl = W.WORKLOADS["dsv3"]
    cfg = B.config_for_workload(wl)
    s2e = np.full(wl.P, -1, np.int32)
    s2e[:wl.E] = np.arange(wl.E)
    s2e[: 5 * 32] = -1
    st, _, _, n_avail = B.moe_plan_routing_state(cfg, s2e, [])
    assert st == B.MOE_OK and n_avail == 96
    assert oracle.failure_set_ok(oracle_cfg(wl), s2e, [])
    # one expert per group in four groups: the four weakest non-empty groups hold 4 < 8
    s2e[:] = -1
    for g in range(8):
        s2e[g * 32: g * 32 + (1 if g < 4 else 32)] = np.arange(g * 32, g * 32 + (1 if g < 4 else 32))
    st, *_ = B.moe_plan_routing_state(cfg, s2e, [])
    assert st == B.MOE_ERR_INSUFFICIENT_EXPERTS
    assert not oracle.failure_set_ok(oracle_cfg(wl), s2e, [])


def test_plan_rejects_bad_inputs():
    wl = W.WORKLOADS["tiny"]
    cfg = B.config_for_workload(wl)
    s2e = W.slot_to_expert(wl)
    assert B.moe_plan_routing_state(cfg, s2e, [5])[0] == B.MOE_ERR_INVALID_ARG      # rank out of range
    assert B.moe_plan_routing_state(cfg, s2e, [-1])[0] == B.MOE_ERR_INVALID_ARG
    assert B.moe_plan_routing_state(cfg, s2e, [2, 2, 2])[0] == B.MOE_OK              # duplicates allowed
    bad = s2e.copy(); bad[3] = 8
    assert B.moe_plan_routing_state(cfg, bad, [])[0] == B.MOE_ERR_INVALID_ARG        # expert id out of range
    crowded = s2e.copy(); crowded[2] = 0
    assert B.moe_plan_routing_state(cfg, crowded, [])[0] == B.MOE_ERR_CAPACITY       # 3 copies > max_replicas
    assert B.moe_plan_routing_state(cfg, s2e, [0, 1, 2, 3])[0] == B.MOE_OK           # experts 0,1 survive on rank 4
    assert B.moe_plan_routing_state(cfg, s2e, [0, 1, 2, 4])[0] == B.MOE_OK           # experts 6,7 on rank 3
    assert B.moe_plan_routing_state(cfg, s2e, [0, 1, 2, 3, 4])[0] == B.MOE_ERR_INSUFFICIENT_EXPERTS


def test_init_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    wl = W.WORKLOADS["tiny"]
    inp = W.make_inputs(wl, with_x=False)
    st, ctx = B.moe_route_init(B.config_for_workload(wl), inp["slot_to_expert"], None, inp["slot_scale"])
    assert st == B.MOE_ERR_CUDA and ctx is None
    with pytest.raises(RuntimeError):
        B.MoeRouter(B.config_for_workload(wl), inp["slot_to_expert"], None, inp["slot_scale"], device="cpu")


def test_binding_structs_match_the_header_layout(tmp_path):
    # the ctypes mirrors of the header's structs must have the C compiler's sizes and offsets
    import ctypes
    import os
    import subprocess
    from paper_2602_21140_b200 import binding as B

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    fields = {"moe_config": [f for f, _ in B.moe_config._fields_],
              "moe_dispatch_out": [f for f, _ in B.moe_dispatch_out._fields_],
              "moe_ep_group": [f for f, _ in B.moe_ep_group._fields_]}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "moe_route.h"', 'int main(void) {']
    for s, fs in fields.items():
        lines.append(f'printf("{s} %zu\\n", sizeof({s}));')
        for f in fs:
            lines.append(f'printf("{s}.{f} %zu\\n", offsetof({s}, {f}));')
    lines += ['return 0; }']
    src, exe = tmp_path / "layout.c", tmp_path / "layout"
    src.write_text("\n".join(lines))
    subprocess.check_call(["gcc", "-I", os.path.join(root, "include"), "-o", str(exe), str(src)])
    got = dict(line.split() for line in subprocess.check_output([str(exe)], text=True).splitlines())
    for s in fields:
        cls = getattr(B, s)
        assert int(got[s]) == ctypes.sizeof(cls), s
        for f in fields[s]:
            assert int(got[f"{s}.{f}"]) == getattr(cls, f).offset, (s, f)


def test_benchmark_byte_accounting():
    # the roofline numerator: rows moved by the method (read x once, write k copies; read k rows,
    # write one) plus the small index traffic, per token and per step at the DeepSeek-V3 shape
    import bench
    from paper_2602_21140_b200 import workloads as W
    wl = W.WORKLOADS["dsv3"]
    per_kernel = bench.algorithmic_bytes(wl, wl.T)
    rows = (2 * wl.k + 2) * 2 * wl.H                       # 18 rows of 14 336 bytes
    assert rows == 258048
    per_token = sum(per_kernel.values()) // wl.T
    assert per_token == rows + 4 * wl.E + 52 * wl.k        # 1 024 B of logits, 416 B of indices
    assert per_token == 259488
    assert per_kernel["k_scatter"] > per_kernel["k_combine"] > 100 * per_kernel["k_route"]
    tiny = W.WORKLOADS["tiny"]
    assert bench.algorithmic_bytes(tiny, 0) == {"k_route": 0, "k_scatter": 0, "k_combine": 0}
