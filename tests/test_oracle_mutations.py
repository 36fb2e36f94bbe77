"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source
(a dropped term, a flipped tie, a wrong index, ...), builds it, and runs the CPU pin tests
against that build in a child process.  Every planted mistake must make at least one pin
fail; the untouched source must pass.  Nothing here touches a GPU or the CUDA library's kernels.
"""
import concurrent.futures
import os
import subprocess
import sys

import pytest

import oracle
from oracle import reference

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "moe_oracle.c")
PIN_FILES = ["tests/test_oracle_pins.py", "tests/test_expert_failures.py", "tests/test_rank_compaction.py",
             "tests/test_dense_ffn_groups.py", "tests/test_expert_parallel.py"]

TOPK_LOOP = ("            for (int e = 0; e < E; ++e) {\n"
             "                if (picked[e] || key[e] == -INFINITY) continue;\n"
             "                if (best < 0 || key[e] > key[best]) best = e;")
GROUP_LOOP = ("                        if (picked[e] || key[e] == -INFINITY) continue;\n"
              "                        if (best < 0 || key[e] > key[best]) best = e;")
GATED_SLOT = ("            int e = ids[j];\n"
              "            topk_slot[(size_t)t * k + j] = live[(size_t)e * P + (t % n_live[e])];")

# name -> (text in the source, what replaces it); each text occurs exactly once
MUTATIONS = {
    "bias dropped from the key": ("key[e] = score[e] + (bias ? bias[e] : 0.0f);", "key[e] = score[e];"),
    "bias leaks into the weights": ("u[j] = (double)score[ids[j]];", "u[j] = (double)key[ids[j]];"),
    "expert tie goes to the higher id": (TOPK_LOOP, TOPK_LOOP.replace("key[e] > key[best]", "key[e] >= key[best]")),
    "group tie goes to the higher group": ("gscore[g] > gscore[best]", "gscore[g] >= gscore[best]"),
    "masked experts poison the group score": (GROUP_LOOP, GROUP_LOOP.replace(" || key[e] == -INFINITY", "")),
    "group score uses one key": ("m = k / c->topk_group;", "m = 1;"),
    "one group too few is kept": ("for (int i = 0; i < c->topk_group; ++i) {", "for (int i = 0; i < c->topk_group - 1; ++i) {"),
    "always the first replica": (GATED_SLOT, GATED_SLOT.replace("(t % n_live[e])", "0")),
    "availability mask dropped": ("if (n_live[e] == 0) key[e] = -INFINITY;", ""),
    "failed ranks keep their slots": ("if (rank_failed[p / c->slots_per_rank]) continue;", ""),
    "slot mapped to the wrong rank": ("rank_failed[p / c->slots_per_rank]", "rank_failed[p % c->num_ranks]"),
    "lost experts still routed": ("if (expert_failed && expert_failed[e]) continue;", ""),
    "weights not renormalised": ("(double)c->route_scale * u[j] / usum", "(double)c->route_scale * u[j]"),
    "softmax weight without exp": ("u[j] = exp((double)d);", "u[j] = 1.0 + (double)d;"),
    "picks stored worst first": ("ids[j] = best;", "ids[k - 1 - j] = best;"),
    "order inside a slot reversed": ("dst_row[i] = slot_offsets[p] + seen[p]++;",
                                     "dst_row[i] = slot_offsets[p] + (slot_counts[p] - 1 - seen[p]++);"),
    "inclusive instead of exclusive offsets": ("            slot_offsets[p] = run;\n            run += slot_counts[p];",
                                               "            run += slot_counts[p];\n            slot_offsets[p] = run;"),
    "rank count keeps the last slot only": ("rank_counts[l] += slot_counts[p];", "rank_counts[l] = slot_counts[p];"),
    "scatter copies the wrong token": ("x + (size_t)(i / k) * H", "x + (size_t)(i % T) * H"),
    "combine forgets the slot scale": ("float coef = topk_weights[i] * slot_scale[topk_slot[i]];",
                                       "float coef = topk_weights[i];"),
    "combine reads row i instead of dst_row[i]": ("buf[(size_t)dst_row[i] * H + h]", "buf[(size_t)i * H + h]"),
    "bf16 rounding truncates": ("q = nearbyint(ldexp(m, bits));", "q = trunc(ldexp(m, bits));"),
    "exp polynomial loses a term": ("    p = fmaf(p, r, 0x1.555556p-3f);     /* 1/6    */\n", ""),
    "sigmoid of the wrong sign": ("float e = oracle_exp_spec(-x);", "float e = oracle_exp_spec(x);"),
    "dense groups: every token to the first healthy group": ("healthy[t % n_healthy]", "healthy[0]"),
    "grouped admission always accepts": ("ok = worst >= c->top_k;", "ok = 1;"),
    "switched device does not take the failed device's rank": (
        "if (cur[i] == replaced_rank) cur[i] = switched_rank;", ";"),
    "gap left by a failed rank is not closed": ("order[m++] = cur[i];", "order[i] = cur[i]; m = i + 1;"),
}


def run_pins(lib_path):
    env = dict(os.environ, MOE_ORACLE_LIB_OVERRIDE=lib_path)
    p = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider",
                        *PIN_FILES], cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    return p.returncode, p.stdout[-1500:]


def build_variant(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, f"{name}: the text to replace occurs {text.count(old)} times"
    tag = "".join(ch if ch.isalnum() else "_" for ch in name)
    src, lib = os.path.join(tmp_path, tag + ".c"), os.path.join(tmp_path, tag + ".so")
    with open(src, "w") as f:
        f.write(text.replace(old, new))
    reference.compile_source(src, lib)
    return lib


@pytest.mark.skipif(os.environ.get("MOE_ORACLE_LIB_OVERRIDE") is not None, reason="inside a mutation run")
def test_every_planted_mistake_fails_a_pin(tmp_path):
    oracle.build()
    control = os.path.join(tmp_path, "control.so")
    reference.compile_source(SRC, control)
    jobs = {"(control)": control}
    for name, (old, new) in MUTATIONS.items():
        jobs[name] = build_variant(str(tmp_path), name, old, new)
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as pool:
        results = dict(zip(jobs, pool.map(run_pins, jobs.values())))
    rc, out = results.pop("(control)")
    assert rc == 0, "the untouched oracle must pass its pins:\n" + out
    survivors = [name for name, (rc, _) in results.items() if rc == 0]
    assert not survivors, f"no pin noticed: {survivors}"
