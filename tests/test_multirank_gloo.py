"""World-size-2 checks (gloo, CPU) of the host logic the multi-GPU benchmark uses: the step
time is the maximum over ranks, replicas draw their own batches, and `bench.py --gpus 2`
starts two ranks by itself, shards tokens and slots, exchanges the per-slot counts and
prints one JSON line (walked here with `--dry-run`, which touches no GPU)."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import numpy as np
import torch.distributed as dist
import bench
from paper_2602_21140_b200 import workloads as W
import oracle

rank, local_rank, world = bench.env_rank()
dist.init_process_group("gloo")
assert world == 2
# max over ranks
assert bench.max_over_ranks(10.0 + rank, world) == 11.0
# ranks draw different batches of the same recipe
wl = W.WORKLOADS["tiny"]
inp = W.make_inputs(wl, seed=bench.shard_seed(wl.seed, rank))
digest = float(inp["logits"].astype(np.float64).sum())
other = [None, None]
dist.all_gather_object(other, digest)
assert other[0] != other[1]
# each rank's batch routes on its own; counts add up per rank with no exchange
cfg = bench.oracle_cfg_for(wl)
ids, w, slot = oracle.route(cfg, inp["slot_to_expert"], wl.failure_sets[0], None, inp["logits"])
perm = oracle.permutation(cfg, slot)
tot = [None, None]
dist.all_gather_object(tot, int(perm["slot_counts"].sum()))
assert tot == [wl.T * wl.k] * 2
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_gloo():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=300)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o


def test_reference_arm_prints_one_json_line():
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "2", "--warmup", "1", "--workload", "tiny", "--failure-set", "0"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0


def test_bench_starts_its_own_ranks_and_prints_one_line():
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run",
                          "--steps", "5", "--warmup", "3"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT,
                         env={k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")})
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1, out.stdout
    rec = json.loads(lines[0])
    assert rec["dry_run"] is True and rec["n_gpus"] == 2 and rec["scaling"] == "strong"
    assert rec["config"]["T_per_gpu"] == 4096 and rec["config"]["slots_per_gpu"] == 144
    assert rec["rows_total"] == 8192 * 8 and rec["max_over_ranks_check"] == 2.0
    for key in ("metric", "unit", "steps", "warmup", "higher_is_better", "vs_baseline", "dtype", "data", "config"):
        assert key in rec, key


def test_token_shards_cover_the_batch():
    import bench
    for T, world in ((8192, 8), (10, 4), (3, 8), (0, 2)):
        spans = [bench.shard_tokens(T, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == T
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1
