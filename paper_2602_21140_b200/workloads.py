"""Seeded synthetic inputs for the five routing workloads.

This module only *draws inputs*: router logits, hidden states, biases,
per-slot scales, the slot-to-expert placement and the failed-rank sets.  None
of the method's arithmetic (gating, selection, counting, scatter, combine)
lives here, so both the CUDA library's tests and the CPU oracle's tests may
feed from it.  Everything is numpy on the host, drawn from a Philox
counter-based generator keyed by (seed, stream), so the same call gives the
same bits on every machine.

The shapes follow published model families (Mixtral, DeepSeek-V3, Qwen3-MoE,
Kimi-K2); the values are synthetic stand-ins for production routing traffic:
logits ~ N(0,1), optionally with a Zipf popularity skew added as
log(E * p_e), hidden states ~ N(0,1) rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SOFTMAX, SIGMOID = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    T: int                  # tokens per step
    H: int                  # hidden width (bf16)
    E: int                  # logical experts
    k: int                  # experts per token
    R: int                  # simulated EP ranks
    S: int                  # physical slots per rank
    score_func: int = SOFTMAX
    n_group: int = 1
    topk_group: int = 1
    zipf_s: float = 0.0     # 0 = no popularity skew
    n_redundant: int = 0    # extra copies of the hottest experts
    seed: int = 0
    failure_sets: tuple = field(default_factory=tuple)  # tuple of tuples of ranks
    max_replicas: int = 2

    @property
    def P(self) -> int:
        return self.R * self.S


def _kimi_failure_sets(seed: int, R: int, n_max: int):
    order = _rng(seed, 7).permutation(R)
    return tuple(tuple(int(r) for r in order[:n]) for n in range(n_max + 1))


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


WORKLOADS = {
    # 10 slots on 5 ranks; experts 0 and 1 have a second copy on rank 4; rank 2 fails.
    "tiny": Workload("tiny", T=128, H=256, E=8, k=2, R=5, S=2, seed=0,
                     n_redundant=2, failure_sets=((2,),)),
    "mixtral": Workload("mixtral", T=4096, H=4096, E=8, k=2, R=8, S=1, seed=1,
                        failure_sets=((3,),), max_replicas=1),
    "dsv3": Workload("dsv3", T=8192, H=7168, E=256, k=8, R=32, S=9, score_func=SIGMOID,
                     n_group=8, topk_group=4, zipf_s=1.1, n_redundant=32, seed=2,
                     failure_sets=((), (7,), (7, 20))),
    "qwen3": Workload("qwen3", T=16384, H=4096, E=128, k=8, R=16, S=8, seed=3,
                      failure_sets=((5,),), max_replicas=1),
    "kimi": Workload("kimi", T=32768, H=7168, E=384, k=8, R=64, S=7, score_func=SIGMOID,
                     zipf_s=1.2, n_redundant=64, seed=4,
                     failure_sets=_kimi_failure_sets(4, 64, 8)),
}


def popularity_rank(wl: Workload) -> np.ndarray:
    """rho[e] in 1..E: 1 = the hottest expert.  A seeded permutation."""
    if wl.zipf_s == 0.0:
        return np.arange(1, wl.E + 1, dtype=np.int64)
    perm = _rng(wl.seed, 5).permutation(wl.E)      # perm[i] = expert with rank i+1
    rho = np.empty(wl.E, dtype=np.int64)
    rho[perm] = np.arange(1, wl.E + 1)
    return rho


def slot_to_expert(wl: Workload) -> np.ndarray:
    """Placement of logical experts on the P = R*S physical slots.

    Slot p lives on rank p // S.  Without redundancy, slot p hosts expert p.
    With redundancy, each rank keeps b = S - 1 consecutive base experts in its
    first b slots and its last slot is an "extra" slot: the n_redundant
    hottest experts are walked hottest first and each gets one more copy on
    the lowest-numbered rank whose extra slot is still free and which is not
    the expert's home rank.  The tiny workload is the hand-laid case: slots
    0..7 host experts 0..7 and rank 4 hosts second copies of experts 0 and 1.
    Unused extra slots are empty (-1).
    """
    P = wl.P
    if wl.name == "tiny":
        return np.array([0, 1, 2, 3, 4, 5, 6, 7, 0, 1], dtype=np.int32)
    if wl.n_redundant == 0:
        assert P == wl.E
        return np.arange(P, dtype=np.int32)
    b = wl.S - 1
    assert wl.R * b == wl.E
    s2e = np.full(P, -1, dtype=np.int32)
    for r in range(wl.R):
        s2e[r * wl.S: r * wl.S + b] = np.arange(r * b, (r + 1) * b)
    rho = popularity_rank(wl)
    hottest = np.argsort(rho, kind="stable")[: wl.n_redundant]
    free = [True] * wl.R
    for e in hottest:
        home = int(e) // b
        for r in range(wl.R):
            if free[r] and r != home:
                s2e[r * wl.S + b] = e
                free[r] = False
                break
    return s2e


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (ties to even) and return the raw uint16 patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_inputs(wl: Workload, T: int | None = None, H: int | None = None,
                seed: int | None = None, with_x: bool = True) -> dict:
    """Draw one batch for ``wl`` (optionally at a reduced T / H for fast tests).

    Returns numpy arrays: ``logits`` [T,E] f32, ``x`` [T,H] bf16 bit patterns
    (uint16), ``bias`` [E] f32 (zeros in softmax mode), ``slot_scale`` [P] f32,
    ``slot_to_expert`` [P] i32.
    """
    T = wl.T if T is None else T
    H = wl.H if H is None else H
    seed = wl.seed if seed is None else seed
    logits = _rng(seed, 1).standard_normal((T, wl.E), dtype=np.float32)
    if wl.zipf_s > 0.0:
        rho = popularity_rank(wl).astype(np.float64)
        p = rho ** (-wl.zipf_s)
        p /= p.sum()
        logits = logits + np.log(wl.E * p).astype(np.float32)[None, :]
    out = {"logits": np.ascontiguousarray(logits, dtype=np.float32)}
    if with_x:
        x = _rng(seed, 2).standard_normal((T, H), dtype=np.float32)
        out["x"] = f32_to_bf16_bits(x)
    if wl.score_func == SIGMOID:
        out["bias"] = (0.05 * _rng(seed, 3).standard_normal(wl.E)).astype(np.float32)
    else:
        out["bias"] = np.zeros(wl.E, dtype=np.float32)
    out["slot_scale"] = _rng(seed, 4).uniform(0.5, 1.5, wl.P).astype(np.float32)
    out["slot_to_expert"] = slot_to_expert(wl)
    return out


# --------------------------------------------------------------------------
# Expert-level failure generators (the two selection policies of the paper's
# lost-expert experiment, Sec. 4.2).  They only choose WHICH experts fail.
# --------------------------------------------------------------------------

def every_nth_mask(E: int, r: float) -> np.ndarray:
    """Uniform policy: fail experts at a fixed step so that a fraction r is lost
    (r = 1/2 fails every even-indexed expert)."""
    step = int(round(1.0 / r))
    return (np.arange(E) % step == 0).astype(np.uint8)


def most_activated_mask(activation_counts, r: float) -> np.ndarray:
    """Worst-case policy: fail the fraction r of experts that were activated most
    often (counts aggregated by the caller; ties go to the lower expert id)."""
    counts = np.asarray(activation_counts, dtype=np.int64)
    n = int(round(r * counts.size))
    order = np.argsort(-counts, kind="stable")
    mask = np.zeros(counts.size, np.uint8)
    mask[order[:n]] = 1
    return mask
