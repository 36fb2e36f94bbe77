"""Shared helpers for the tests (no arithmetic of the method)."""
import numpy as np

import oracle
from paper_2602_21140_b200 import workloads as W


def oracle_cfg(wl: W.Workload, route_scale: float = 1.0) -> oracle.OracleConfig:
    return oracle.OracleConfig(num_experts=wl.E, top_k=wl.k, num_ranks=wl.R,
                               slots_per_rank=wl.S, score_func=wl.score_func,
                               n_group=wl.n_group, topk_group=wl.topk_group,
                               route_scale=route_scale)


def small_grouped_workload(E=16, k=4, n_group=4, topk_group=2, R=4, S=4, score_func=W.SIGMOID,
                           seed=11, name="grouped-small"):
    return W.Workload(name, T=64, H=64, E=E, k=k, R=R, S=S, score_func=score_func,
                      n_group=n_group, topk_group=topk_group, seed=seed)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return W.bf16_bits_to_f32(bits).astype(np.float64)
