"""Plain definition of the multi-GPU dispatch / combine exchange (Sec. 2.3).

TEST INFRASTRUCTURE ONLY.  Slow, explicit loops over receive buffers, slots,
senders and assignments, written from the definition of the layout:

  * GPU d of `world` hosts the physical slots [d*spg, (d+1)*spg), spg = P/world.
  * Receive buffer of GPU d: for its slots in ascending order, for the sending
    GPUs in ascending order, the sender's assignments i = t*k + j on that slot in
    ascending i; each contributes a bit copy of the sender's row x[t].
  * Combine on GPU g: y[t] = bf16( sum_j (w[t,j] * slot_scale[slot[t,j]]) *
    row of assignment (g, t, j) in its owner's buffer ), double accumulation,
    one rounding (the single-GPU combine of ``reference.combine`` applied to the
    fetched rows).

Routing of each sender's tokens is the single-GPU ``reference.route`` on that
sender's own batch (token index t is the index inside the batch).
"""
from __future__ import annotations

import numpy as np

from . import reference as R


def ep_dispatch(cfg: R.OracleConfig, world: int, slot_to_expert, failed_ranks, bias, logits_list, x_list,
                failed_experts=None):
    """Returns (per_sender, per_owner): lists of dicts.

    per_sender[g]: topk_ids, topk_weights, topk_slot, slot_counts [P], dst_row [T_g*k] (row in the owner's buffer)
    per_owner[d]:  recv_buf [rows_d, H] uint16, recv_slot_offsets [spg+1], recv_src [rows_d, 2] = (sender, i)
    """
    assert len(logits_list) == world and len(x_list) == world
    P, k = cfg.num_slots, cfg.top_k
    assert P % world == 0 and cfg.num_ranks % world == 0
    spg = P // world
    per_sender = []
    for g in range(world):
        ids, w, slot = R.route(cfg, slot_to_expert, failed_ranks, bias, logits_list[g], failed_experts)
        counts = np.zeros(P, np.int32)
        for s in slot.reshape(-1):
            counts[s] += 1
        per_sender.append(dict(topk_ids=ids, topk_weights=w, topk_slot=slot, slot_counts=counts,
                               dst_row=np.full(slot.size, -1, np.int32)))
    per_owner = []
    for d in range(world):
        rows, src, offsets = [], [], [0]
        for p in range(d * spg, (d + 1) * spg):
            for g in range(world):
                flat = per_sender[g]["topk_slot"].reshape(-1)
                x = np.asarray(x_list[g], dtype=np.uint16)
                for i in np.nonzero(flat == p)[0]:          # ascending i
                    per_sender[g]["dst_row"][i] = len(rows)
                    rows.append(x[i // k])
                    src.append((g, int(i)))
            offsets.append(len(rows))
        H = np.asarray(x_list[0]).shape[1]
        per_owner.append(dict(recv_buf=np.array(rows, np.uint16).reshape(len(rows), H),
                              recv_slot_offsets=np.array(offsets, np.int32),
                              recv_src=np.array(src, np.int32).reshape(len(src), 2)))
    return per_sender, per_owner


def ep_combine(cfg: R.OracleConfig, world: int, g: int, sender: dict, per_owner, slot_scale) -> np.ndarray:
    """y of sender g: fetch each assignment's row from its owner's buffer, then the single-GPU combine."""
    k = cfg.top_k
    spg = cfg.num_slots // world
    slot = sender["topk_slot"]
    T = slot.shape[0]
    H = per_owner[0]["recv_buf"].shape[1]
    fetched = np.empty((T * k, H), np.uint16)
    flat = slot.reshape(-1)
    for i in range(T * k):
        fetched[i] = per_owner[flat[i] // spg]["recv_buf"][sender["dst_row"][i]]
    return R.combine(fetched, np.arange(T * k, dtype=np.int32), sender["topk_weights"], slot, slot_scale)
