"""Expert parallelism over several GPUs: orchestration of ``moe_ep_*`` (marshalling only).

The exchange itself happens inside the kernels (rows are stored straight into the
owners' receive buffers and read back from them through peer pointers); this
module only wires the pieces together:

* ``EmulatedEpGroup`` runs a whole group on ONE device: one context per virtual
  GPU, the "peers" being buffers of the same device.  The virtual GPUs run one
  after the other on one stream, never as kernels that wait for each other.
* ``DistributedEp`` is the one-process-per-GPU form: ``torch.distributed``
  all-gathers the per-slot counts and orders the streams between the exchange
  steps; the receive buffers are allocated as symmetric memory so that every
  rank obtains peer pointers to all of them.
"""
from __future__ import annotations

import os

# The receive buffers are reached with plain peer loads, stores and (non-multicast) bulk
# copies only, so they are never bound to an NVLink multicast object, and the collectives
# used here (an all-gather of a few KB, one-word all-reduces) gain nothing from in-switch
# reduction.  Both libraries read these settings when they initialise, so they are set
# on import, before the caller creates its process group; a caller's own setting wins.
os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")
os.environ.setdefault("NCCL_NVLS_ENABLE", "0")

import torch  # noqa: E402

from . import binding as B  # noqa: E402


def gather_counts(slot_counts: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of one [P] int32 count vector per rank into [world, P] (any backend)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    flat = torch.empty(world * slot_counts.numel(), dtype=slot_counts.dtype, device=slot_counts.device)
    dist.all_gather_into_tensor(flat, slot_counts.contiguous().view(-1), group=group)
    return flat.view(world, slot_counts.numel())


class EmulatedEpGroup:
    """`world` virtual GPUs on one CUDA device, for checking the multi-GPU path where only one GPU exists."""

    def __init__(self, world: int, cfg: B.moe_config, slot_to_expert, bias, slot_scale, recv_rows: int,
                 device="cuda:0"):
        self.world, self.cfg, self.device = world, cfg, torch.device(device)
        self.routers = [B.MoeRouter(cfg, slot_to_expert, bias, slot_scale, device=device) for _ in range(world)]
        self.recv_rows = recv_rows
        self.recv_bufs = [torch.zeros((recv_rows, cfg.hidden), dtype=torch.bfloat16, device=self.device)
                          for _ in range(world)]
        ptrs = [b.data_ptr() for b in self.recv_bufs]
        for g, r in enumerate(self.routers):
            r.ep_attach(world, g, ptrs, recv_rows)
        P = cfg.num_ranks * cfg.slots_per_rank
        self.recv_slot_offsets = [torch.zeros(P // world + 1, dtype=torch.int32, device=self.device)
                                  for _ in range(world)]
        self.outs = None

    def set_failed_ranks(self, ranks) -> None:
        for r in self.routers:
            r.set_failed_ranks(ranks)

    def dispatch(self, logits_list, x_list):
        """Route on every virtual GPU, exchange the counts, scatter into the owners' buffers."""
        self.outs = [r.alloc_outputs(lg.shape[0]) for r, lg in zip(self.routers, logits_list)]
        for r, lg, out in zip(self.routers, logits_list, self.outs):
            r.ep_route(lg, out)
        counts_all = torch.stack([o.slot_counts for o in self.outs]).contiguous()   # the all-gather
        for g, (r, x) in enumerate(zip(self.routers, x_list)):
            r.ep_scatter(x, counts_all, self.recv_slot_offsets[g])
        return self.outs

    def combine(self, T_list):
        return [r.ep_combine(T) for r, T in zip(self.routers, T_list)]

    def device_status(self):
        return [r.device_status() for r in self.routers]

    def close(self) -> None:
        for r in self.routers:
            r.close()


class DistributedEp:
    """One rank of a real group (one process per GPU, NCCL).  The default process group is used."""

    def __init__(self, cfg: B.moe_config, slot_to_expert, bias, slot_scale, recv_rows: int, device):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        self.dist = dist
        self.world, self.rank = dist.get_world_size(), dist.get_rank()
        self.device = torch.device(device)
        self.router = B.MoeRouter(cfg, slot_to_expert, bias, slot_scale, device=device)
        # symmetric allocation: the rendezvous hands every rank a pointer to every rank's buffer
        self.recv_buf = symm_mem.empty((recv_rows, cfg.hidden), dtype=torch.bfloat16, device=self.device)
        handle = symm_mem.rendezvous(self.recv_buf, dist.group.WORLD)
        self._handle = handle
        self.router.ep_attach(self.world, self.rank, [int(p) for p in handle.buffer_ptrs], recv_rows)
        P = cfg.num_ranks * cfg.slots_per_rank
        self.recv_slot_offsets = torch.zeros(P // self.world + 1, dtype=torch.int32, device=self.device)
        self._token = torch.zeros(1, dtype=torch.int32, device=self.device)

    def _order_streams(self) -> None:
        # a collective on the current stream: it completes on a rank only after every rank has
        # reached it, i.e. after every rank's preceding kernels on that stream
        self.dist.all_reduce(self._token)

    def dispatch(self, logits: torch.Tensor, x: torch.Tensor, out: B.DispatchBuffers) -> B.DispatchBuffers:
        self.router.ep_route(logits, out)
        counts_all = gather_counts(out.slot_counts)
        self.router.ep_scatter(x, counts_all, self.recv_slot_offsets)
        self._order_streams()            # all rows have landed before anyone reads a receive buffer
        return out

    def combine(self, T: int, y: torch.Tensor | None = None) -> torch.Tensor:
        y = self.router.ep_combine(T, y)
        self._order_streams()            # all reads are done before the next scatter overwrites
        return y

    def close(self) -> None:
        self.router.close()
