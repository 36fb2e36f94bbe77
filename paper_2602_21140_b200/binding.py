"""Python binding of the C ABI in ``include/moe_route.h``.

Argument marshalling only: every step of the path runs in the CUDA kernels of
``csrc/libmoe_route.so``.  PyTorch supplies device memory and streams.  If the
compiled library is missing the import of any ``moe_*`` name fails loudly;
there is no CPU or PyTorch fallback.

Two layers:
  * ``moe_route_init`` ... ``moe_route_destroy``: one function per C entry point,
    same names, taking raw pointers / ctypes structs.
  * ``MoeRouter``: a small convenience class that owns a context and the output
    tensors of a dispatch, and passes ``tensor.data_ptr()`` and the current
    stream to the functions above.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "csrc", "libmoe_route.so")
_lib_handle = None

MOE_OK = 0
MOE_ERR_INVALID_ARG = 1
MOE_ERR_CUDA = 2
MOE_ERR_INSUFFICIENT_EXPERTS = 3
MOE_ERR_CAPACITY = 4
MOE_ERR_DEVICE_TIMEOUT = 5
MOE_SCORE_SOFTMAX = 0
MOE_SCORE_SIGMOID = 1
MOE_ROUTE_DENSE_TP = 2
# options of moe_set_tuning (include/moe_route.h, moe_tuning_option)
(MOE_TUNE_PDL, MOE_TUNE_SCATTER_IMPL, MOE_TUNE_SCATTER_BULK_STAGES, MOE_TUNE_SCATTER_BULK_CTAS_PER_SM,
 MOE_TUNE_SCATTER_BLOCKS_PER_SM, MOE_TUNE_SCATTER_UNROLL, MOE_TUNE_COMBINE_IMPL, MOE_TUNE_COMBINE_CHUNK,
 MOE_TUNE_COMBINE_STAGES, MOE_TUNE_COMBINE_WARPS, MOE_TUNE_COMBINE_CTAS_PER_SM,
 MOE_TUNE_ROUTE_LANES_PER_TOKEN, MOE_TUNE_ROUTE_TOKENS_PER_TILE, MOE_TUNE_SPIN_LIMIT,
 MOE_TUNE_ROUTE_PREFETCH, MOE_TUNE_SCATTER_STORE_POLICY) = range(16)

EXPORTED_SYMBOLS = (
    "moe_route_init", "moe_set_failed_ranks", "moe_update_replica_map", "moe_dispatch",
    "moe_combine", "moe_step_host", "moe_step_host_async", "moe_set_timing_event", "moe_get_device_status", "moe_plan_routing_state",
    "moe_workspace_bytes", "moe_route_destroy", "moe_status_string", "moe_permute_static",
    "moe_set_failed_experts", "moe_compact_ranks", "moe_set_rank_order",
    "moe_ep_attach", "moe_ep_route", "moe_ep_scatter", "moe_ep_combine", "moe_ep_plan_host",
    "moe_set_tuning", "moe_debug_skip_ticket",
)


class MoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {moe_status_string(status)}")


class moe_config(ctypes.Structure):
    _fields_ = [("num_experts", ctypes.c_int32), ("top_k", ctypes.c_int32),
                ("hidden", ctypes.c_int32), ("max_tokens", ctypes.c_int32),
                ("num_ranks", ctypes.c_int32), ("slots_per_rank", ctypes.c_int32),
                ("max_replicas", ctypes.c_int32), ("score_func", ctypes.c_int32),
                ("n_group", ctypes.c_int32), ("topk_group", ctypes.c_int32),
                ("replica_policy", ctypes.c_int32), ("route_scale", ctypes.c_float)]


class moe_dispatch_out(ctypes.Structure):
    _fields_ = [("topk_ids", ctypes.c_void_p), ("topk_weights", ctypes.c_void_p),
                ("topk_slot", ctypes.c_void_p), ("slot_counts", ctypes.c_void_p),
                ("slot_offsets", ctypes.c_void_p), ("rank_counts", ctypes.c_void_p),
                ("rank_offsets", ctypes.c_void_p), ("dst_row", ctypes.c_void_p),
                ("src_index", ctypes.c_void_p), ("send_buf", ctypes.c_void_p)]


class moe_ep_group(ctypes.Structure):
    _fields_ = [("world", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("recv_bufs", ctypes.POINTER(ctypes.c_void_p)), ("recv_rows", ctypes.c_int64)]


def library_path() -> str:
    return _LIB_PATH


def _lib():
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with "
                "`python -m paper_2602_21140_b200.build` (needs nvcc); there is no fallback path")
        lib = ctypes.CDLL(_LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        lib.moe_route_init.restype = ctypes.c_int
        lib.moe_route_init.argtypes = [ctypes.POINTER(moe_config), vp, vp, vp, vp, ctypes.POINTER(vp)]
        lib.moe_set_failed_ranks.restype = ctypes.c_int
        lib.moe_set_failed_ranks.argtypes = [vp, vp, i32, vp]
        lib.moe_set_failed_experts.restype = ctypes.c_int
        lib.moe_set_failed_experts.argtypes = [vp, vp, i32, vp]
        lib.moe_compact_ranks.restype = ctypes.c_int
        lib.moe_compact_ranks.argtypes = [i32, vp, i32, i32, i32, vp, ctypes.POINTER(i32)]
        lib.moe_set_rank_order.restype = ctypes.c_int
        lib.moe_set_rank_order.argtypes = [vp, vp, i32, vp]
        lib.moe_update_replica_map.restype = ctypes.c_int
        lib.moe_update_replica_map.argtypes = [vp, vp, vp]
        lib.moe_dispatch.restype = ctypes.c_int
        lib.moe_dispatch.argtypes = [vp, vp, vp, i32, ctypes.POINTER(moe_dispatch_out), vp]
        lib.moe_combine.restype = ctypes.c_int
        lib.moe_combine.argtypes = [vp, vp, i32, vp, vp]
        lib.moe_step_host.restype = ctypes.c_int
        lib.moe_step_host.argtypes = [vp, vp, vp, i32, ctypes.POINTER(moe_dispatch_out), vp, vp, vp, vp, vp]
        lib.moe_step_host_async.restype = ctypes.c_int
        lib.moe_step_host_async.argtypes = [vp, vp, vp, i32, ctypes.POINTER(moe_dispatch_out), vp, vp, vp, vp, vp]
        lib.moe_set_timing_event.restype = ctypes.c_int
        lib.moe_set_timing_event.argtypes = [vp, vp]
        lib.moe_get_device_status.restype = ctypes.c_int
        lib.moe_get_device_status.argtypes = [vp, ctypes.POINTER(i32)]
        lib.moe_plan_routing_state.restype = ctypes.c_int
        lib.moe_plan_routing_state.argtypes = [ctypes.POINTER(moe_config), vp, vp, i32, vp, vp,
                                               ctypes.POINTER(i32)]
        lib.moe_workspace_bytes.restype = ctypes.c_size_t
        lib.moe_workspace_bytes.argtypes = [ctypes.POINTER(moe_config)]
        lib.moe_route_destroy.restype = ctypes.c_int
        lib.moe_route_destroy.argtypes = [vp]
        lib.moe_permute_static.restype = ctypes.c_int
        lib.moe_permute_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.moe_ep_attach.restype = ctypes.c_int
        lib.moe_ep_attach.argtypes = [vp, ctypes.POINTER(moe_ep_group), vp]
        lib.moe_ep_route.restype = ctypes.c_int
        lib.moe_ep_route.argtypes = [vp, vp, i32, ctypes.POINTER(moe_dispatch_out), vp]
        lib.moe_ep_scatter.restype = ctypes.c_int
        lib.moe_ep_scatter.argtypes = [vp, vp, i32, vp, vp, vp]
        lib.moe_ep_combine.restype = ctypes.c_int
        lib.moe_ep_combine.argtypes = [vp, i32, vp, vp]
        lib.moe_ep_plan_host.restype = ctypes.c_int
        lib.moe_ep_plan_host.argtypes = [vp, i32, i32, i32, vp, vp]
        lib.moe_set_tuning.restype = ctypes.c_int
        lib.moe_set_tuning.argtypes = [vp, i32, i32]
        lib.moe_debug_skip_ticket.restype = ctypes.c_int
        lib.moe_debug_skip_ticket.argtypes = [vp]
        lib.moe_status_string.restype = ctypes.c_char_p
        lib.moe_status_string.argtypes = [ctypes.c_int]
        _lib_handle = lib
    return _lib_handle


def _np_ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float32)


# --------------------------------------------------------------------------
# one function per C entry point
# --------------------------------------------------------------------------

def moe_status_string(status: int) -> str:
    return _lib().moe_status_string(int(status)).decode()


def moe_workspace_bytes(cfg: moe_config) -> int:
    return int(_lib().moe_workspace_bytes(ctypes.byref(cfg)))


def moe_plan_routing_state(cfg: moe_config, slot_to_expert, failed_ranks):
    """Host-only remap planning.  Returns (status, rank_alive u32[], replica_table i32[E,max_rep], n_available)."""
    s2e = _i32(slot_to_expert)
    fr = _i32(list(failed_ranks))
    words = (cfg.num_ranks + 31) // 32
    alive = np.zeros(max(words, 1), np.uint32)
    table = np.full((max(cfg.num_experts, 1), max(cfg.max_replicas, 1)), -1, np.int32)
    n_avail = ctypes.c_int32(0)
    st = _lib().moe_plan_routing_state(ctypes.byref(cfg), _np_ptr(s2e), _np_ptr(fr) if fr.size else None,
                                       fr.size, _np_ptr(alive), _np_ptr(table), ctypes.byref(n_avail))
    return st, alive, table, int(n_avail.value)


def moe_route_init(cfg: moe_config, slot_to_expert, bias, slot_scale, cuda_stream: int = 0):
    """Returns (status, ctx handle or None)."""
    s2e = _i32(slot_to_expert)
    b = None if bias is None else _f32(bias)
    sc = _f32(slot_scale)
    if s2e.size != cfg.num_ranks * cfg.slots_per_rank or sc.size != s2e.size:
        return MOE_ERR_INVALID_ARG, None
    if b is not None and b.size != cfg.num_experts:
        return MOE_ERR_INVALID_ARG, None
    ctx = ctypes.c_void_p()
    st = _lib().moe_route_init(ctypes.byref(cfg), _np_ptr(s2e), _np_ptr(b), _np_ptr(sc),
                               ctypes.c_void_p(cuda_stream), ctypes.byref(ctx))
    return st, (ctx if st == MOE_OK else None)


def moe_set_failed_ranks(ctx, ranks, cuda_stream: int = 0) -> int:
    r = _i32(list(ranks))
    return _lib().moe_set_failed_ranks(ctx, _np_ptr(r) if r.size else None, r.size,
                                       ctypes.c_void_p(cuda_stream))


def moe_set_failed_experts(ctx, mask, cuda_stream: int = 0) -> int:
    """mask: iterable of num_experts flags (non-zero = lost), or None / empty to clear."""
    m = np.zeros(0, np.uint8) if mask is None else np.ascontiguousarray(np.asarray(mask) != 0, dtype=np.uint8)
    return _lib().moe_set_failed_experts(ctx, _np_ptr(m) if m.size else None, m.size,
                                         ctypes.c_void_p(cuda_stream))


def moe_compact_ranks(num_ranks: int, failed_ranks, switched_rank: int = -1, replaced_rank: int = -1):
    """Host-only rank compaction.  Returns (status, list of physical ranks in new logical order)."""
    fr = _i32(list(failed_ranks))
    out = np.full(max(num_ranks, 1), -1, np.int32)
    n = ctypes.c_int32(0)
    st = _lib().moe_compact_ranks(num_ranks, _np_ptr(fr) if fr.size else None, fr.size, switched_rank,
                                  replaced_rank, _np_ptr(out), ctypes.byref(n))
    return st, out[: n.value].tolist()


def moe_set_rank_order(ctx, logical_to_physical, cuda_stream: int = 0) -> int:
    o = _i32(list(logical_to_physical))
    return _lib().moe_set_rank_order(ctx, _np_ptr(o) if o.size else None, o.size, ctypes.c_void_p(cuda_stream))


def moe_update_replica_map(ctx, slot_to_expert, cuda_stream: int = 0) -> int:
    s2e = _i32(slot_to_expert)
    return _lib().moe_update_replica_map(ctx, _np_ptr(s2e), ctypes.c_void_p(cuda_stream))


def moe_dispatch(ctx, logits_ptr: int, x_ptr: int, T: int, out: moe_dispatch_out,
                 cuda_stream: int = 0) -> int:
    return _lib().moe_dispatch(ctx, ctypes.c_void_p(logits_ptr), ctypes.c_void_p(x_ptr), T,
                               ctypes.byref(out), ctypes.c_void_p(cuda_stream))


def moe_combine(ctx, expert_buf_ptr: int, T: int, y_ptr: int, cuda_stream: int = 0) -> int:
    return _lib().moe_combine(ctx, ctypes.c_void_p(expert_buf_ptr), T, ctypes.c_void_p(y_ptr),
                              ctypes.c_void_p(cuda_stream))


def moe_step_host(ctx, logits_host_ptr: int, x_host_ptr: int, T: int, out: moe_dispatch_out,
                  logits_dev_ptr: int, x_dev_ptr: int, y_dev_ptr: int, y_host_ptr: int,
                  cuda_stream: int = 0) -> int:
    vp = ctypes.c_void_p
    return _lib().moe_step_host(ctx, vp(logits_host_ptr), vp(x_host_ptr), T, ctypes.byref(out),
                                vp(logits_dev_ptr), vp(x_dev_ptr), vp(y_dev_ptr), vp(y_host_ptr),
                                vp(cuda_stream))


def moe_step_host_async(ctx, logits_host_ptr: int, x_host_ptr: int, T: int, out: moe_dispatch_out,
                        logits_dev_ptr: int, x_dev_ptr: int, y_dev_ptr: int, y_host_ptr: int,
                        cuda_stream: int = 0) -> int:
    vp = ctypes.c_void_p
    return _lib().moe_step_host_async(ctx, vp(logits_host_ptr), vp(x_host_ptr), T, ctypes.byref(out),
                                      vp(logits_dev_ptr), vp(x_dev_ptr), vp(y_dev_ptr), vp(y_host_ptr),
                                      vp(cuda_stream))


def moe_set_timing_event(ctx, cuda_event: int) -> int:
    return _lib().moe_set_timing_event(ctx, ctypes.c_void_p(cuda_event) if cuda_event else None)


def moe_set_tuning(ctx, option: int, value: int) -> int:
    return _lib().moe_set_tuning(ctx, int(option), int(value))


def moe_debug_skip_ticket(ctx) -> int:
    return _lib().moe_debug_skip_ticket(ctx)


def moe_get_device_status(ctx):
    code = ctypes.c_int32(0)
    st = _lib().moe_get_device_status(ctx, ctypes.byref(code))
    return st, int(code.value)


def moe_permute_static(topk_slot_ptr: int, n_assign: int, num_ranks: int, slots_per_rank: int,
                       slot_counts_ptr: int, slot_offsets_ptr: int, rank_counts_ptr: int,
                       rank_offsets_ptr: int, dst_row_ptr: int, src_index_ptr: int,
                       cuda_stream: int = 0) -> int:
    """Count / scan / stable permutation from caller-owned device buffers, using only the
    library's built-in scratch array: for callers that are not able to allocate device
    memory (see include/moe_route.h).  All pointer arguments are raw device addresses."""
    vp = ctypes.c_void_p
    return _lib().moe_permute_static(vp(topk_slot_ptr), n_assign, num_ranks, slots_per_rank,
                                     vp(slot_counts_ptr), vp(slot_offsets_ptr), vp(rank_counts_ptr),
                                     vp(rank_offsets_ptr), vp(dst_row_ptr), vp(src_index_ptr),
                                     vp(cuda_stream))


def moe_ep_attach(ctx, world: int, rank: int, recv_buf_ptrs, recv_rows: int, cuda_stream: int = 0) -> int:
    """recv_buf_ptrs: `world` raw device addresses, usable from the calling GPU."""
    ptrs = (ctypes.c_void_p * max(world, 1))(*[int(a) for a in recv_buf_ptrs])
    group = moe_ep_group(world, rank, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), recv_rows)
    return _lib().moe_ep_attach(ctx, ctypes.byref(group), ctypes.c_void_p(cuda_stream))


def moe_ep_route(ctx, logits_ptr: int, T: int, out: moe_dispatch_out, cuda_stream: int = 0) -> int:
    return _lib().moe_ep_route(ctx, ctypes.c_void_p(logits_ptr), T, ctypes.byref(out),
                               ctypes.c_void_p(cuda_stream))


def moe_ep_scatter(ctx, x_ptr: int, T: int, counts_all_ptr: int, recv_slot_offsets_ptr: int,
                   cuda_stream: int = 0) -> int:
    vp = ctypes.c_void_p
    return _lib().moe_ep_scatter(ctx, vp(x_ptr), T, vp(counts_all_ptr), vp(recv_slot_offsets_ptr),
                                 vp(cuda_stream))


def moe_ep_combine(ctx, T: int, y_ptr: int, cuda_stream: int = 0) -> int:
    return _lib().moe_ep_combine(ctx, T, ctypes.c_void_p(y_ptr), ctypes.c_void_p(cuda_stream))


def moe_ep_plan_host(counts_all, rank: int):
    """Host-only layout of the exchange.  counts_all: [world, P] ints.
    Returns (status, src_base i32[P], recv_slot_offsets i32[P/world + 1])."""
    c = _i32(counts_all)
    world, P = c.shape
    src_base = np.zeros(P, np.int32)
    recv_off = np.zeros(P // max(world, 1) + 1, np.int32)
    st = _lib().moe_ep_plan_host(_np_ptr(c), world, rank, P, _np_ptr(src_base), _np_ptr(recv_off))
    return st, src_base, recv_off


def moe_route_destroy(ctx) -> int:
    return _lib().moe_route_destroy(ctx)


# --------------------------------------------------------------------------
# convenience layer over torch tensors
# --------------------------------------------------------------------------

@dataclass
class DispatchBuffers:
    """Device tensors written by one dispatch (caller-owned, reusable)."""
    topk_ids: torch.Tensor
    topk_weights: torch.Tensor
    topk_slot: torch.Tensor
    slot_counts: torch.Tensor
    slot_offsets: torch.Tensor
    rank_counts: torch.Tensor
    rank_offsets: torch.Tensor
    dst_row: torch.Tensor
    src_index: torch.Tensor
    send_buf: torch.Tensor

    def as_struct(self) -> moe_dispatch_out:
        return moe_dispatch_out(*(getattr(self, f).data_ptr() for f, _ in moe_dispatch_out._fields_))


def make_config(num_experts, top_k, hidden, max_tokens, num_ranks, slots_per_rank, max_replicas=2,
                score_func=MOE_SCORE_SOFTMAX, n_group=1, topk_group=1, route_scale=1.0) -> moe_config:
    return moe_config(num_experts, top_k, hidden, max_tokens, num_ranks, slots_per_rank,
                      max_replicas, score_func, n_group, topk_group, 0, route_scale)


class MoeRouter:
    """Owns one library context on a CUDA device."""

    def __init__(self, cfg: moe_config, slot_to_expert, bias, slot_scale, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise RuntimeError("MoeRouter needs a CUDA device; there is no CPU path")
        self._ctx = None
        with torch.cuda.device(self.device):
            st, ctx = moe_route_init(cfg, slot_to_expert, bias, slot_scale, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_route_init")
        self._ctx = ctx

    # -- helpers ----------------------------------------------------------
    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    @property
    def num_slots(self) -> int:
        return self.cfg.num_ranks * self.cfg.slots_per_rank

    def alloc_outputs(self, T: int) -> DispatchBuffers:
        c, dev = self.cfg, self.device
        n = T * c.top_k
        i32 = dict(dtype=torch.int32, device=dev)
        return DispatchBuffers(
            topk_ids=torch.empty((T, c.top_k), **i32),
            topk_weights=torch.empty((T, c.top_k), dtype=torch.float32, device=dev),
            topk_slot=torch.empty((T, c.top_k), **i32),
            slot_counts=torch.empty(self.num_slots, **i32),
            slot_offsets=torch.empty(self.num_slots + 1, **i32),
            rank_counts=torch.empty(c.num_ranks, **i32),
            rank_offsets=torch.empty(c.num_ranks + 1, **i32),
            dst_row=torch.empty(n, **i32),
            src_index=torch.empty(n, **i32),
            send_buf=torch.empty((n, c.hidden), dtype=torch.bfloat16, device=dev))

    # -- recovery -----------------------------------------------------------
    def set_failed_ranks(self, ranks) -> None:
        st = moe_set_failed_ranks(self._ctx, ranks, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_set_failed_ranks")

    def set_failed_experts(self, mask) -> None:
        st = moe_set_failed_experts(self._ctx, mask, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_set_failed_experts")

    def set_rank_order(self, logical_to_physical) -> None:
        st = moe_set_rank_order(self._ctx, logical_to_physical, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_set_rank_order")

    def update_replica_map(self, slot_to_expert) -> None:
        st = moe_update_replica_map(self._ctx, slot_to_expert, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_update_replica_map")

    # -- hot path -----------------------------------------------------------
    def dispatch(self, logits: torch.Tensor, x: torch.Tensor, out: DispatchBuffers | None = None) -> DispatchBuffers:
        T = logits.shape[0]
        assert logits.dtype == torch.float32 and logits.is_contiguous() and logits.shape[1] == self.cfg.num_experts
        assert x.dtype == torch.bfloat16 and x.is_contiguous() and tuple(x.shape) == (T, self.cfg.hidden)
        if out is None:
            out = self.alloc_outputs(T)
        struct = out.as_struct()
        st = moe_dispatch(self._ctx, logits.data_ptr(), x.data_ptr(), T, struct, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_dispatch")
        return out

    def combine(self, expert_buf: torch.Tensor, T: int, y: torch.Tensor | None = None) -> torch.Tensor:
        assert expert_buf.dtype == torch.bfloat16 and expert_buf.is_contiguous()
        if y is None:
            y = torch.empty((T, self.cfg.hidden), dtype=torch.bfloat16, device=self.device)
        st = moe_combine(self._ctx, expert_buf.data_ptr(), T, y.data_ptr(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_combine")
        return y

    # -- expert parallelism over several GPUs -------------------------------
    def ep_attach(self, world: int, rank: int, recv_buf_ptrs, recv_rows: int) -> None:
        st = moe_ep_attach(self._ctx, world, rank, recv_buf_ptrs, recv_rows, self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_ep_attach")

    def ep_route(self, logits: torch.Tensor, out: DispatchBuffers) -> DispatchBuffers:
        T = logits.shape[0]
        assert logits.dtype == torch.float32 and logits.is_contiguous() and logits.shape[1] == self.cfg.num_experts
        st = moe_ep_route(self._ctx, logits.data_ptr(), T, out.as_struct(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_ep_route")
        return out

    def ep_scatter(self, x: torch.Tensor, counts_all: torch.Tensor, recv_slot_offsets: torch.Tensor) -> None:
        T = x.shape[0]
        assert x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[1] == self.cfg.hidden
        assert counts_all.dtype == torch.int32 and counts_all.is_contiguous()
        assert recv_slot_offsets.dtype == torch.int32 and recv_slot_offsets.is_contiguous()
        st = moe_ep_scatter(self._ctx, x.data_ptr(), T, counts_all.data_ptr(),
                            recv_slot_offsets.data_ptr(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_ep_scatter")

    def ep_combine(self, T: int, y: torch.Tensor | None = None) -> torch.Tensor:
        if y is None:
            y = torch.empty((T, self.cfg.hidden), dtype=torch.bfloat16, device=self.device)
        st = moe_ep_combine(self._ctx, T, y.data_ptr(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_ep_combine")
        return y

    def step_host(self, logits_host: torch.Tensor, x_host: torch.Tensor, out: DispatchBuffers,
                  logits_dev: torch.Tensor, x_dev: torch.Tensor, y_dev: torch.Tensor,
                  y_host: torch.Tensor) -> None:
        T = logits_host.shape[0]
        st = moe_step_host(self._ctx, logits_host.data_ptr(), x_host.data_ptr(), T, out.as_struct(),
                           logits_dev.data_ptr(), x_dev.data_ptr(), y_dev.data_ptr(),
                           y_host.data_ptr(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_step_host")

    def step_host_async(self, logits_host: torch.Tensor, x_host: torch.Tensor, out: DispatchBuffers,
                        logits_dev: torch.Tensor, x_dev: torch.Tensor, y_dev: torch.Tensor,
                        y_host: torch.Tensor) -> None:
        """As step_host, but returns once the work is enqueued on the current stream."""
        T = logits_host.shape[0]
        st = moe_step_host_async(self._ctx, logits_host.data_ptr(), x_host.data_ptr(), T, out.as_struct(),
                                 logits_dev.data_ptr(), x_dev.data_ptr(), y_dev.data_ptr(),
                                 y_host.data_ptr(), self._stream())
        if st != MOE_OK:
            raise MoeError(st, "moe_step_host_async")

    def set_timing_event(self, event: "torch.cuda.Event | None") -> None:
        """Record `event` between the routing and the scatter kernel of every dispatch."""
        handle = 0
        if event is not None:
            event.record(torch.cuda.current_stream(self.device))   # forces creation of the handle
            handle = event.cuda_event
        st = moe_set_timing_event(self._ctx, handle)
        if st != MOE_OK:
            raise MoeError(st, "moe_set_timing_event")

    def set_tuning(self, option: int, value: int) -> None:
        """Override one launch choice of the context (see moe_tuning_option); -1 = automatic."""
        st = moe_set_tuning(self._ctx, option, value)
        if st != MOE_OK:
            raise MoeError(st, "moe_set_tuning")

    def device_status(self) -> int:
        st, code = moe_get_device_status(self._ctx)
        if st != MOE_OK:
            raise MoeError(st, "moe_get_device_status")
        return code

    def close(self) -> None:
        if self._ctx is not None:
            moe_route_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def config_for_workload(wl, max_tokens: int | None = None, hidden: int | None = None,
                        route_scale: float = 1.0) -> moe_config:
    """moe_config for one of ``workloads.WORKLOADS`` (shape bookkeeping only)."""
    return make_config(num_experts=wl.E, top_k=wl.k, hidden=wl.H if hidden is None else hidden,
                       max_tokens=wl.T if max_tokens is None else max_tokens, num_ranks=wl.R,
                       slots_per_rank=wl.S, max_replicas=wl.max_replicas, score_func=wl.score_func,
                       n_group=wl.n_group, topk_group=wl.topk_group, route_scale=route_scale)
