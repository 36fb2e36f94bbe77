"""ctypes front end of the C oracle (``moe_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Argument marshalling between numpy arrays and the
plain C functions; no arithmetic of the method lives here.  bf16 tensors are
numpy ``uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")
# The mutation test points this front end at deliberately broken builds of the C source.
_OVERRIDE = os.environ.get("MOE_ORACLE_LIB_OVERRIDE")
_lib = None


def compile_source(src: str, lib: str) -> None:
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call(
        ["gcc", "-O2", "-ffp-contract=off", "-std=c11", "-Wall", "-shared", "-fPIC",
         "-o", tmp, src, "-lm"])
    os.replace(tmp, lib)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (contraction off) if the library is stale."""
    if _OVERRIDE:
        return _OVERRIDE
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        compile_source(_SRC, _LIB)
    return _LIB


class _Cfg(ctypes.Structure):
    _fields_ = [("num_experts", ctypes.c_int32), ("top_k", ctypes.c_int32),
                ("num_ranks", ctypes.c_int32), ("slots_per_rank", ctypes.c_int32),
                ("score_func", ctypes.c_int32), ("n_group", ctypes.c_int32),
                ("topk_group", ctypes.c_int32), ("route_scale", ctypes.c_float)]


@dataclass
class OracleConfig:
    num_experts: int
    top_k: int
    num_ranks: int
    slots_per_rank: int
    score_func: int = 0      # 0 softmax, 1 sigmoid + bias
    n_group: int = 1
    topk_group: int = 1
    route_scale: float = 1.0

    @property
    def num_slots(self) -> int:
        return self.num_ranks * self.slots_per_rank

    def _c(self) -> _Cfg:
        return _Cfg(self.num_experts, self.top_k, self.num_ranks, self.slots_per_rank,
                    self.score_func, self.n_group, self.topk_group, self.route_scale)


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_exp_spec.restype = ctypes.c_float
        lib.oracle_exp_spec.argtypes = [ctypes.c_float]
        lib.oracle_sigmoid_spec.restype = ctypes.c_float
        lib.oracle_sigmoid_spec.argtypes = [ctypes.c_float]
        lib.oracle_exp_spec_array.restype = None
        lib.oracle_sigmoid_spec_array.restype = None
        lib.oracle_double_to_bf16.restype = ctypes.c_uint16
        lib.oracle_double_to_bf16.argtypes = [ctypes.c_double]
        lib.oracle_failure_set_ok.restype = ctypes.c_int32
        lib.oracle_route.restype = ctypes.c_int32
        lib.oracle_permutation.restype = None
        lib.oracle_compact_ranks.restype = ctypes.c_int32
        lib.oracle_scatter.restype = None
        lib.oracle_combine.restype = None
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _arr(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def _failed_mask(cfg: OracleConfig, failed_ranks) -> np.ndarray:
    m = np.zeros(cfg.num_ranks, dtype=np.uint8)
    for r in failed_ranks:
        m[int(r)] = 1
    return m


def exp_spec(z) -> np.ndarray:
    lib = _load()
    z = _arr(z, np.float32)
    out = np.empty_like(z)
    lib.oracle_exp_spec_array(_p(z), _p(out), ctypes.c_int64(z.size))
    return out


def sigmoid_spec(x) -> np.ndarray:
    lib = _load()
    x = _arr(x, np.float32)
    out = np.empty_like(x)
    lib.oracle_sigmoid_spec_array(_p(x), _p(out), ctypes.c_int64(x.size))
    return out


def double_to_bf16(d) -> np.ndarray:
    lib = _load()
    d = _arr(d, np.float64)
    return np.array([lib.oracle_double_to_bf16(float(v)) for v in d.ravel()],
                    dtype=np.uint16).reshape(d.shape)


def _expert_mask(cfg: OracleConfig, failed_experts):
    if failed_experts is None:
        return None
    m = np.ascontiguousarray(np.asarray(failed_experts) != 0, dtype=np.uint8)
    assert m.size == cfg.num_experts
    return m


def failure_set_ok(cfg: OracleConfig, slot_to_expert, failed_ranks, failed_experts=None) -> bool:
    lib = _load()
    s2e = _arr(slot_to_expert, np.int32)
    assert s2e.size == cfg.num_slots
    failed = _failed_mask(cfg, failed_ranks)
    lost = _expert_mask(cfg, failed_experts)
    c = cfg._c()
    return bool(lib.oracle_failure_set_ok(ctypes.byref(c), _p(s2e), _p(failed),
                                          None if lost is None else _p(lost)))


def route(cfg: OracleConfig, slot_to_expert, failed_ranks, bias, logits, failed_experts=None):
    """Returns (topk_ids [T,k] i32, topk_weights [T,k] f32, topk_slot [T,k] i32)."""
    lib = _load()
    s2e = _arr(slot_to_expert, np.int32)
    assert s2e.size == cfg.num_slots
    failed = _failed_mask(cfg, failed_ranks)
    logits = _arr(logits, np.float32)
    T, E = logits.shape                       # dense mode (score_func 2) reads only the shape
    assert E == cfg.num_experts
    k = cfg.top_k
    b = None if bias is None else _arr(bias, np.float32)
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    slot = np.empty((T, k), np.int32)
    lost = _expert_mask(cfg, failed_experts)
    c = cfg._c()
    rc = lib.oracle_route(ctypes.byref(c), _p(s2e), _p(failed), None if lost is None else _p(lost),
                          None if b is None else _p(b), _p(logits), ctypes.c_int32(T),
                          _p(ids), _p(w), _p(slot))
    if rc != 0:
        raise ValueError("fewer than k selectable experts for some token")
    return ids, w, slot


def full_rank_order(cfg: OracleConfig, rank_order):
    """The listed ranks first, then the unlisted ones ascending (they own no rows)."""
    if rank_order is None:
        return None
    listed = [int(r) for r in rank_order]
    rest = [r for r in range(cfg.num_ranks) if r not in listed]
    return _arr(listed + rest, np.int32)


def compact_ranks(num_ranks: int, failed_ranks, switched_rank: int = -1, replaced_rank: int = -1):
    lib = _load()
    failed = np.zeros(num_ranks, np.uint8)
    for r in failed_ranks:
        failed[int(r)] = 1
    out = np.full(num_ranks, -1, np.int32)
    n = lib.oracle_compact_ranks(ctypes.c_int32(num_ranks), _p(failed), ctypes.c_int32(switched_rank),
                                 ctypes.c_int32(replaced_rank), _p(out))
    return out[:n].tolist()


def permutation(cfg: OracleConfig, topk_slot, rank_order=None):
    lib = _load()
    order = full_rank_order(cfg, rank_order)
    slot = _arr(topk_slot, np.int32)
    T, k = slot.shape
    assert k == cfg.top_k
    P, R = cfg.num_slots, cfg.num_ranks
    out = dict(slot_counts=np.empty(P, np.int32), slot_offsets=np.empty(P + 1, np.int32),
               rank_counts=np.empty(R, np.int32), rank_offsets=np.empty(R + 1, np.int32),
               dst_row=np.empty(T * k, np.int32), src_index=np.empty(T * k, np.int32))
    c = cfg._c()
    lib.oracle_permutation(ctypes.byref(c), _p(slot), ctypes.c_int32(T),
                           None if order is None else _p(order),
                           _p(out["slot_counts"]), _p(out["slot_offsets"]),
                           _p(out["rank_counts"]), _p(out["rank_offsets"]),
                           _p(out["dst_row"]), _p(out["src_index"]))
    return out


def scatter(x_bf16, dst_row, k: int) -> np.ndarray:
    lib = _load()
    x = _arr(x_bf16, np.uint16)
    T, H = x.shape
    dst = _arr(dst_row, np.int32)
    assert dst.size == T * k
    send = np.empty((T * k, H), np.uint16)
    lib.oracle_scatter(_p(x), _p(dst), ctypes.c_int32(T), ctypes.c_int32(k),
                       ctypes.c_int32(H), _p(send))
    return send


def combine(buf_bf16, dst_row, topk_weights, topk_slot, slot_scale) -> np.ndarray:
    lib = _load()
    buf = _arr(buf_bf16, np.uint16)
    w = _arr(topk_weights, np.float32)
    slot = _arr(topk_slot, np.int32)
    T, k = w.shape
    H = buf.shape[1]
    assert buf.shape[0] == T * k
    dst = _arr(dst_row, np.int32)
    scale = _arr(slot_scale, np.float32)
    y = np.empty((T, H), np.uint16)
    lib.oracle_combine(_p(buf), _p(dst), _p(w), _p(slot), _p(scale),
                       ctypes.c_int32(T), ctypes.c_int32(k), ctypes.c_int32(H), _p(y))
    return y


def dispatch(cfg: OracleConfig, slot_to_expert, failed_ranks, bias, logits, x_bf16, failed_experts=None,
             rank_order=None):
    """Route, count, permute and scatter: everything ``moe_dispatch`` produces."""
    ids, w, slot = route(cfg, slot_to_expert, failed_ranks, bias, logits, failed_experts)
    out = permutation(cfg, slot, rank_order)
    out.update(topk_ids=ids, topk_weights=w, topk_slot=slot)
    out["send_buf"] = scatter(x_bf16, out["dst_row"], cfg.top_k)
    return out
