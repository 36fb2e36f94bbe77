"""Helpers for the GPU parity tests: run the CUDA library through its binding and
compare every output with the CPU oracle on the same seeded inputs."""
import numpy as np
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from util import bf16_to_f64, oracle_cfg

WEIGHT_RTOL = 1e-6        # renormalised weights, relative
Y_RTOL, Y_ATOL = 1e-2, 1e-3   # combined bf16 output: relative OR absolute

INT_FIELDS = ("topk_ids", "topk_slot", "slot_counts", "slot_offsets", "rank_counts",
              "rank_offsets", "dst_row", "src_index")


def to_dev(a: np.ndarray, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is torch.bfloat16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def make_router(wl, inp, max_tokens, hidden=None, route_scale=1.0, tuning=None) -> B.MoeRouter:
    """`tuning`: {moe_tuning_option: value} applied right after the context is created."""
    cfg = B.config_for_workload(wl, max_tokens=max_tokens, hidden=hidden, route_scale=route_scale)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    router = B.MoeRouter(cfg, inp["slot_to_expert"], bias, inp["slot_scale"])
    for option, value in (tuning or {}).items():
        router.set_tuning(option, value)
    return router


def assert_y_close(got_bits: np.ndarray, want_bits: np.ndarray):
    got, want = bf16_to_f64(got_bits), bf16_to_f64(want_bits)
    err = np.abs(got - want)
    ok = (err <= Y_RTOL * np.abs(want)) | (err <= Y_ATOL)
    assert ok.all(), f"{(~ok).sum()} of {ok.size} outputs outside tolerance, max err {err.max()}"


def check_dispatch(out: B.DispatchBuffers, ref: dict, check_send=True):
    for f in INT_FIELDS:
        got = getattr(out, f).cpu().numpy()
        assert np.array_equal(got.reshape(-1), ref[f].reshape(-1)), f
    w = out.topk_weights.cpu().numpy().astype(np.float64)
    rw = ref["topk_weights"].astype(np.float64)
    assert np.all(np.abs(w - rw) <= WEIGHT_RTOL * np.abs(rw)), "topk_weights"
    if check_send:
        assert np.array_equal(bf16_bits(out.send_buf), ref["send_buf"]), "send_buf"


def run_and_check(wl, inp, failed, router=None, route_scale=1.0, tuning=None):
    """Dispatch + combine on the GPU, compare everything with the oracle."""
    T, H = inp["x"].shape
    own = router is None
    if own:
        router = make_router(wl, inp, max_tokens=max(T, 1), hidden=H, route_scale=route_scale, tuning=tuning)
        router.set_failed_ranks(failed)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    out = router.dispatch(logits, x)
    y = router.combine(out.send_buf, T)
    torch.cuda.synchronize()
    assert router.device_status() == 0
    cfg = oracle_cfg(wl, route_scale)
    bias = inp["bias"] if wl.score_func == W.SIGMOID else None
    ref = oracle.dispatch(cfg, inp["slot_to_expert"], failed, bias, inp["logits"], inp["x"])
    check_dispatch(out, ref)
    ref_y = oracle.combine(ref["send_buf"], ref["dst_row"], ref["topk_weights"], ref["topk_slot"],
                           inp["slot_scale"])
    assert_y_close(bf16_bits(y), ref_y)
    if own:
        router.close()
    return out, y, ref
