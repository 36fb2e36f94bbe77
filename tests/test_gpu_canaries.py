"""Out-of-bounds writes: every output of dispatch and combine sits between two
guard zones filled with a sentinel; after the kernels ran the guards must be
untouched.  (A memory checker is not available on the GPU pool, so the library's
index arithmetic is checked this way, on shapes with ragged tiles and tails.)"""
import numpy as np
import pytest
import torch

from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import make_router, to_dev

pytestmark = pytest.mark.gpu
GUARD = 256          # elements on each side


def _guarded(shape, dtype, fill):
    n = int(np.prod(shape))
    pad = GUARD
    whole = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
    return whole, whole[pad:pad + n].view(shape)


def _intact(whole, n, fill):
    return bool((whole[:GUARD] == fill).all()) and bool((whole[GUARD + n:] == fill).all())


@pytest.mark.parametrize("name,T,H", [("dsv3", 1037, 7168), ("kimi", 333, 264), ("tiny", 128, 256),
                                      ("qwen3", 1, 8), ("mixtral", 65, 4096), ("dsv3", 33, 1000)])
def test_guard_zones_stay_intact(name, T, H):
    wl = W.WORKLOADS[name]
    inp = W.make_inputs(wl, T=T, H=H)
    router = make_router(wl, inp, max_tokens=T, hidden=H)
    router.set_failed_ranks(wl.failure_sets[-1])
    n, k, P, R = T * wl.k, wl.k, wl.P, wl.R
    I32, SENT = torch.int32, -123456789
    bufs, views = {}, {}
    for f, shape in (("topk_ids", (T, k)), ("topk_slot", (T, k)), ("slot_counts", (P,)),
                     ("slot_offsets", (P + 1,)), ("rank_counts", (R,)), ("rank_offsets", (R + 1,)),
                     ("dst_row", (n,)), ("src_index", (n,))):
        bufs[f], views[f] = _guarded(shape, I32, SENT)
    bufs["topk_weights"], views["topk_weights"] = _guarded((T, k), torch.float32, -7.0)
    # bf16 guards: H is a multiple of 8, so GUARD elements keep the 16-byte alignment of the payload
    bufs["send_buf"], views["send_buf"] = _guarded((n, H), torch.bfloat16, -3.0)
    ywhole, y = _guarded((T, H), torch.bfloat16, -3.0)
    out = B.DispatchBuffers(**views)
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    for _ in range(2):
        router.dispatch(logits, x, out)
        router.combine(out.send_buf, T, y)
    torch.cuda.synchronize()
    assert router.device_status() == 0
    for f, whole in bufs.items():
        fill = -7.0 if f == "topk_weights" else (-3.0 if f == "send_buf" else SENT)
        assert _intact(whole, views[f].numel(), fill), f
    assert _intact(ywhole, y.numel(), -3.0), "y"
    # and everything inside was written
    for f in ("topk_ids", "topk_slot", "slot_counts", "slot_offsets", "rank_counts", "rank_offsets",
              "dst_row", "src_index"):
        assert not bool((views[f] == SENT).any()), f
    router.close()
