"""The give-up path of the bounded device waits, exercised without hanging or faulting anything.

A routing tile waits for the count rows of all earlier tiles of its step.  The
wait is bounded: after a number of polls (a per-context setting) the tile sets
the context's status word to MOE_ERR_DEVICE_TIMEOUT and returns.  The test hook
`moe_debug_skip_ticket` makes the wait run out on purpose: the step's first tile
is never routed, so its flag is never published, and every other tile gives up
after a few thousand polls (about a millisecond).  The kernel returns on its own,
`moe_get_device_status` reports the timeout, clears it and re-arms the context,
and the next ordinary step matches the oracle again.
"""
import time

import numpy as np
import pytest
import torch

from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import make_router, run_and_check, to_dev

pytestmark = pytest.mark.gpu

POLLS = 2000


def _setup(T=1037, H=256):
    wl = W.WORKLOADS["dsv3"]
    inp = W.make_inputs(wl, T=T, H=H)
    router = make_router(wl, inp, max_tokens=T, hidden=H, tuning={B.MOE_TUNE_SPIN_LIMIT: POLLS})
    router.set_failed_ranks((7,))
    return wl, inp, router


def test_routing_alone_gives_up_reports_and_recovers():
    wl, inp, router = _setup()
    T = inp["logits"].shape[0]
    run_and_check(wl, inp, (7,), router=router)               # a healthy step first
    recv = torch.zeros((T * wl.k, inp["x"].shape[1]), dtype=torch.bfloat16, device="cuda")
    router.ep_attach(1, 0, [recv.data_ptr()], recv.shape[0])  # moe_ep_route launches the routing kernel alone
    out = router.alloc_outputs(T)
    for f in B.moe_dispatch_out._fields_:
        getattr(out, f[0]).zero_()
    assert B.moe_debug_skip_ticket(router._ctx) == B.MOE_OK
    t0 = time.perf_counter()
    router.ep_route(to_dev(inp["logits"]), out)
    torch.cuda.synchronize()                                  # the kernel returns by itself
    assert time.perf_counter() - t0 < 2.0
    assert router.device_status() == B.MOE_ERR_DEVICE_TIMEOUT
    assert router.device_status() == 0                        # reading cleared it
    # the skipped tile was never routed: its outputs are still the zeros put there
    tile = 32
    assert int(out.topk_weights[:tile].abs().sum()) == 0
    for _ in range(2):
        run_and_check(wl, inp, (7,), router=router)           # ordinary steps are exact again
    router.close()


def test_whole_step_behind_a_given_up_routing_stays_in_bounds():
    # dispatch + combine are enqueued behind the routing kernel that gives up (as in a captured
    # graph, where the host cannot step in): stale indices must be skipped, never followed
    wl, inp, router = _setup(T=777, H=128)
    T, H = inp["x"].shape
    run_and_check(wl, inp, (7,), router=router)
    out = router.alloc_outputs(T)
    guard = 64
    send = torch.full((T * wl.k + 2 * guard, H), 3.0, dtype=torch.bfloat16, device="cuda")
    yy = torch.full((T + 2 * guard, H), 3.0, dtype=torch.bfloat16, device="cuda")
    src = torch.full((T * wl.k + 2 * guard,), -5, dtype=torch.int32, device="cuda")
    out.send_buf = send[guard:guard + T * wl.k]
    out.src_index = src[guard:guard + T * wl.k]
    out.topk_slot.fill_(10 ** 6)                              # garbage that the routing kernel will not overwrite for tile 0
    out.dst_row.fill_(2 ** 30)
    assert B.moe_debug_skip_ticket(router._ctx) == B.MOE_OK
    logits, x = to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16)
    router.dispatch(logits, x, out)
    router.combine(out.send_buf, T, yy[guard:guard + T])
    torch.cuda.synchronize()
    assert router.device_status() == B.MOE_ERR_DEVICE_TIMEOUT
    for buf in (send, yy):
        assert bool((buf[:guard] == 3.0).all()) and bool((buf[-guard:] == 3.0).all())
    assert bool((src[:guard] == -5).all()) and bool((src[-guard:] == -5).all())
    assert bool(torch.isfinite(yy.float()).all())
    rows = out.dst_row
    assert bool(((rows >= -1) & (rows < T * wl.k)).all())
    assert router.device_status() == 0
    run_and_check(wl, inp, (7,), router=router)
    router.close()
