"""The allocation-free entry point (`moe_permute_static`) against the regular path and the oracle.

Some users of the library run inside a process that may not allocate device
memory after start-up (for instance a serving engine that has already claimed
all of HBM for its own pool).  They cannot build a context, so they call
`moe_permute_static`, which keeps its scratch in a fixed array inside the
library.  Here its counts, offsets and permutation are compared, bit for bit
(they are integers), with what `moe_dispatch` produces for the same slot
assignments AND with the CPU oracle's permutation of those assignments — twice
in a row with different inputs, because the second call finds the first call's
leftovers in the shared scratch.  The second call is also watched for device
allocations: the free-memory figure of the device must not move across it.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_21140_b200 import binding as B
from paper_2602_21140_b200 import workloads as W
from gpu_util import make_router, to_dev
from util import oracle_cfg

pytestmark = pytest.mark.gpu

FIELDS = ("slot_counts", "slot_offsets", "rank_counts", "rank_offsets", "dst_row", "src_index")


def _static_permute(wl, topk_slot: torch.Tensor):
    n = topk_slot.numel()
    i32 = dict(dtype=torch.int32, device="cuda")
    # poison the outputs so that an element the call fails to write is noticed
    res = {"slot_counts": torch.full((wl.P,), -7, **i32), "slot_offsets": torch.full((wl.P + 1,), -7, **i32),
           "rank_counts": torch.full((wl.R,), -7, **i32), "rank_offsets": torch.full((wl.R + 1,), -7, **i32),
           "dst_row": torch.full((n,), -7, **i32), "src_index": torch.full((n,), -7, **i32)}
    st = B.moe_permute_static(topk_slot.data_ptr(), n, wl.R, wl.S, *(res[f].data_ptr() for f in FIELDS),
                              torch.cuda.current_stream().cuda_stream)
    assert st == B.MOE_OK, B.moe_status_string(st)
    return res


def _regular_dispatch(wl, T, failed, seed):
    inp = W.make_inputs(wl, T=T, H=64, seed=seed)
    router = make_router(wl, inp, max_tokens=T, hidden=64)
    router.set_failed_ranks(failed)
    out = router.dispatch(to_dev(inp["logits"]), to_dev(inp["x"], torch.bfloat16))
    torch.cuda.synchronize()
    assert router.device_status() == 0
    router.close()
    return out


def test_two_calls_in_a_row_match_the_regular_path_and_the_oracle():
    # first call: large, skewed, 448 slots; second call: smaller and a different layout, so
    # stale histogram rows of the first call sit in the scratch the second call uses
    for call, (name, T, failed, seed) in enumerate((("kimi", 5000 + 13, (3, 40), 21), ("dsv3", 1037, (7, 20), 22))):
        wl = W.WORKLOADS[name]
        out = _regular_dispatch(wl, T, failed, seed)
        slots = out.topk_slot.reshape(-1)
        if call == 0:
            got = _static_permute(wl, slots)
        else:
            # by now the library's device code is loaded and the scratch address is known: this
            # call must leave the device's free memory exactly where it was (torch's own output
            # tensors are created before the first reading and stay alive past the second)
            warm = _static_permute(wl, slots)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            st = B.moe_permute_static(slots.data_ptr(), slots.numel(), wl.R, wl.S,
                                      *(warm[f].data_ptr() for f in FIELDS),
                                      torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            assert st == B.MOE_OK
            assert torch.cuda.mem_get_info()[0] == free_before, "moe_permute_static allocated device memory"
            got = warm
        torch.cuda.synchronize()
        ref = oracle.permutation(oracle_cfg(wl), slots.cpu().numpy().reshape(T, wl.k))
        for f in FIELDS:
            assert torch.equal(got[f], getattr(out, f).reshape(-1)), (name, f)
            assert np.array_equal(got[f].cpu().numpy(), ref[f].reshape(-1)), (name, f, "oracle")


def test_sizes_beyond_the_built_in_scratch_are_refused():
    i32 = dict(dtype=torch.int32, device="cuda")
    buf = torch.zeros(1024, **i32)
    args = [buf.data_ptr()] * 6
    assert B.moe_permute_static(buf.data_ptr(), 262144 + 1, 4, 4, *args, 0) == B.MOE_ERR_CAPACITY
    assert B.moe_permute_static(buf.data_ptr(), 16, 64, 9, *args, 0) == B.MOE_ERR_CAPACITY     # 576 slots
    assert B.moe_permute_static(buf.data_ptr(), -1, 4, 4, *args, 0) == B.MOE_ERR_INVALID_ARG
    assert B.moe_permute_static(0, 16, 4, 4, *args, 0) == B.MOE_ERR_INVALID_ARG
    # empty input: counts and offsets are all zero
    wl = W.WORKLOADS["tiny"]
    got = _static_permute(wl, torch.empty(0, **i32))
    torch.cuda.synchronize()
    assert int(got["slot_counts"].abs().sum()) == 0 and int(got["slot_offsets"].abs().sum()) == 0
    assert int(got["rank_offsets"].abs().sum()) == 0
