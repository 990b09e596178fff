"""The allocation-free master update (qs_unpack_accumulate_static) against the regular one and the oracle.

Some users of the library may not allocate device memory at the moment the update runs (their
memory is handed out once by another component, or an allocation would stall the device in the
middle of a serving loop), so that entry point keeps its scratch in a fixed array inside the
library.  This file checks, through the C boundary, that it changes x exactly as
qs_unpack_accumulate and the CPU oracle's master update do, twice in a row on the same array (the
second call meets whatever the first one left behind), that the call leaves the amount of free
device memory as it found it, and that it refuses what it cannot take: sizes its array cannot
hold, and the plain sparsifier (32-bit values in the record), which it does not decode.  It is collected last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_1906_02367_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("quantizer,s", [(0, 16), (1, 4), (2, 1), (4, 1)])
def test_static_update_matches_the_regular_one_twice(quantizer, s):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1906_02367_b200 import binding as B
    R, d, k = 6, 200003, 1500
    x, xw, mem = I.gaussian_round(R, d, seed=41)
    xw[3] = xw[1]                       # two identical workers: their indices collide
    mem[3] = mem[1]
    gx, gxw, gmem = (torch.from_numpy(a.copy()).cuda() for a in (x, xw, mem))
    ctx = B.Context(R, d, k, s, B.QS_TOPK, quantizer, seed=5)
    ctx.bind(gx, gxw, gmem)
    wire = ctx.new_wire()
    masks = [None, np.array([1, 0, 1, 1, 0, 1], np.uint8)]
    for rnd, mask in enumerate(masks):
        gxw.add_(torch.from_numpy(I.gaussian_drift(R, d, 3, rnd, std=1e-2)).cuda())
        ctx.compress_feedback(rnd, mask)
        ctx.pack(wire)
        x_static = gx.clone()
        x_oracle = gx.cpu().numpy().copy()
        ctx.unpack_accumulate(wire, mask)                              # regular entry point
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = B.unpack_accumulate_static(R, d, k, s, quantizer, x_static, wire, mask)
        assert rc == 0
        assert ctx.sync_status() == 0, ctx.last_error()
        torch.cuda.synchronize()
        if rnd:                                                        # (the first call on a device may load the module)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call must not allocate device memory"
        assert np.array_equal(_bits(x_static), _bits(gx)), f"call {rnd}"
        # the oracle's master update on the same records
        plan = O.Plan(R, d, k=k, s=s, quantizer=quantizer, seed=5)
        assert O.unpack_accumulate(plan, x_oracle, wire.cpu().numpy().view(np.uint32), mask=mask) == 0
        assert np.array_equal(_bits(x_static), x_oracle.view(np.uint32)), f"call {rnd} against the oracle"
        assert not np.array_equal(_bits(gx), x.view(np.uint32))        # the update did something
        ctx.broadcast(mask)
    ctx.destroy()


def test_static_update_rejects_what_it_cannot_hold():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1906_02367_b200 import binding as B
    x = torch.zeros(16, device="cuda")
    wire = torch.zeros((2, 64), dtype=torch.int32, device="cuda")
    assert B.unpack_accumulate_static(2, B.QS_STATIC_MAX_D + 1, 4, 16, 0, x, wire) == B.QS_TOO_LARGE
    assert B.unpack_accumulate_static(2, 16, 17, 16, 0, x, wire) == B.QS_INVALID_ARG
    assert B.unpack_accumulate_static(33, 16, 4, 16, 0, x, wire) == B.QS_INVALID_ARG
    assert B.unpack_accumulate_static(2, 16, 4, 16, B.QS_NONE, x, wire) == B.QS_INVALID_ARG   # values in the record: not decoded here
    small = torch.zeros((2, 3), dtype=torch.int32, device="cuda")
    assert B.unpack_accumulate_static(2, 16, 4, 16, 0, x, small) == B.QS_CAPACITY
    assert B.unpack_accumulate_static(2, 16, 4, 16, 0, x, wire) == 0   # empty records: nothing to add
    torch.cuda.synchronize()
    assert float(x.abs().sum()) == 0.0
