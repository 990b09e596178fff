"""Gap-coded records on the GPU (qs_recode_gaps / qs_decode_gaps through the C boundary) against the
oracle's, word for word: the packed rows, their bit counts, and the plain rows they decode back to.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_1906_02367_b200 import inputs as I

import test_gpu_parity as T

pytestmark = pytest.mark.gpu


def setup_module(module):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1906_02367_b200 import binding
    T.B = binding


def both_ways(p, out, mask=None):
    """p: a Pair whose GPU wire holds the records of `out` (the oracle's round)."""
    R = p.plan.R
    dev = p.wire.device
    want = O.recode_gaps(p.plan, out["wire"], mask=mask)
    assert want["rc"] == 0
    assert p.ctx.gap_words() == want["stride"] == O.gap_words(p.plan)
    packed = torch.full((R, want["stride"] + 3), -1, dtype=torch.int32, device=dev)      # stale words, a wider stride
    bits = torch.zeros(R, dtype=torch.int64, device=dev)
    p.ctx.recode_gaps(p.wire, packed, mask, bits)
    assert p.ctx.sync_status() == 0, p.ctx.last_error()
    got = packed.cpu().numpy().view(np.uint32)
    act = [r for r in range(R) if mask is None or mask[r]]
    for r in act:
        assert np.array_equal(got[r, :want["stride"]], want["packed"][r]), f"packed record, worker {r}"
        assert int(bits[r]) == int(want["bits"][r])
    for r in set(range(R)) - set(act):
        assert np.all(got[r] == 0xFFFFFFFF)                                             # not written
    back = torch.full_like(p.wire, -1)
    p.ctx.decode_gaps(packed, back, mask)
    assert p.ctx.sync_status() == 0, p.ctx.last_error()
    b = back.cpu().numpy().view(np.uint32)
    w = p.wire.cpu().numpy().view(np.uint32)
    for r in act:
        assert np.array_equal(b[r], w[r]) and np.array_equal(b[r], out["wire"][r]), f"decoded record, worker {r}"
    # the oracle's decoder agrees on what the GPU packed
    assert np.array_equal(O.decode_gaps(p.plan, got[:, :want["stride"]], mask=mask)["wire"][act], out["wire"][act])
    return want


@pytest.mark.parametrize("qz,s", [(O.QSGD, 4), (O.QSGD_SCALED, 2), (O.SIGN_L1, 1), (O.SIGN_L2, 1), (O.NONE, 1), (O.MINMAX, 8)])
@pytest.mark.parametrize("sp", [O.TOPK, O.RANDK])
def test_segments_of_every_kind(qz, s, sp):
    # a segment kept whole (all gaps 0), a single coordinate, one entry of many, ragged sizes, a masked worker
    R = 3
    sizes = [700, 1, 64, 3000, 5]
    off = I.segments_from_sizes(sizes)
    kseg = np.array([40, 1, 64, 7, 2], np.int64)
    d = int(off[-1])
    x, xw, mem = I.gaussian_round(R, d, seed=71)
    p = T.Pair(R, d, s=s, sparsifier=sp, quantizer=qz, seed=5, offsets=off, kseg=kseg, x=x, xw=xw, mem=mem)
    mask = np.array([1, 0, 1], np.uint8)
    out = p.round_fused(3, mask)
    both_ways(p, out, mask)
    out = p.round_split(4)
    both_ways(p, out)
    p.close()


@pytest.mark.parametrize("d,k", [(1, 1), (33, 33), (4097, 1), (300_000, 5000), (1 << 20, 70_000)])
def test_one_segment_from_one_entry_to_many_chunks(d, k):
    R = 2
    x, xw, mem = I.gaussian_round(R, d, seed=72)
    for qz, s in ((O.SIGN_L1, 1), (O.QSGD, 16)):
        p = T.Pair(R, d, k=k, s=s, quantizer=qz, seed=1, x=x, xw=xw, mem=mem)
        out = p.round_fused(0)
        want = both_ways(p, out)
        if k >= 5000 and qz == O.SIGN_L1:                 # indices spread over d: well under the plain record
            assert all(int(b) < 0.9 * int(a) for a, b in zip(out["bits"], want["bits"]))
        p.close()


def test_resnet50_shape_flat_and_per_tensor_full_size():
    sizes = I.resnet50_tensor_sizes()
    off = I.segments_from_sizes(sizes)
    d, R = int(off[-1]), 8
    scales = I.tensor_scales(len(sizes), seed=0)
    x = I.model_init(d, seed=0)
    for kw in (dict(k=I.k_from_ratio(d, 1, 1000)), dict(offsets=off, kseg=I.k_per_tensor_capped(sizes, 1000))):
        p = T.Pair(R, d, s=1, quantizer=O.SIGN_L1, seed=3, x=x, xw=np.broadcast_to(x, (R, d)).copy(),
                   mem=np.zeros((R, d), np.float32), **kw)
        p.drift(I.laplace_drift(R, off, scales, 0, 0))
        out = O.sync_round(p.plan, 0, p.x, p.xw, p.mem, nthreads=8)
        p.ctx.sync_round(p.wire, 0, None, p.gbits)
        want = both_ways(p, out)
        plain, gap = int(out["bits"].sum()), int(want["bits"].sum())
        assert gap < plain
        p.close()
