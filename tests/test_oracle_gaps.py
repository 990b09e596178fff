"""Pins of the oracle's gap-coded record (first index of a segment, then the gaps between successive
indices in short fields, the gaps too large for a field in a stream of exceptions), without a GPU.

What fixes it from outside the oracle: two records worked by hand (tests/golden/gap_record_example.txt,
one of them with an exception), an independent Python reader of the packed words, the round trip back
to the plain record word for word, the bit count's closed form, a brute-force search for the best
width, the degenerate cases (all indices consecutive, one entry, no entry), and the saving on indices
that are spread evenly or in clusters.
"""
import os

import numpy as np

from oracle import oracle as O
from paper_1906_02367_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gap_record_example.txt")


def clog2(v):
    return max(1, (int(v) - 1).bit_length())


def read_bits(words, bitpos, width):
    v = 0
    for b in range(width):
        q, o = divmod(bitpos + b, 32)
        v |= ((int(words[q]) >> o) & 1) << b
    return v


def words_for(n, width):
    return (n * width + 31) // 32


def rest_words(plan, n):
    bl = clog2(plan.s)
    if plan.quantizer == O.NONE:
        return n
    if plan.quantizer == O.MINMAX:
        return words_for(n, bl)
    return words_for(n, 1) + (words_for(n, bl) if plan.quantizer in (O.QSGD, O.QSGD_SCALED) else 0)


def python_indices(plan, packed_row):
    """Segment-local indices of every segment, read from the packed words with the format's
    description alone; also the word count and the bit count it implies."""
    sizes = np.diff(plan.offsets)
    at = 5 * plan.nseg
    out, bits = [], 0
    bl = clog2(plan.s)
    for g in range(plan.nseg):
        n = int(plan.kseg[g]) if plan.quantizer == O.MINMAX else int(packed_row[5 * g])
        w, first, x = (int(v) for v in packed_row[5 * g + 2:5 * g + 5])
        bi = clog2(sizes[g])
        gw = words_for(n - 1, w) if n else 0
        idx, taken = [], 0
        for j in range(n):
            if j == 0:
                idx.append(first)
                continue
            gap = read_bits(packed_row[at:], (j - 1) * w, w)
            if w and gap == (1 << w) - 1:                  # the escape: the gap is the next exception
                gap = read_bits(packed_row[at + gw:], taken * bi, bi)
                taken += 1
            idx.append(idx[-1] + gap + 1)
        assert taken == x
        out.append(idx)
        per_entry = {O.NONE: 32, O.MINMAX: bl, O.SIGN_L1: 1, O.SIGN_L2: 1}.get(plan.quantizer, 1 + bl)
        bits += 64 + 6 + (bi + (n - 1) * w + x * bi if n else 0) + n * per_entry
        at += gw + words_for(x, bi) + rest_words(plan, n)
    return out, at, bits


def best_width(gaps, bi):
    """(w, x, cost) by trying every width: the smallest w among the cheapest."""
    best = None
    for w in range(0, bi + 1):
        if w == 0:
            if any(gaps):
                continue
            x = 0
        else:
            x = sum(1 for g in gaps if g >= (1 << w) - 1)
        cost = len(gaps) * w + x * bi
        if best is None or cost < best[2]:
            best = (w, x, cost)
    return best


def plain_indices(plan, wire_row):
    sizes = np.diff(plan.offsets)
    at = 2 * plan.nseg
    out = []
    for g in range(plan.nseg):
        n = int(plan.kseg[g]) if plan.quantizer == O.MINMAX else int(wire_row[2 * g])
        bi = clog2(sizes[g])
        out.append([read_bits(wire_row[at:], j * bi, bi) for j in range(n)])
        at += words_for(n, bi) + rest_words(plan, n)
    return out


def golden():
    rows = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows[key] = vals
    return [(np.array([int(v, 16) for v in rows["plain" + t]], np.uint32),
             np.array([int(v, 16) for v in rows["packed" + t]], np.uint32), int(rows["bits" + t][0])) for t in "12"]


def test_the_records_worked_by_hand():
    for k, (plain, packed, bits) in zip((4, 5), golden()):
        plan = O.Plan(1, 32, k=k, s=1, quantizer=O.SIGN_L1)
        assert plan.wire_words() == 4 and O.gap_words(plan) == 5 + 1 + 1 + 1      # header, (k - 1) b_idx <= 20 bits, the spare word, signs
        out = O.recode_gaps(plan, plain[None, :])
        assert out["rc"] == 0
        row = list(out["packed"][0])
        assert row[:len(packed)] == list(packed) and not any(row[len(packed):]) and int(out["bits"][0]) == bits
        back = O.decode_gaps(plan, out["packed"])
        assert back["rc"] == 0 and list(back["wire"][0]) == list(plain)


def test_round_trip_reader_and_bit_count_for_every_quantizer():
    R = 3
    sizes = [700, 1, 64, 3000]
    off = I.segments_from_sizes(sizes)
    kseg = np.array([40, 1, 64, 7], np.int64)                  # (a segment kept whole: all gaps 0; a single entry)
    d = int(off[-1])
    for qz, s in ((O.QSGD, 4), (O.QSGD_SCALED, 2), (O.SIGN_L1, 1), (O.SIGN_L2, 1), (O.NONE, 1), (O.MINMAX, 8)):
        for sp in (O.TOPK, O.RANDK):
            x, xw, mem = I.gaussian_round(R, d, seed=61)
            plan = O.Plan(R, d, s=s, sparsifier=sp, quantizer=qz, seed=5, offsets=off, kseg=kseg)
            cf = O.compress_feedback(plan, 2, x, xw, mem.copy(), details=True)
            assert cf["rc"] == 0
            mask = np.array([1, 0, 1], np.uint8)
            out = O.recode_gaps(plan, cf["wire"], mask=mask)
            assert out["rc"] == 0 and not out["packed"][1].any()              # a masked worker's row is not written
            for r in (0, 2):
                got, words, bits = python_indices(plan, out["packed"][r])
                assert got == plain_indices(plan, cf["wire"][r])
                assert all(a < b for seg in got for a, b in zip(seg, seg[1:]))
                assert words <= out["stride"] and not out["packed"][r, words:].any()
                assert bits == int(out["bits"][r])
                for g, seg in enumerate(got):                                  # the width is the cheapest one
                    if len(seg) >= 2:
                        w, x, _ = best_width([b - a - 1 for a, b in zip(seg, seg[1:])], clog2(sizes[g]))
                        assert (int(out["packed"][r, 5 * g + 2]), int(out["packed"][r, 5 * g + 4])) == (w, x)
                if qz not in (O.QSGD, O.QSGD_SCALED):                          # (QSGD drops its level-0 entries)
                    assert int(out["packed"][r, 5 * 2 + 2]) == 0                # the whole segment: width 0, no gap words
            back = O.decode_gaps(plan, out["packed"], mask=mask)
            assert back["rc"] == 0
            assert np.array_equal(back["wire"][[0, 2]], cf["wire"][[0, 2]]) and not back["wire"][1].any()


def test_a_segment_that_sends_nothing_or_one_entry():
    # QSGD may drop every kept entry of a segment (level 0): n = 0; written by hand in the plain format
    plan = O.Plan(1, 48, s=4, quantizer=O.QSGD, offsets=np.array([0, 16, 48], np.int64), kseg=np.array([2, 3], np.int64))
    wire = np.zeros((1, plan.wire_words()), np.uint32)
    wire[0, 0], wire[0, 1] = 0, np.float32(2.0).view(np.uint32)                # segment 0: nothing sent
    wire[0, 2], wire[0, 3] = 1, np.float32(0.5).view(np.uint32)                # segment 1: one entry, index 17
    wire[0, 4], wire[0, 5], wire[0, 6] = 17, 1, 2                              # index, sign, level - 1
    out = O.recode_gaps(plan, wire)
    assert out["rc"] == 0
    assert list(out["packed"][0][:10]) == [0, wire[0, 1], 0, 0, 0, 1, wire[0, 3], 0, 17, 0]
    assert list(out["packed"][0][10:12]) == [1, 2] and not out["packed"][0][12:].any()
    assert int(out["bits"][0]) == (64 + 6) + (64 + 6 + 5 + 1 * (1 + 2))
    assert np.array_equal(O.decode_gaps(plan, out["packed"])["wire"], wire)


def test_spread_and_clustered_indices_cost_fewer_bits():
    R, d, k = 2, 200_000, 200
    x, xw, mem = I.gaussian_round(R, d, seed=62)
    bi = clog2(d)                                                              # 18 bits an index in the plain record
    for sp in (O.TOPK, O.RANDK):
        plan = O.Plan(R, d, k=k, s=1, sparsifier=sp, quantizer=O.SIGN_L1, seed=9)
        cf = O.compress_feedback(plan, 0, x, xw, mem.copy(), details=True)
        out = O.recode_gaps(plan, cf["wire"])
        for r in range(R):
            idx = plain_indices(plan, cf["wire"][r])[0]
            w, xc, cost = best_width([b - a - 1 for a, b in zip(idx, idx[1:])], bi)
            assert (int(out["packed"][r, 2]), int(out["packed"][r, 4])) == (w, xc)
            assert int(out["bits"][r]) == 64 + 6 + bi + cost + k
            assert int(cf["bits"][r]) == 64 + k * (bi + 1)
            # gaps of k points spread over d: mean d / k = 1000, so about 11 bits a gap and a few exceptions
            assert 9 <= w <= 13 and int(out["bits"][r]) < 0.8 * int(cf["bits"][r])
        # never more than 6 bits a segment above the plain record: the widest field has no exceptions
        assert all(int(b) <= int(a) + 6 for a, b in zip(cf["bits"], out["bits"]))
    # clusters far apart (kept coordinates of a few tensors of large scale): the long gaps become exceptions
    plan = O.Plan(1, d, k=k, s=1, quantizer=O.SIGN_L1)
    xw1 = np.zeros((1, d), np.float32)
    hot = np.concatenate([np.arange(1000, 1400, 4), np.arange(150_000, 150_400, 4)])
    xw1[0, hot] = 1.0 + np.arange(hot.size, dtype=np.float32)
    cf = O.compress_feedback(plan, 0, np.zeros(d, np.float32), -xw1, np.zeros((1, d), np.float32), details=True)
    assert plain_indices(plan, cf["wire"][0])[0] == sorted(hot.tolist())
    out = O.recode_gaps(plan, cf["wire"])
    assert (int(out["packed"][0, 2]), int(out["packed"][0, 4])) == (3, 1)      # gaps of 3 in fields of 3 bits (escape 7), one exception
    assert int(out["bits"][0]) == 64 + 6 + bi + 199 * 3 + 1 * bi + k
