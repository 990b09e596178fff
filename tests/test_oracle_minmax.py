"""Pins of the oracle's stochastic s-level quantizer between the smallest and the largest kept entry
(Section 2.1, Definition 1, example 2), without a GPU.

What fixes it from outside the oracle: unbiasedness and the error bound k / (2 (s-1)^2) ||v||^2 of
Definition 1 / the cited mean-estimation quantizer, levels inside [min, max], the two end points
(no randomness there), k = 1 (the entry itself), many levels (close to the identity), the empirical
probability of rounding up, and an independent Python reader of the record.
"""
import math

import numpy as np

from oracle import oracle as O
from paper_1906_02367_b200 import inputs as I


def clog2(v):
    return max(1, (int(v) - 1).bit_length())


def read_bits(words, bitpos, width):
    v = 0
    for b in range(width):
        q, o = divmod(bitpos + b, 32)
        v |= ((int(words[q]) >> o) & 1) << b
    return v


def details(plan, rnd, x, xw, mem):
    m = mem.copy()
    out = O.compress_feedback(plan, rnd, x, xw, m, details=True)
    assert out["rc"] == 0
    u = mem + (x[None, :] - xw)
    return out, u, m


def python_values(plan, row, k, d):
    """(indices, values) of a one-segment record, read with nothing but the format's description:
    header pair (min, max), k indices of ceil(log2 d) bits, k level fields of ceil(log2 s) bits."""
    lo, hi = row[0:1].view(np.float32)[0], row[1:2].view(np.float32)[0]
    bi, bl = clog2(d), clog2(plan.s)
    wi = -(-k * bi // 32)
    idx = [read_bits(row[2:], j * bi, bi) for j in range(k)]
    lev = [read_bits(row[2 + wi:], j * bl, bl) for j in range(k)]
    D = np.float32(np.float32(hi - lo) / np.float32(plan.s - 1))
    vals = [np.float32(lo + np.float32(np.float32(j) * D)) for j in lev]
    return lo, hi, idx, lev, np.array(vals, np.float32)


def test_levels_lie_between_min_and_max_and_the_record_decodes():
    R, d, k, s = 2, 300, 37, 8
    x, xw, mem = I.gaussian_round(R, d, seed=51)
    plan = O.Plan(R, d, k=k, s=s, quantizer=O.MINMAX, seed=3)
    out, u, m = details(plan, 4, x, xw, mem)
    for r in range(R):
        sel = out["sel"][r]
        v = u[r, sel]
        lo, hi, idx, lev, vals = python_values(plan, out["wire"][r], k, d)
        assert lo == v.min() and hi == v.max()
        assert idx == list(sel) and idx == sorted(idx)
        assert list(np.array(lev) + 1) == list(out["level"][r]) and min(lev) >= 0 and max(lev) <= s - 1
        # each value is one of the two levels that bracket the entry
        D = (float(hi) - float(lo)) / (s - 1)
        assert np.all(np.abs(vals.astype(np.float64) - v.astype(np.float64)) <= D * (1 + 1e-5))
        assert np.all(vals >= lo) and np.all(vals <= np.float32(hi) + np.float32(abs(hi)) * np.float32(1e-6))
        # memory: m = u - g on the kept set, m = u elsewhere
        want = u[r].copy()
        want[sel] = v - vals
        assert np.array_equal(m[r].view(np.uint32), want.view(np.uint32))
        assert out["bits"][r] == 64 + k * (clog2(d) + clog2(s)) and out["n"][r, 0] == k
        # the master reads the same values back
        acc = np.zeros(d, np.float32)
        assert O.unpack_accumulate(O.Plan(1, d, k=k, s=s, quantizer=O.MINMAX), acc, out["wire"][r:r + 1]) == 0
        assert np.array_equal(-acc[sel], vals) and np.count_nonzero(acc) == np.count_nonzero(vals)      # x = 0 - g / 1


def test_end_points_and_single_entry_carry_no_randomness():
    for w in (0, 1 << 31, 0xFFFFFFFF):
        assert O.minmax_level(-2.0, -2.0, 3.0, 6, w) == 1           # the smallest entry: level 1 = min
        assert O.minmax_level(3.0, -2.0, 3.0, 6, w) == 6            # the largest: level s = max
        assert O.minmax_level(1.5, 1.5, 1.5, 6, w) == 1             # min = max: one level
    assert O.value_minmax(-2.0, 3.0, 6, 1) == -2.0 and O.value_minmax(-2.0, 3.0, 6, 6) == 3.0
    # k = 1: the kept entry is its own minimum and maximum, g = u and the memory becomes 0
    R, d = 2, 50
    x, xw, mem = I.gaussian_round(R, d, seed=52)
    out, u, m = details(O.Plan(R, d, k=1, s=4, quantizer=O.MINMAX, seed=1), 0, x, xw, mem)
    for r in range(R):
        i = int(out["sel"][r, 0])
        assert i == int(np.argmax(np.abs(u[r]))) and m[r, i] == 0.0 and out["level"][r, 0] == 1


def test_unbiased_with_the_error_bound_of_definition_1():
    R, d, k, s, T = 1, 64, 12, 5, 4000
    x, xw, mem = I.gaussian_round(R, d, seed=53)
    plan = O.Plan(R, d, k=k, s=s, quantizer=O.MINMAX, seed=9)
    mean, err2 = np.zeros(k), 0.0
    for t in range(T):
        out, u, _ = details(plan, t, x, xw, mem)
        sel = out["sel"][0]
        v = u[0, sel].astype(np.float64)
        _, _, _, _, vals = python_values(plan, out["wire"][0], k, d)
        q = vals.astype(np.float64)
        mean += q / T
        err2 += float((q - v) @ (q - v)) / T
    D = (v.max() - v.min()) / (s - 1)
    assert np.allclose(mean, v, atol=5 * D / 2 / math.sqrt(T) + 1e-7)       # E[Q(v)] = v
    assert err2 <= k / (2 * (s - 1) ** 2) * float(v @ v) * 1.02             # E||Q(v) - v||^2 <= beta ||v||^2
    assert err2 <= k * D * D / 4 * 1.02                                     # each entry: at most D^2 / 4


def test_probability_of_rounding_up_is_the_fraction():
    s, T = 5, 6000                                   # levels 0, 1, 2, 3, 4 between lo = 0 and hi = 4
    f = 0.3
    ups = sum(O.minmax_level(2.0 + f, 0.0, 4.0, s, int(w)) == 4 for w in np.random.default_rng(1).integers(0, 2**32, T))
    frac = float(np.float32(np.float32(2.3) / np.float32(1.0)) - 2)
    assert abs(ups / T - frac) < 5 * math.sqrt(frac * (1 - frac) / T)
    assert all(O.minmax_level(2.3, 0.0, 4.0, s, int(w)) in (3, 4) for w in (0, 123456789, 0xFFFFFFFF))


def test_many_levels_approach_the_identity_and_segments_are_quantized_apart():
    R = 2
    sizes = [40, 1, 500]
    off = I.segments_from_sizes(sizes)
    kseg = np.array([6, 1, 30], np.int64)
    d = int(off[-1])
    x, xw, mem = I.gaussian_round(R, d, seed=54)
    plan = O.Plan(R, d, s=65535, quantizer=O.MINMAX, seed=2, offsets=off, kseg=kseg)
    out, u, m = details(plan, 1, x, xw, mem)
    for r in range(R):
        pos = 0
        for g, k in enumerate(kseg):
            sel = out["sel"][r, pos:pos + k]
            v = u[r, sel]
            lo = out["wire"][r, 2 * g:2 * g + 1].view(np.float32)[0]
            hi = out["wire"][r, 2 * g + 1:2 * g + 2].view(np.float32)[0]
            assert lo == v.min() and hi == v.max()                # Corollary 1: each piece has its own range
            assert np.all(np.abs(m[r, sel]) <= (float(hi) - float(lo)) / 65534 * 1.001 + 1e-12)
            pos += k
    assert plan.wire_words() == 2 * 3 + sum(-(-int(k) * clog2(n) // 32) + -(-int(k) * 16 // 32) for k, n in zip(kseg, sizes))
