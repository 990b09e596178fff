"""Pins of the CPU oracle against what the paper and the mathematics fix.

Every check here compares oracle/qs_oracle.cpp with something that is not the oracle:
published known-answer vectors, brute force in Python on tiny inputs, exact rational
arithmetic, closed forms and inequalities from the paper.  No GPU is needed.
"""
import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as O
from paper_1906_02367_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_bits(v):
    return struct.unpack("<I", struct.pack("<f", float(v)))[0]


def abs_key(v):
    return f32_bits(v) & 0x7FFFFFFF


# ----------------------------------------------------------------------------- Philox
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) >= 2
    for row in rows:
        v = [int(h, 16) for h in row]
        out = O.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]


def test_philox_word_keying():
    # counter = (element >> 2, worker, round_lo, (round_hi << 8) | stream), key = seed halves
    cases = [(0, 0, 0, 0, 0), (0x1234567890ABCDEF, 7, 3, 1001, 1), (5, (3 << 32) | 9, 15, 2**33 + 6, 0)]
    for seed, rnd, worker, el, stream in cases:
        ctr = [(el >> 2) & 0xFFFFFFFF, worker, rnd & 0xFFFFFFFF, (((rnd >> 32) << 8) | stream) & 0xFFFFFFFF]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        assert O.philox_word(seed, rnd, worker, el, stream) == int(O.philox4x32_10(ctr, key)[el & 3])
    # the four words of one block serve four consecutive elements
    blk = O.philox4x32_10([10, 2, 5, 0], [99, 0])
    assert [O.philox_word(99, 5, 2, 40 + j, 0) for j in range(4)] == [int(b) for b in blk]


def test_philox_words_look_uniform():
    w = np.array([O.philox_word(1, 0, 0, i, 1) for i in range(20000)], dtype=np.float64) / 2**32
    assert abs(w.mean() - 0.5) < 0.01 and abs(w.var() - 1 / 12) < 0.005


# ----------------------------------------------------------------------------- Top_k
def brute_topk(u, k):
    order = sorted(range(len(u)), key=lambda i: (-abs_key(u[i]), i))
    return sorted(order[:k])


CRAFTED = [
    ([3.0, -3.0, 3.0, 1.0, -3.0], 2),            # ties on the threshold: lower index wins
    ([0.0, -0.0, 0.0, 0.0], 2),                  # all zero, +0 and -0 are one key
    ([1.0] * 9, 4),                              # all equal
    ([1e-45, -1e-45, 2e-45, 0.0], 2),            # subnormals
    ([5.0, 4.0, -6.0, 0.5], 1),                  # k = 1
    ([5.0, 4.0, -6.0, 0.5], 4),                  # k = d
    ([2.0, -7.0, 7.0, 7.0, -7.0, 1.0, 7.0], 3),  # more ties than slots
    ([-1.5], 1),                                 # d = 1
]


@pytest.mark.parametrize("vals,k", CRAFTED)
def test_topk_crafted(vals, k):
    u = np.array(vals, dtype=np.float32)
    for mode in (O.SORT, O.NTH):
        assert list(O.select_topk(u, k, mode)) == brute_topk(u, k)


def test_topk_random_bruteforce_and_nth():
    g = np.random.default_rng(3)
    for n, k in [(31, 5), (32, 32), (33, 1), (257, 40), (1000, 10)]:
        u = g.standard_normal(n).astype(np.float32)
        u[g.integers(0, n, n // 4)] = np.float32(0.75)  # plant ties
        want = brute_topk(u, k)
        assert list(O.select_topk(u, k, O.SORT)) == want
        assert list(O.select_topk(u, k, O.NTH)) == want
    u = g.standard_normal(60000).astype(np.float32)
    u[::7] = np.float32(-2.0)
    for k in (1, 600, 9000):
        a, b = O.select_topk(u, k, O.SORT), O.select_topk(u, k, O.NTH)
        assert np.array_equal(a, b)
        keys = np.abs(u).view(np.uint32)
        rest = np.setdiff1d(np.arange(u.size), a)
        assert keys[rest].max() <= keys[a].min()   # Section 2.2: the k largest in magnitude


# ----------------------------------------------------------------------------- Rand_k
def test_randk_enumeration():
    seed, rnd, worker, lo, n, k = 11, 4, 2, 37, 200, 17
    h = [(O.philox_word(seed, rnd, worker, lo + i, 1), i) for i in range(n)]
    want = sorted(i for _, i in sorted(h)[:k])
    for mode in (O.SORT, O.NTH):
        assert list(O.select_randk(seed, rnd, worker, lo, n, k, mode)) == want


def test_randk_inclusion_probability():
    # proof of Lemma 8: each coordinate is in the random k-subset with probability k/d
    n, k, rounds = 40, 10, 3000
    hits = np.zeros(n)
    for t in range(rounds):
        hits[O.select_randk(5, t, 0, 0, n, k)] += 1
    p = k / n
    sd = math.sqrt(p * (1 - p) / rounds)
    assert np.all(np.abs(hits / rounds - p) < 5 * sd)
    # independent across workers and rounds
    assert list(O.select_randk(5, 1, 0, 0, n, k)) != list(O.select_randk(5, 1, 1, 0, n, k))


# ----------------------------------------------------------------------------- norms
def exact_l2(v):
    s = sum(Fraction(float(a)) ** 2 for a in v)
    return np.float32(math.sqrt(float(s)))     # Fraction -> float is correctly rounded


def exact_l1(v):
    return np.float32(float(sum(abs(Fraction(float(a))) for a in v)))


def test_norms_exact_rational():
    g = np.random.default_rng(5)
    cases = [np.array([3.0, 4.0], np.float32), np.array([1e-30, 1e30, -1e-30], np.float32),
             np.array([1e-45, 1e-45, -3e-45], np.float32), np.array([3.4e38, 3.4e38], np.float32) * 0.5,
             np.array([1.0] + [2.0 ** -24] * 7, np.float32),
             (g.standard_normal(500) * 10.0 ** g.integers(-20, 15, 500)).astype(np.float32),
             g.standard_normal(4097).astype(np.float32), np.zeros(5, np.float32)]
    for v in cases:
        assert O.norm_l2(v) == exact_l2(v), v[:4]
        assert O.norm_l1(v) == exact_l1(v), v[:4]
    for a in (1.5, -2.25e-12, 7e20, 1e-45):       # k = 1: the norm is |u| itself
        v = np.array([a], np.float32)
        assert O.norm_l2(v) == abs(v[0]) and O.norm_l1(v) == abs(v[0])


def test_norm_is_order_independent_where_fp64_is_not():
    v = np.array([1e19, 1.0, -1e19, 1.0] * 50 + [3e-10] * 9, np.float32)
    g = np.random.default_rng(1)
    want = exact_l1(v)
    for _ in range(5):
        assert O.norm_l1(g.permutation(v)) == want
        assert O.norm_l2(g.permutation(v)) == exact_l2(v)


# ----------------------------------------------------------------------------- QSGD level
def test_qsgd_level_rule():
    g = np.random.default_rng(7)
    for _ in range(2000):
        s = int(g.choice([1, 2, 3, 4, 15, 16, 256, 65535]))
        N = np.float32(abs(g.standard_normal()) + 0.1)
        u = np.float32(g.uniform(-1, 1)) * N
        w = int(g.integers(0, 2**32))
        p = np.float32(np.float32(abs(u)) * np.float32(s)) / N
        lo = int(np.floor(p))
        f = float(np.float32(p - np.float32(lo)))
        U = (w >> 8) / 2**24
        want = min(lo + (1 if U < f else 0), s)
        assert O.qsgd_level(float(u), float(N), s, w) == want
        assert O.qsgd_level(float(u), float(N), s, 0) == min(lo + (1 if f > 0 else 0), s)
    assert O.qsgd_level(1.0, 0.0, 16, 123) == 0             # zero norm: nothing to send
    assert O.qsgd_level(2.0, 2.0, 16, 0xFFFFFFFF) == 16     # |u| = N sits on the top level


def test_beta_formula():
    # Section 2.1, example 1: beta_{d,s} = min(d/s^2, sqrt(d)/s)
    for k, s in [(655, 16), (100, 16), (40, 3), (1, 1), (99400, 15)]:
        assert O.beta_qsgd(k, s) == pytest.approx(min(k / s**2, math.sqrt(k) / s), rel=1e-15)


# ----------------------------------------------------------------------------- a round
def run_details(plan, rnd, x, xw, mem, **kw):
    mem2 = mem.copy()
    out = O.compress_feedback(plan, rnd, x, xw, mem2, details=True, **kw)
    assert out["rc"] == 0
    u = (mem + (x[None, :] - xw)).astype(np.float32) if kw.get("anchors") is None else \
        (mem + (kw["anchors"] - xw)).astype(np.float32)
    return out, u, mem2


def values_from_details(plan, out, r):
    """g on the kept coordinates rebuilt in numpy fp32 from (norm, level, sign)."""
    g = np.zeros(plan.K, np.float32)
    pos = 0
    for sg in range(plan.nseg):
        k = int(plan.kseg[sg])
        N = out["norm"][r, sg]
        lv = out["level"][r, pos:pos + k].astype(np.float32)
        if plan.quantizer in (O.SIGN_L1, O.SIGN_L2):
            mag = np.full(k, N / np.float32(k), np.float32)
        else:
            mag = (N * lv) / np.float32(plan.s)
            if plan.quantizer == O.QSGD_SCALED:
                c = np.float32(1.0 / (1.0 + min(k / plan.s**2, math.sqrt(k) / plan.s)))
                mag = (mag * c).astype(np.float32)
        g[pos:pos + k] = np.where(out["sign"][r, pos:pos + k] == 1, -mag, mag)
        pos += k
    return g


def test_k1_reduces_to_identity_on_the_kept_coordinate():
    # with one kept coordinate the norm is |u|, the level is s and g = u: memory becomes 0
    x, xw, mem = I.gaussian_round(3, 50, seed=2)
    for s in (1, 4, 16):
        plan = O.Plan(3, 50, k=1, s=s, quantizer=O.QSGD, seed=8)
        out, u, mem2 = run_details(plan, 0, x, xw, mem)
        for r in range(3):
            i = int(out["sel"][r, 0])
            assert i == int(np.argmax(np.abs(u[r])))
            assert out["level"][r, 0] == s and out["norm"][r, 0] == abs(u[r, i])
            assert mem2[r, i] == 0.0
            rest = np.arange(50) != i
            assert np.array_equal(mem2[r, rest].view(np.uint32), u[r, rest].view(np.uint32))


@pytest.mark.parametrize("quantizer", [O.QSGD, O.QSGD_SCALED, O.SIGN_L1])
@pytest.mark.parametrize("sparsifier", [O.TOPK, O.RANDK])
def test_round_pieces_against_python(quantizer, sparsifier):
    R, d, k, s = 3, 700, 23, 16
    x, xw, mem = I.gaussian_round(R, d, seed=4)
    plan = O.Plan(R, d, k=k, s=s, sparsifier=sparsifier, quantizer=quantizer, seed=21)
    out, u, mem2 = run_details(plan, 6, x, xw, mem)
    for r in range(R):
        sel = out["sel"][r]
        if sparsifier == O.TOPK:
            assert list(sel) == brute_topk(u[r], k)
        else:
            h = sorted((O.philox_word(21, 6, r, i, 1), i) for i in range(d))
            assert list(sel) == sorted(i for _, i in h[:k])
        kept = u[r, sel]
        N = out["norm"][r, 0]
        assert N == (exact_l1(kept) if quantizer == O.SIGN_L1 else exact_l2(kept))
        assert np.array_equal(out["sign"][r], (kept < 0).astype(np.uint8))   # Definition 2
        if quantizer != O.SIGN_L1:
            for j, i in enumerate(sel):
                w = O.philox_word(21, 6, r, int(i), 0)
                p = np.float32(np.float32(abs(kept[j])) * np.float32(s)) / N
                assert out["level"][r, j] in (int(np.floor(p)), min(int(np.floor(p)) + 1, s))
                assert out["level"][r, j] == O.qsgd_level(float(kept[j]), float(N), s, w)
            assert out["n"][r, 0] == int((out["level"][r] > 0).sum()) <= k   # ||C||_0 <= k
        else:
            assert out["n"][r, 0] == k
        g = values_from_details(plan, out, r)
        if quantizer != O.SIGN_L1:
            g[out["level"][r] == 0] = 0.0
        # memory: m <- u - g on the kept set, m <- u elsewhere
        want = u[r].copy()
        want[sel] = (kept - g).astype(np.float32)
        assert np.array_equal(mem2[r].view(np.uint32), want.view(np.uint32))
        err = np.abs(kept.astype(np.float64) - g.astype(np.float64) - mem2[r, sel].astype(np.float64))
        assert np.all(err <= 0.5 * np.spacing(np.abs(mem2[r, sel])).astype(np.float64) + 1e-300)


def test_scaled_operator_is_the_unscaled_one_times_c():
    R, d, k, s = 2, 400, 30, 4
    x, xw, mem = I.gaussian_round(R, d, seed=6)
    a, u, _ = run_details(O.Plan(R, d, k=k, s=s, quantizer=O.QSGD, seed=3), 1, x, xw, mem)
    b, _, _ = run_details(O.Plan(R, d, k=k, s=s, quantizer=O.QSGD_SCALED, seed=3), 1, x, xw, mem)
    assert np.array_equal(a["sel"], b["sel"]) and np.array_equal(a["level"], b["level"])
    assert np.array_equal(a["wire"], b["wire"])      # same record; the scale is applied at decode
    beta = min(k / s**2, math.sqrt(k) / s)
    assert beta > 1                                  # outside Lemma 1's regime, inside Lemma 2's
    c = np.float32(1.0 / (1.0 + beta))
    xa, xb = np.zeros(d, np.float32), np.zeros(d, np.float32)   # x = 0: the update is -g exactly
    O.unpack_accumulate(O.Plan(1, d, k=k, s=s, quantizer=O.QSGD), xa, a["wire"][:1])
    O.unpack_accumulate(O.Plan(1, d, k=k, s=s, quantizer=O.QSGD_SCALED), xb, b["wire"][:1])
    ga, gb = -xa.astype(np.float64), -xb.astype(np.float64)
    nz = ga != 0
    assert nz.sum() > 0 and np.allclose(gb[nz] / ga[nz], float(c), rtol=2e-7)


# ----------------------------------------------------------------------------- statistics
def decode_dense(plan, out, r):
    dense = np.zeros(plan.d, np.float64)
    g = values_from_details(plan, out, r).astype(np.float64)
    if plan.quantizer not in (O.SIGN_L1, O.SIGN_L2):
        g[out["level"][r] == 0] = 0.0
    dense[out["sel"][r]] = g
    return dense


def test_qsgd_unbiased_and_second_moment():
    # Definition 1: E[Q(v)] = v and E||Q(v)||^2 <= (1 + beta_{k,s}) ||v||^2 on the kept k-vector
    R, d, k, s, T = 1, 64, 12, 4, 4000
    x, xw, mem = I.gaussian_round(R, d, seed=9)
    plan = O.Plan(R, d, k=k, s=s, quantizer=O.QSGD, seed=77)
    mean = np.zeros(d)
    m2 = 0.0
    for t in range(T):
        out, u, _ = run_details(plan, t, x, xw, mem)
        q = decode_dense(plan, out, 0)
        mean += q / T
        m2 += float(q @ q) / T
    sel = out["sel"][0]
    v = u[0, sel].astype(np.float64)
    N = float(out["norm"][0, 0])
    assert np.allclose(mean[sel], v, atol=5 * N / s / math.sqrt(T))
    assert np.all(mean[np.setdiff1d(np.arange(d), sel)] == 0)
    beta = min(k / s**2, math.sqrt(k) / s)
    assert m2 <= (1 + beta) * float(v @ v) * 1.02


def test_bump_probability_is_the_fraction():
    # one kept coordinate at a known fraction between two levels
    s, T = 4, 6000
    u = np.zeros((1, 8), np.float32)
    u[0, 0], u[0, 1] = 4.0, 3.0             # N = 5, p = 4*3/5 = 2.4 for the second one
    x = np.zeros(8, np.float32)
    plan = O.Plan(1, 8, k=2, s=s, quantizer=O.QSGD, seed=5)
    ups = 0
    for t in range(T):
        out = O.compress_feedback(plan, t, x, -u, np.zeros_like(u), details=True)
        assert out["norm"][0, 0] == 5.0 and out["level"][0, 1] in (2, 3)
        ups += int(out["level"][0, 1] == 3)
    f = float(np.float32(np.float32(12.0) / np.float32(5.0)) - 2)
    assert abs(ups / T - f) < 5 * math.sqrt(f * (1 - f) / T)


def test_sign_l1_closed_form_and_k_equals_d():
    # proof of Lemma 3 with m = 1: ||u - N1 Sign/k||^2 = ||u||^2 - N1^2 / k
    R, d = 2, 300
    x, xw, mem = I.gaussian_round(R, d, seed=12)
    for k in (1, 17, d):
        plan = O.Plan(R, d, k=k, quantizer=O.SIGN_L1)
        out, u, mem2 = run_details(plan, 0, x, xw, mem)
        for r in range(R):
            N1 = float(out["norm"][r, 0])
            lhs = float((mem2[r].astype(np.float64) ** 2).sum())
            rhs = float((u[r].astype(np.float64) ** 2).sum()) - N1 * N1 / k
            assert lhs == pytest.approx(rhs, rel=1e-5)
    # k = d: the scaled sign compressor (||u||_1 / d) sign(u)
    dense = decode_dense(plan, out, 0)
    want = np.where(u[0] < 0, -1.0, 1.0) * float(np.abs(u[0].astype(np.float64)).sum()) / d
    assert np.allclose(dense, want, rtol=1e-6)


def test_contraction_inequalities():
    # Definition 3 with gamma of Lemma 2 (scaled QSGD) and of Rand_k (k/d), in expectation
    R, d, k, s, T = 1, 128, 16, 2, 1500
    x, xw, mem = I.gaussian_round(R, d, seed=15)
    for sp, qz in [(O.TOPK, O.QSGD_SCALED), (O.RANDK, O.QSGD_SCALED), (O.RANDK, O.SIGN_L1)]:
        plan = O.Plan(R, d, k=k, s=s, sparsifier=sp, quantizer=qz, seed=31)
        ratio = 0.0
        for t in range(T):
            out, u, mem2 = run_details(plan, t, x, xw, mem)
            ratio += float((mem2[0].astype(np.float64) ** 2).sum() / (u[0].astype(np.float64) ** 2).sum()) / T
        beta = min(k / s**2, math.sqrt(k) / s)
        gamma = k / (d * (1 + beta)) if qz == O.QSGD_SCALED else 1.0 / d
        assert ratio <= (1 - gamma) * 1.01, (sp, qz, ratio, 1 - gamma)


# ----------------------------------------------------------------------------- wire
def read_bits(words, bitpos, width):
    v = 0
    for b in range(width):
        v |= ((int(words[(bitpos + b) // 32]) >> ((bitpos + b) % 32)) & 1) << b
    return v


def clog2(v):
    return max(1, (int(v) - 1).bit_length())


def python_decode(plan, words):
    """Independent reader of one worker's record -> list per segment of (n, norm, idx, sign, level)."""
    has_lvl = plan.quantizer != O.SIGN_L1
    bl = clog2(plan.s)
    pos = 2 * plan.nseg
    recs = []
    for g in range(plan.nseg):
        n = int(words[2 * g])
        norm = np.array([words[2 * g + 1]], np.uint32).view(np.float32)[0]
        bi = clog2(plan.offsets[g + 1] - plan.offsets[g])
        wi, ws = -(-n * bi // 32), -(-n // 32)
        wl = -(-n * bl // 32) if has_lvl else 0
        idx = [read_bits(words[pos:], j * bi, bi) for j in range(n)]
        sgn = [read_bits(words[pos + wi:], j, 1) for j in range(n)]
        lvl = [read_bits(words[pos + wi + ws:], j * bl, bl) + 1 for j in range(n)] if has_lvl else [1] * n
        recs.append((n, norm, idx, sgn, lvl, pos, wi + ws + wl))
        pos += wi + ws + wl
    return recs, pos


@pytest.mark.parametrize("quantizer,s", [(O.QSGD, 16), (O.QSGD, 2), (O.QSGD, 3), (O.QSGD, 256), (O.SIGN_L1, 1)])
def test_wire_roundtrip_and_bit_count(quantizer, s):
    R = 3
    sizes = [64, 1, 1000, 33, 4096]
    off = I.segments_from_sizes(sizes)
    kseg = np.array([5, 1, 40, 33, 7], np.int64)
    d = int(off[-1])
    x, xw, mem = I.gaussian_round(R, d, seed=18)
    plan = O.Plan(R, d, s=s, quantizer=quantizer, seed=2, offsets=off, kseg=kseg)
    out, u, _ = run_details(plan, 3, x, xw, mem)
    has_lvl = quantizer != O.SIGN_L1
    for r in range(R):
        recs, used = python_decode(plan, out["wire"][r])
        assert used <= plan.wire_words() == out["stride"]
        assert np.all(out["wire"][r, used:] == 0)
        bits, pos = 0, 0
        for g, (n, norm, idx, sgn, lvl, wpos, wlen) in enumerate(recs):
            k = int(kseg[g])
            keep = out["level"][r, pos:pos + k] > 0
            assert n == int(keep.sum()) == out["n"][r, g]
            assert norm.view(np.uint32) == out["norm"][r, g].view(np.uint32)
            assert idx == list(out["sel"][r, pos:pos + k][keep] - off[g]) and idx == sorted(idx)
            assert sgn == list(out["sign"][r, pos:pos + k][keep])
            assert lvl == list(out["level"][r, pos:pos + k][keep])
            bi = clog2(sizes[g])
            bits += 64 + n * (bi + 1 + (clog2(s) if has_lvl else 0))
            # padding bits of each stream are zero
            wi, ws = -(-n * bi // 32), -(-n // 32)
            for start, width, cnt in ((wpos, bi, wi), (wpos + wi, 1, ws)):
                tail = cnt * 32 - n * width
                if tail:
                    assert int(out["wire"][r, start + cnt - 1]) >> (32 - tail) == 0
            pos += k
        assert bits == out["bits"][r]
    # capacity formula: directory + streams sized for n = k
    want = 2 * len(sizes) + sum(-(-int(k) * clog2(n) // 32) + -(-int(k) // 32) +
                                (-(-int(k) * clog2(s) // 32) if has_lvl else 0)
                                for k, n in zip(kseg, sizes))
    assert plan.wire_words() == want


# ----------------------------------------------------------------------------- master, piecewise
def test_master_update_against_numpy():
    R, d, k = 4, 500, 60
    x, xw, mem = I.gaussian_round(R, d, seed=20)
    xw[1] = xw[0]            # two workers with identical updates: every index collides
    mem[1] = mem[0]
    for qz in (O.QSGD, O.SIGN_L1):
        plan = O.Plan(R, d, k=k, s=16, quantizer=qz, seed=1)
        out, u, _ = run_details(plan, 0, x, xw, mem)
        acc = np.zeros(d, np.float32)
        for r in range(R):
            recs, _ = python_decode(plan, out["wire"][r])
            n, N, idx, sgn, lvl, _, _ = recs[0]
            for j in range(n):
                mag = N / np.float32(k) if qz == O.SIGN_L1 else (N * np.float32(lvl[j])) / np.float32(16)
                acc[idx[j]] = acc[idx[j]] + (-mag if sgn[j] else mag)
        want = (x - acc / np.float32(R)).astype(np.float32)
        x2 = x.copy()
        assert O.unpack_accumulate(plan, x2, out["wire"]) == 0
        assert np.array_equal(x2.view(np.uint32), want.view(np.uint32))
        # Algorithm 1, master line: x_{t+1} = x_t - (1/R) sum_r g_r
        dense = sum(decode_dense(plan, out, r) for r in range(R))
        assert np.allclose(x2, x.astype(np.float64) - dense / R, rtol=1e-6, atol=1e-7)


def test_piecewise_equals_per_segment_operator():
    # Corollary 1: C(x) = [C_1(x_1) ... C_L(x_L)]; checked with the deterministic operator
    sizes = [50, 7, 300]
    off = I.segments_from_sizes(sizes)
    kseg = np.array([5, 7, 11], np.int64)
    d = int(off[-1])
    x, xw, mem = I.gaussian_round(2, d, seed=23)
    whole, u, mem_w = run_details(O.Plan(2, d, quantizer=O.SIGN_L1, offsets=off, kseg=kseg), 0, x, xw, mem)
    pos = 0
    for g, n in enumerate(sizes):
        sl = slice(int(off[g]), int(off[g + 1]))
        part, _, mem_p = run_details(O.Plan(2, n, k=int(kseg[g]), quantizer=O.SIGN_L1), 0,
                                     np.ascontiguousarray(x[sl]), np.ascontiguousarray(xw[:, sl]),
                                     np.ascontiguousarray(mem[:, sl]))
        k = int(kseg[g])
        assert np.array_equal(whole["sel"][:, pos:pos + k] - off[g], part["sel"])
        assert np.array_equal(whole["norm"][:, g], part["norm"][:, 0])
        assert np.array_equal(mem_w[:, sl], mem_p)
        pos += k


# ----------------------------------------------------------------------------- Algorithm 1 / 2
def test_memory_maintenance_identity():
    # Lemma 6: mean_r xhat_r - xtilde = mean_r m_r, where the virtual sequence xtilde takes
    # every local gradient step uncompressed.
    R, d, k, H, T = 4, 256, 12, 3, 24
    g = np.random.default_rng(2)
    plan = O.Plan(R, d, k=k, s=16, quantizer=O.QSGD, seed=4)
    x = np.zeros(d, np.float32)
    xw = np.zeros((R, d), np.float32)
    mem = np.zeros((R, d), np.float32)
    xt = np.zeros(d, np.float64)
    eta = 0.05
    for t in range(T):
        grad = g.standard_normal((R, d)).astype(np.float32)
        x_before, mem_before = x.copy(), mem.copy()
        O.local_step(plan, xw, grad, eta)
        xt -= float(np.float32(eta)) * grad.astype(np.float64).mean(axis=0)
        if (t + 1) % H == 0:
            assert O.sync_round(plan, t, x, xw, mem)["rc"] == 0
            assert np.array_equal(xw, np.broadcast_to(x, xw.shape))
        else:                                   # between synchronisations x and m do not move
            assert np.array_equal(x, x_before) and np.array_equal(mem, mem_before)
        lhs = xw.astype(np.float64).mean(axis=0) - xt
        assert np.allclose(lhs, mem.astype(np.float64).mean(axis=0), atol=2e-5)


def test_async_round_uses_divisor_R_and_touches_only_the_subset():
    R, d, k = 4, 200, 9
    x, xw, mem = I.gaussian_round(R, d, seed=30)
    anchors = (x[None, :] + 0.01 * np.random.default_rng(1).standard_normal((R, d))).astype(np.float32)
    mask = np.array([1, 0, 1, 0], np.uint8)
    plan = O.Plan(R, d, k=k, quantizer=O.SIGN_L1)
    x2, xw2, mem2, an2 = x.copy(), xw.copy(), mem.copy(), anchors.copy()
    out = O.sync_round(plan, 0, x2, xw2, mem2, anchors=an2, mask=mask)
    assert out["rc"] == 0
    for r in (1, 3):                            # not in S: nothing of theirs changes
        assert np.array_equal(xw2[r], xw[r]) and np.array_equal(mem2[r], mem[r])
        assert np.array_equal(an2[r], anchors[r])
    total = np.zeros(d)
    for r in (0, 2):
        u = (mem[r] + (anchors[r] - xw[r])).astype(np.float32)   # Algorithm 2 uses the worker's anchor
        sel = brute_topk(u, k)
        gval = np.abs(u[sel].astype(np.float64)).sum() / k
        total[sel] += np.where(u[sel] < 0, -gval, gval)
        assert np.array_equal(xw2[r], x2) and np.array_equal(an2[r], x2)
    assert np.allclose(x2, x - total / R, rtol=1e-6, atol=1e-7)  # divisor R, not |S|
    assert not np.allclose(x2, x - total / 2, rtol=1e-4, atol=1e-6)


def test_nonfinite_and_bad_arguments():
    x, xw, mem = I.gaussian_round(2, 40, seed=1)
    mem[1, 3] = np.inf
    assert O.compress_feedback(O.Plan(2, 40, k=4), 0, x, xw, mem)["rc"] == -5
    assert O.Plan(2, 40, k=0).wire_words() == -1
    assert O.Plan(2, 40, k=41).wire_words() == -1


# ----------------------------------------------------------------------------- shape table
def test_resnet50_table_matches_the_paper():
    want = dict(l.split() for l in open(os.path.join(GOLDEN, "resnet50_table.txt"))
                if l.strip() and not l.startswith("#"))
    sizes = I.resnet50_tensor_sizes()
    assert len(sizes) == int(want["tensors"])
    assert sum(sizes) == int(want["elements"])
    assert int(I.k_per_tensor_capped(sizes).sum()) == int(want["sum_min_dt_1000"])
    assert I.k_from_ratio(65536, 1, 100) == 655


def test_single_worker_entry_equals_the_batch_entry():
    R, d, k = 3, 5000, 50
    x, xw, mem = I.gaussian_round(R, d, seed=1)
    plan = O.Plan(R, d, k=k, s=4, sparsifier=O.RANDK, quantizer=O.QSGD, seed=9)
    m2 = mem.copy()
    out = O.compress_feedback(plan, 5, x, xw, m2)
    for r in range(R):
        mr = mem[r].copy()
        one = O.compress_worker(plan, 5, r, x, xw[r].copy(), mr)
        assert one["rc"] == 0 and np.array_equal(one["wire"], out["wire"][r])
        assert np.array_equal(mr, m2[r]) and one["bits"] == out["bits"][r]


# ----------------------------------------------------------------------------- sparsifier alone
def test_plain_sparsifier_is_topk_itself():
    # quantizer NONE: C(u) = Top_k(u) (Section 2.2), memory 0 on the kept set, gamma = k/d holds surely
    R, d, k = 3, 900, 37
    x, xw, mem = I.gaussian_round(R, d, seed=33)
    plan = O.Plan(R, d, k=k, quantizer=O.NONE)
    out, u, mem2 = run_details(plan, 2, x, xw, mem)
    bi = clog2(d)
    assert plan.wire_words() == 2 + -(-k * bi // 32) + k
    acc = np.zeros(d, np.float64)
    for r in range(R):
        sel = brute_topk(u[r], k)
        assert list(out["sel"][r]) == sel and out["n"][r, 0] == k
        words = out["wire"][r]
        assert int(words[0]) == k and int(words[1]) == 0
        idx = [read_bits(words[2:], j * bi, bi) for j in range(k)]
        vals = words[2 + -(-k * bi // 32): 2 + -(-k * bi // 32) + k].view(np.float32)
        assert idx == sel and np.array_equal(vals.view(np.uint32), u[r, sel].view(np.uint32))
        assert out["bits"][r] == 64 + k * (bi + 32)
        want = u[r].copy()
        want[sel] = 0.0
        assert np.array_equal(mem2[r].view(np.uint32), want.view(np.uint32))
        lhs = float((mem2[r].astype(np.float64) ** 2).sum())
        assert lhs <= (1 - k / d) * float((u[r].astype(np.float64) ** 2).sum())
        acc[sel] += u[r, sel].astype(np.float64)
    x2 = x.copy()
    assert O.unpack_accumulate(plan, x2, out["wire"]) == 0
    assert np.allclose(x2, x - acc / R, rtol=1e-6, atol=1e-7)


def test_plain_randk_contracts_in_expectation():
    # E||u - Rand_k(u)||^2 = (1 - k/d) ||u||^2 (Section 2.2 with the proof of Lemma 8)
    d, k, T = 60, 15, 3000
    x, xw, mem = I.gaussian_round(1, d, seed=35)
    plan = O.Plan(1, d, k=k, sparsifier=O.RANDK, quantizer=O.NONE, seed=3)
    ratio = 0.0
    for t in range(T):
        out, u, mem2 = run_details(plan, t, x, xw, mem)
        ratio += float((mem2[0].astype(np.float64) ** 2).sum() / (u[0].astype(np.float64) ** 2).sum()) / T
    assert abs(ratio - (1 - k / d)) < 0.01


# ---------------------------------------------------------------- momentum on the local iterations (Section 5.1)
def test_momentum_step_with_mu_zero_is_the_plain_step():
    R, d = 3, 97
    g = np.random.default_rng(11)
    plan = O.Plan(R, d, k=5, s=4)
    xw = g.standard_normal((R, d)).astype(np.float32)
    grad = g.standard_normal((R, d)).astype(np.float32)
    a, b = xw.copy(), xw.copy()
    vel = g.standard_normal((R, d)).astype(np.float32)      # ignored when mu = 0
    O.local_step(plan, a, grad, 0.1)
    O.local_step_momentum(plan, b, vel, grad, 0.1, 0.0)
    assert np.array_equal(a, b)
    assert np.array_equal(vel, grad)                        # v <- 0 * v + grad


def test_momentum_constant_gradient_closed_form():
    """Constant gradient c: v_n = c (1 - mu^n) / (1 - mu) and
    x_n = x_0 - eta c (n - mu (1 - mu^n) / (1 - mu)) / (1 - mu)."""
    R, d, n, eta, mu = 2, 64, 40, 0.01, 0.9
    g = np.random.default_rng(12)
    plan = O.Plan(R, d, k=4, s=4)
    c = g.standard_normal((R, d)).astype(np.float32)
    x0 = g.standard_normal((R, d)).astype(np.float32)
    xw, vel = x0.copy(), np.zeros((R, d), np.float32)
    for _ in range(n):
        O.local_step_momentum(plan, xw, vel, c, eta, mu)
    mu64, eta64, c64 = float(np.float32(mu)), float(np.float32(eta)), c.astype(np.float64)
    v_n = c64 * (1 - mu64 ** n) / (1 - mu64)
    x_n = x0.astype(np.float64) - eta64 * c64 * (n - mu64 * (1 - mu64 ** n) / (1 - mu64)) / (1 - mu64)
    assert np.allclose(vel, v_n, rtol=1e-5, atol=1e-6)
    assert np.allclose(xw, x_n, rtol=1e-5, atol=1e-5)
    # a wrong sign or a velocity that is not carried would be far outside these tolerances
    assert np.abs(xw - x0).max() > 10 * eta64 * np.abs(c64).max()


def test_momentum_step_respects_the_mask():
    R, d = 4, 33
    g = np.random.default_rng(13)
    plan = O.Plan(R, d, k=3, s=4)
    xw = g.standard_normal((R, d)).astype(np.float32)
    vel = g.standard_normal((R, d)).astype(np.float32)
    grad = g.standard_normal((R, d)).astype(np.float32)
    xw0, vel0 = xw.copy(), vel.copy()
    O.local_step_momentum(plan, xw, vel, grad, 0.1, 0.9, mask=[1, 0, 0, 1])
    assert np.array_equal(xw[1:3], xw0[1:3]) and np.array_equal(vel[1:3], vel0[1:3])
    v = (np.float32(0.9) * vel0[0]).astype(np.float32) + grad[0]
    assert np.array_equal(vel[0], v.astype(np.float32))
    assert np.array_equal(xw[0], (xw0[0] - (np.float32(0.1) * v).astype(np.float32)).astype(np.float32))


# ---------------------------------------------------------------- Lemma 3 with m = 2 (sign scaled by the l2 norm)
def test_sign_l2_closed_form_contraction_and_record():
    R, d = 2, 300
    x, xw, mem = I.gaussian_round(R, d, seed=14)
    for k in (1, 17, d):
        plan = O.Plan(R, d, k=k, quantizer=O.SIGN_L2)
        out, u, mem2 = run_details(plan, 0, x, xw, mem)
        assert plan.wire_words() == O.Plan(R, d, k=k, quantizer=O.SIGN_L1).wire_words()
        for r in range(R):
            kept = u[r][out["sel"][r]]
            N2 = out["norm"][r, 0]
            assert N2 == exact_l2(kept)                               # the norm in the record is the l2 norm
            u64 = u[r].astype(np.float64)
            N1 = float(np.abs(kept.astype(np.float64)).sum())
            lhs = float((mem2[r].astype(np.float64) ** 2).sum())
            # sum over the kept set of (u_i - a sgn_i)^2 with a = N2/k, plus the untouched rest
            rhs = float((u64 ** 2).sum()) - 2.0 * float(N2) / k * N1 + float(N2) ** 2 / k
            assert lhs == pytest.approx(rhs, rel=1e-5)
            # compression operator with gamma_2 = k^(2/2 - 1) / d = 1/d, surely for Top_k
            assert lhs <= (1.0 - 1.0 / d) * float((u64 ** 2).sum()) * (1 + 1e-6)
            # the record decodes to +-N2/k on the kept set
            dense = decode_dense(plan, out, r)
            want = np.zeros(d)
            want[out["sel"][r]] = np.where(kept < 0, -1.0, 1.0) * float(np.float32(N2) / np.float32(k))
            assert np.array_equal(dense, want)
            if k == 1:                                                # one kept entry: C(u) = u there, memory 0
                assert mem2[r][out["sel"][r][0]] == 0.0
    # the same kept set as the l1-scaled operator (the sparsifier does not see the quantizer)
    a, _, _ = run_details(O.Plan(R, d, k=17, quantizer=O.SIGN_L1), 0, x, xw, mem)
    b, _, _ = run_details(O.Plan(R, d, k=17, quantizer=O.SIGN_L2), 0, x, xw, mem)
    assert np.array_equal(a["sel"], b["sel"]) and np.array_equal(a["sign"], b["sign"])


def test_sign_l2_master_decodes_the_record():
    R, d, k = 3, 500, 20
    x, xw, mem = I.gaussian_round(R, d, seed=15)
    plan = O.Plan(R, d, k=k, quantizer=O.SIGN_L2)
    out, u, _ = run_details(plan, 0, x, xw, mem)
    acc = np.zeros(d, np.float32)
    for r in range(R):
        g = np.zeros(d, np.float32)
        g[out["sel"][r]] = values_from_details(plan, out, r)
        acc = (acc + g).astype(np.float32)
    want = x.copy()
    touched = np.zeros(d, bool)
    for r in range(R):
        touched[out["sel"][r]] = True
    want[touched] = (x[touched] - acc[touched] / np.float32(R)).astype(np.float32)
    x2 = x.copy()
    assert O.unpack_accumulate(plan, x2, out["wire"]) == 0
    assert np.array_equal(x2, want)
