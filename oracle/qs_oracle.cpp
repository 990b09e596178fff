// Qsparse-local-SGD synchronisation round: plain sequential CPU statement.
//
// TEST INFRASTRUCTURE ONLY.  This file is the checker that the CUDA library is
// compared against; nothing in the product path may call it.  It shares no code
// with the CUDA sources: every constant, table and helper here is written out
// again on this side.
//
// What it computes (Basu, Data, Karakus, Diggavi, "Qsparse-local-SGD"):
//   worker r, Algorithm 1 worker branch at a synchronisation index:
//       u_r   = m_r + (x_t - xhat_r)                (argument of the compressor)
//       g_r   = Q Comp_k(u_r)                       (Section 2.2/2.3 operators)
//       m_r  <- u_r - g_r                           (memory update)
//       send g_r                                    (wire record, format below)
//   master, Algorithm 1 master branch:
//       x_{t+1} = x_t - (1/R) sum_r g_r,  broadcast, xhat_r <- x_{t+1}
//   Algorithm 2 (asynchronous) differs in three places: the worker uses its own
//   anchor x_t^{(r)}, only workers in the set S take part, and the divisor stays R.
//
// Readings of what the paper leaves open (each is mirrored, independently, by
// the CUDA library):
//   [order]   u = m + (x - xhat) in fp32, two roundings, no fused multiply-add.
//   [top-k]   key = bit pattern of |u| as uint32; order (key descending, index
//             ascending); exactly k indices are taken (the paper's index set is
//             a k-subset), zeros included.  Non-finite u is an error.
//   [rand-k]  h_i = one Philox4x32-10 word per (seed, round, worker, element,
//             stream 1); the k smallest (h_i, i) inside the segment are taken.
//   [qsgd]    the quantizer of the QSGD paper the text defers to:
//             Q_s(v)_i = ||v||_2 sgn(v_i) xi_i, xi_i in {l/s,(l+1)/s},
//             l = floor(s|v_i|/||v||_2), P(up) = s|v_i|/||v||_2 - l, applied to
//             the length-k vector of kept entries (proof of Lemma 1).
//             fp32 recipe: a = |u|*s; p = a/N; l = floor(p); f = p - l;
//             U = (w >> 8) * 2^-24 with w the Philox word of stream 0;
//             level = min(l + (U < f), s); N == 0 gives level 0 everywhere.
//   [norm]    the exact real sum of squares (or magnitudes) rounded once to
//             fp64; l2: sqrt in fp64 then rounded to fp32; l1: rounded to fp32.
//   [value]   QSGD: g = (N*level)/s, times c = fl32(1/(1+beta_{k,s})) for the
//             scaled operator of Lemma 2, beta_{k,s} = min(k/s^2, sqrt(k)/s)
//             in fp64; Sign (Lemma 3, m = 1): g = N1/k.  The sign is applied
//             last by negation; Sign(0) = +1 (Definition 2), so the sign bit is
//             (u < 0), not the IEEE sign bit.
//   [none]    quantizer 3 sends the kept values themselves (the sparsifier alone, a compression
//             operator with gamma = k/d, Section 2.2; the Top_k-SGD scheme of the comparisons):
//             g = u on the kept set, so the memory becomes 0 there; the record carries 32-bit
//             values instead of signs and levels, and all k entries.
//   [sign-l2] quantizer 4 is Lemma 3's operator with m = 2: g = N2/k with N2 the l2 norm of
//             the kept vector ([norm]); record as for quantizer 2.  m >= 3 is not provided (its
//             sum of m-th powers has no exact fp64 terms, and gamma_m only shrinks with m).
//   [min-max] quantizer 5 is the stochastic s-level quantizer of Definition 1's example 2: s levels
//             between the smallest entry lo and the largest entry hi of the kept vector (signed
//             values), lo + j D, j = 0 .. s-1, D = (hi - lo)/(s - 1); an entry goes to the level
//             below or above it, up with probability (v - lo)/D - floor((v - lo)/D) (unbiased,
//             independently per component; error at most k/(2 (s-1)^2) ||v||^2 in expectation, the
//             bound of the mean-estimation paper the text cites; the text's d/(2 s^2) counts the
//             intervals as s).  fp32 recipe: D = (hi - lo)/(s-1); p = (v - lo)/D; l = floor(p);
//             f = p - l; U as for [qsgd]; j = min(l + (U < f), s - 1); g = lo + j * D (product and
//             sum rounded on their own); hi == lo: every entry gets j = 0.  Needs s >= 2.  Every
//             kept entry is sent (j = 0 stands for lo, not for nothing): in the record the count
//             is implied (n = k), the header pair carries (lo, hi), there is no sign stream and the
//             level stream holds j; bits = sum_seg 64 + k (b_idx + b_lvl).  Levels are reported
//             as j + 1 (1 .. s), like QSGD's.
//   [pieces]  Corollary 1: each segment has its own k, norm, beta.
//   [momentum] Section 5.1 applies momentum 0.9 on the local iterations and prints no
//             formula: the heavy-ball form v <- mu v + grad, xhat <- xhat - eta v is taken,
//             every product and sum rounded to fp32 on its own.
//   [master]  acc = 0; acc += g_r in worker order; x = x - acc/R; indices no
//             worker sent are left untouched.
//   [wire]    per worker: a directory of nseg (n, norm bits) word pairs, then
//             for each segment in order three bit streams, each padded to a
//             32-bit word, fields LSB first: n segment-local indices
//             (ascending) of b_idx = max(1, ceil(log2 d_seg)) bits, n sign
//             bits, and for QSGD n fields (level-1) of b_lvl = max(1,
//             ceil(log2 s)) bits.  QSGD drops level-0 entries; Sign sends all
//             k.  bits = sum_seg 64 + n (b_idx + 1 + b_lvl).
//   [gap coding] the paper counts transmitted bits and leaves the coding of the k
//             indices open: a second form of the record sends the first index of a
//             segment and then the gaps between successive indices in short fields,
//             the few gaps too large for a field in a stream of exceptions; the width
//             is the one that makes the record smallest (format above gap_words).
//   [philox]  key = (seed_lo, seed_hi); counter = (element >> 2, worker,
//             round_lo, (round_hi << 8) | stream); word = out[element & 3];
//             element is the global coordinate index.
//
// Pins (tests/test_oracle_*.py, run without a GPU): Philox known-answer vectors
// of the published generator; brute-force Python sorts on tiny inputs with
// crafted ties; exact rational arithmetic for the norms; k = 1 special case
// (level = s, g = u, m = 0); unbiasedness and the second-moment bound of
// Definition 1; the closed form of Lemma 3's proof for m = 1; inclusion
// probability k/d of Rand_k; an independent Python bit reader for the wire;
// the memory-maintenance identity of Lemma 6; the async divisor R; for the
// gap-coded record a hand-worked example, an independent Python reader, the round
// trip and the saving on uniformly spread indices.
//
// Build: g++ -O2 -ffp-contract=off -shared -fPIC (see oracle/build.py).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <utility>
#include <vector>

namespace {

enum { SP_TOPK = 0, SP_RANDK = 1 };
enum { QZ_QSGD = 0, QZ_QSGD_SCALED = 1, QZ_SIGN_L1 = 2, QZ_NONE = 3, QZ_SIGN_L2 = 4, QZ_MINMAX = 5 };
inline bool is_sign(int quantizer) { return quantizer == QZ_SIGN_L1 || quantizer == QZ_SIGN_L2; }
enum { ERR_OK = 0, ERR_ARG = -1, ERR_CAPACITY = -4, ERR_NONFINITE = -5 };

// ---------------------------------------------------------------- Philox
// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11).
void philox4x32_10(const uint32_t c_in[4], const uint32_t k_in[2], uint32_t out[4]) {
    uint32_t c0 = c_in[0], c1 = c_in[1], c2 = c_in[2], c3 = c_in[3];
    uint32_t k0 = k_in[0], k1 = k_in[1];
    for (int rnd = 0; rnd < 10; ++rnd) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

uint32_t philox_word(uint64_t seed, uint64_t round, uint32_t worker, uint64_t element,
                     uint32_t stream) {
    uint32_t ctr[4], key[2], out[4];
    ctr[0] = (uint32_t)(element >> 2);
    ctr[1] = worker;
    ctr[2] = (uint32_t)round;
    ctr[3] = ((uint32_t)(round >> 32) << 8) | stream;
    key[0] = (uint32_t)seed;
    key[1] = (uint32_t)(seed >> 32);
    philox4x32_10(ctr, key, out);
    return out[element & 3];
}

// ---------------------------------------------------------------- exact sums
// Non-negative big integer in base 2^32; bit 0 stands for 2^-BIAS.
struct BigAcc {
    static const int BIAS = 320;
    std::vector<uint64_t> digit;
    BigAcc() : digit(32, 0) {}
    // add mant * 2^e2
    void add(uint64_t mant, int e2) {
        int pos = e2 + BIAS;
        int q = pos / 32, o = pos % 32;
        unsigned __int128 v = (unsigned __int128)mant << o;
        uint64_t carry = 0;
        for (int j = q; j < (int)digit.size(); ++j) {
            uint64_t t = digit[j] + (uint64_t)(v & 0xffffffffu) + carry;
            digit[j] = t & 0xffffffffu;
            carry = t >> 32;
            v >>= 32;
            if (v == 0 && carry == 0) break;
        }
    }
    int bit(int p) const { return p < 0 ? 0 : (int)((digit[p / 32] >> (p % 32)) & 1u); }
    // value rounded to the nearest double, ties to even
    double to_double() const {
        int top = -1;
        for (int j = (int)digit.size() - 1; j >= 0 && top < 0; --j)
            if (digit[j]) {
                int b = 31;
                while (!((digit[j] >> b) & 1u)) --b;
                top = j * 32 + b;
            }
        if (top < 0) return 0.0;
        uint64_t mant = 0;
        for (int p = top; p > top - 53; --p) mant = (mant << 1) | (uint64_t)bit(p);
        int guard = bit(top - 53);
        int sticky = 0;
        for (int p = top - 54; p >= 0 && !sticky; --p) sticky = bit(p);
        if (guard && (sticky || (mant & 1u))) mant += 1;
        return std::ldexp((double)mant, top - 52 - BIAS);
    }
};

inline void split_f32(float v, uint64_t* mant, int* e2) {
    uint32_t b;
    std::memcpy(&b, &v, 4);
    uint32_t e = (b >> 23) & 0xffu, m = b & 0x7fffffu;
    if (e == 0) { *mant = m; *e2 = -149; }
    else        { *mant = m | 0x800000u; *e2 = (int)e - 150; }
}

float norm_l2_exact(const float* v, int64_t n) {
    BigAcc acc;
    for (int64_t i = 0; i < n; ++i) {
        uint64_t m; int e;
        split_f32(v[i], &m, &e);
        acc.add(m * m, 2 * e);
    }
    double sum = acc.to_double();
    return (float)std::sqrt(sum);
}

float norm_l1_exact(const float* v, int64_t n) {
    BigAcc acc;
    for (int64_t i = 0; i < n; ++i) {
        uint64_t m; int e;
        split_f32(v[i], &m, &e);
        acc.add(m, e);
    }
    return (float)acc.to_double();
}

// ---------------------------------------------------------------- selection
inline uint32_t abs_key(float v) {
    uint32_t b;
    std::memcpy(&b, &v, 4);
    return b & 0x7fffffffu;
}

typedef std::pair<uint32_t, int64_t> KeyIdx;

struct TopOrder {  // larger key first, then lower index
    bool operator()(const KeyIdx& a, const KeyIdx& b) const {
        if (a.first != b.first) return a.first > b.first;
        return a.second < b.second;
    }
};
struct RandOrder {  // smaller hash first, then lower index
    bool operator()(const KeyIdx& a, const KeyIdx& b) const {
        if (a.first != b.first) return a.first < b.first;
        return a.second < b.second;
    }
};

// mode 0: full sort of the segment (the definition); mode 1: nth_element.
template <class Order>
void take_first_k(std::vector<KeyIdx>& items, int64_t k, int mode, int64_t* idx_out) {
    if (mode == 0) std::sort(items.begin(), items.end(), Order());
    else if (k < (int64_t)items.size())
        std::nth_element(items.begin(), items.begin() + k, items.end(), Order());
    std::vector<int64_t> chosen(k);
    for (int64_t j = 0; j < k; ++j) chosen[j] = items[j].second;
    std::sort(chosen.begin(), chosen.end());
    for (int64_t j = 0; j < k; ++j) idx_out[j] = chosen[j];
}

// Top_k over u[0..n): segment-local indices, ascending.
void select_topk(const float* u, int64_t n, int64_t k, int mode, int64_t* idx_out) {
    std::vector<KeyIdx> items(n);
    for (int64_t i = 0; i < n; ++i) items[i] = KeyIdx(abs_key(u[i]), i);
    take_first_k<TopOrder>(items, k, mode, idx_out);
}

// Rand_k over global elements [lo, lo+n): segment-local indices, ascending.
void select_randk(uint64_t seed, uint64_t round, uint32_t worker, int64_t lo, int64_t n,
                  int64_t k, int mode, int64_t* idx_out) {
    std::vector<KeyIdx> items(n);
    for (int64_t i = 0; i < n; ++i)
        items[i] = KeyIdx(philox_word(seed, round, worker, (uint64_t)(lo + i), 1u), i);
    take_first_k<RandOrder>(items, k, mode, idx_out);
}

// ---------------------------------------------------------------- quantizers
int qsgd_level(float u, float N, int s, uint32_t w) {
    if (N == 0.0f) return 0;
    float a = std::fabs(u) * (float)s;
    float p = a / N;
    float l = std::floor(p);
    float f = p - l;
    float U = (float)(w >> 8) * 5.9604644775390625e-08f;  // 2^-24
    int level = (int)l + (U < f ? 1 : 0);
    return level < s ? level : s;
}

double beta_qsgd(int64_t k, int s) {
    double a = (double)k / ((double)s * (double)s);
    double b = std::sqrt((double)k) / (double)s;
    return a < b ? a : b;
}

float value_qsgd(float N, int level, int s, int scaled, float c, int negative) {
    float g = (N * (float)level) / (float)s;
    if (scaled) g = g * c;
    return negative ? -g : g;
}

// Stochastic s-level quantizer between the smallest and the largest entry of the kept vector
// (Section 2.1, Definition 1, example 2): s levels lo, lo + D, .., lo + (s-1) D with D = (hi - lo) /
// (s - 1); an entry between two levels goes to the upper one with the probability that makes the
// result unbiased.  Levels are numbered 1 .. s here (level l stands for lo + (l - 1) D), so that
// the record's level field holds l - 1 as for QSGD.  fp32, every operation rounded on its own; the
// uniform draw is the top 24 bits of the Philox word, as for QSGD.  hi == lo: one level.
int minmax_level(float v, float lo, float hi, int s, uint32_t w) {
    float D = (hi - lo) / (float)(s - 1);
    if (!(D > 0.0f)) return 1;
    float p = (v - lo) / D;
    float l = std::floor(p);
    float f = p - l;
    float U = (float)(w >> 8) * 5.9604644775390625e-08f;  // 2^-24
    int j = (int)l + (U < f ? 1 : 0);
    if (j < 0) j = 0;
    if (j > s - 1) j = s - 1;
    return j + 1;
}

float value_minmax(float lo, float hi, int s, int level) {
    float D = (hi - lo) / (float)(s - 1);
    float step = (float)(level - 1) * D;
    return lo + step;
}

float value_sign(float N1, int64_t k, int negative) {
    float g = N1 / (float)k;
    return negative ? -g : g;
}

// ---------------------------------------------------------------- wire
int ceil_log2(int64_t v) {  // smallest b with 2^b >= v
    int b = 0;
    while (((int64_t)1 << b) < v) ++b;
    return b;
}
int bits_idx(int64_t dseg) { int b = ceil_log2(dseg); return b < 1 ? 1 : b; }
int bits_lvl(int s) { int b = ceil_log2(s); return b < 1 ? 1 : b; }
int64_t words_for(int64_t nfields, int width) { return (nfields * width + 31) / 32; }

void put_bits(uint32_t* w, int64_t bitpos, int width, uint32_t val) {
    for (int b = 0; b < width; ++b)
        if ((val >> b) & 1u) w[(bitpos + b) / 32] |= 1u << ((bitpos + b) % 32);
}
uint32_t get_bits(const uint32_t* w, int64_t bitpos, int width) {
    uint32_t v = 0;
    for (int b = 0; b < width; ++b)
        v |= ((w[(bitpos + b) / 32] >> ((bitpos + b) % 32)) & 1u) << b;
    return v;
}

// words of the streams of a segment that sends n entries, and bits per entry
int64_t payload_words(int64_t n, int bi, int bl, int quantizer) {
    if (quantizer == QZ_NONE) return words_for(n, bi) + n;                 // indices, then 32-bit values
    if (quantizer == QZ_MINMAX) return words_for(n, bi) + words_for(n, bl); // indices, then levels (no signs)
    return words_for(n, bi) + words_for(n, 1) + (!is_sign(quantizer) ? words_for(n, bl) : 0);
}
int entry_bits(int bi, int bl, int quantizer) {
    if (quantizer == QZ_NONE) return bi + 32;
    if (quantizer == QZ_MINMAX) return bi + bl;
    return bi + 1 + (!is_sign(quantizer) ? bl : 0);
}

struct Plan {
    int R; int64_t d; int nseg; const int64_t* off; const int64_t* kseg;
    int s, sparsifier, quantizer; uint64_t seed;
};

int64_t wire_words(const Plan& P) {
    int64_t w = 2 * (int64_t)P.nseg;
    for (int g = 0; g < P.nseg; ++g)
        w += payload_words(P.kseg[g], bits_idx(P.off[g + 1] - P.off[g]), bits_lvl(P.s), P.quantizer);
    return w;
}

// ---------------------------------------------------------------- worker side
// One worker's compress + feedback.  anchor is x_t (sync) or x_t^{(r)} (async).
// Outputs, all optional except wire: selected global indices (sum kseg), their
// levels and signs, per-segment norm and n.
int worker_compress(const Plan& P, uint64_t round, int r, const float* anchor, const float* xw,
                    float* mem, uint32_t* wire, int64_t* bits_out, int mode, int64_t* sel_out,
                    int32_t* lvl_out, uint8_t* sgn_out, float* norm_out, int64_t* n_out) {
    const int64_t d = P.d;
    std::vector<float> u(d);
    for (int64_t i = 0; i < d; ++i) {
        float diff = anchor[i] - xw[i];
        u[i] = mem[i] + diff;
        if (!std::isfinite(u[i])) return ERR_NONFINITE;
    }
    const int has_levels = P.quantizer == QZ_QSGD || P.quantizer == QZ_QSGD_SCALED;
    const int plain = P.quantizer == QZ_NONE;   // sparsifier alone: the kept values travel as they are
    const int minmax = P.quantizer == QZ_MINMAX;
    const int bl = bits_lvl(P.s);
    int64_t payload = 2 * (int64_t)P.nseg;  // word offset of the next segment's streams
    int64_t bits = 0, selpos = 0;
    std::memset(wire, 0, sizeof(uint32_t) * (size_t)wire_words(P));
    for (int g = 0; g < P.nseg; ++g) {
        const int64_t lo = P.off[g], n_el = P.off[g + 1] - lo, k = P.kseg[g];
        std::vector<int64_t> idx(k);
        if (P.sparsifier == SP_TOPK) select_topk(&u[lo], n_el, k, mode, idx.data());
        else select_randk(P.seed, round, (uint32_t)r, lo, n_el, k, mode, idx.data());
        std::vector<float> kept(k);
        for (int64_t j = 0; j < k; ++j) kept[j] = u[lo + idx[j]];
        float vlo = kept[0], vhi = kept[0];     // smallest and largest kept entry (min/max quantizer)
        for (int64_t j = 1; j < k; ++j) { if (kept[j] < vlo) vlo = kept[j]; if (kept[j] > vhi) vhi = kept[j]; }
        const float N = (plain || minmax) ? 0.0f
                      : (has_levels || P.quantizer == QZ_SIGN_L2) ? norm_l2_exact(kept.data(), k) : norm_l1_exact(kept.data(), k);
        const float c = (float)(1.0 / (1.0 + beta_qsgd(k, P.s)));
        std::vector<int64_t> s_idx; std::vector<int> s_lvl, s_neg; std::vector<float> s_val;
        for (int64_t j = 0; j < k; ++j) {
            const int64_t gi = lo + idx[j];
            const float v = u[gi];
            const int neg = v < 0.0f ? 1 : 0;
            int level; float gval;
            if (has_levels) {
                level = qsgd_level(v, N, P.s, philox_word(P.seed, round, (uint32_t)r, (uint64_t)gi, 0u));
                gval = value_qsgd(N, level, P.s, P.quantizer == QZ_QSGD_SCALED, c, neg);
                if (level == 0) gval = 0.0f;
            } else if (plain) {
                level = 1;
                gval = v;
            } else if (minmax) {
                level = minmax_level(v, vlo, vhi, P.s, philox_word(P.seed, round, (uint32_t)r, (uint64_t)gi, 0u));
                gval = value_minmax(vlo, vhi, P.s, level);
            } else {
                level = 1;
                gval = value_sign(N, k, neg);
            }
            mem[gi] = v - gval;
            if (sel_out) sel_out[selpos + j] = gi;
            if (lvl_out) lvl_out[selpos + j] = level;
            if (sgn_out) sgn_out[selpos + j] = (uint8_t)(minmax ? 0 : neg);   // (no sign travels with the min/max quantizer)
            if (level != 0) { s_idx.push_back(idx[j]); s_lvl.push_back(level); s_neg.push_back(neg); s_val.push_back(v); }
        }
        // coordinates outside the kept set: C(u) = 0 there, so m <- u
        {
            std::vector<char> is_kept(n_el, 0);
            for (int64_t j = 0; j < k; ++j) is_kept[idx[j]] = 1;
            for (int64_t i = 0; i < n_el; ++i) if (!is_kept[i]) mem[lo + i] = u[lo + i];
        }
        selpos += k;
        const int64_t n = (int64_t)s_idx.size();
        const int bi = bits_idx(n_el);
        uint32_t nb; std::memcpy(&nb, &N, 4);
        wire[2 * g] = (uint32_t)n;
        wire[2 * g + 1] = nb;
        if (minmax) {   // every kept entry is sent, so the count is implied (n = k): the pair carries (min, max)
            std::memcpy(&wire[2 * g], &vlo, 4);
            std::memcpy(&wire[2 * g + 1], &vhi, 4);
        }
        uint32_t* w_idx = wire + payload;
        uint32_t* w_sgn = w_idx + words_for(n, bi);
        uint32_t* w_lvl = w_sgn + words_for(n, 1);
        for (int64_t j = 0; j < n; ++j) {
            put_bits(w_idx, j * bi, bi, (uint32_t)s_idx[j]);
            if (plain) {
                std::memcpy(&w_sgn[j], &s_val[j], 4);          // the value stream follows the indices
            } else if (minmax) {
                put_bits(w_sgn, j * bl, bl, (uint32_t)(s_lvl[j] - 1));   // the level stream follows the indices
            } else {
                put_bits(w_sgn, j, 1, (uint32_t)s_neg[j]);
                if (has_levels) put_bits(w_lvl, j * bl, bl, (uint32_t)(s_lvl[j] - 1));
            }
        }
        payload += payload_words(n, bi, bl, P.quantizer);
        bits += 64 + n * entry_bits(bi, bl, P.quantizer);
        if (norm_out) norm_out[g] = minmax ? vhi : N;
        if (n_out) n_out[g] = n;
    }
    if (bits_out) *bits_out = bits;
    return ERR_OK;
}

// ---------------------------------------------------------------- master side
// Decodes one worker's record from its wire words and adds it into acc.
void master_add_record(const Plan& P, const uint32_t* wire, float* acc) {
    const int has_levels = P.quantizer == QZ_QSGD || P.quantizer == QZ_QSGD_SCALED;
    const int plain = P.quantizer == QZ_NONE;
    const int minmax = P.quantizer == QZ_MINMAX;
    const int bl = bits_lvl(P.s);
    int64_t payload = 2 * (int64_t)P.nseg;
    for (int g = 0; g < P.nseg; ++g) {
        const int64_t lo = P.off[g], n_el = P.off[g + 1] - lo, k = P.kseg[g];
        const int64_t n = minmax ? k : wire[2 * g];
        float N; std::memcpy(&N, &wire[2 * g + 1], 4);
        float vlo; std::memcpy(&vlo, &wire[2 * g], 4);    // (min, max) in the header pair of the min/max quantizer
        const int bi = bits_idx(n_el);
        const float c = (float)(1.0 / (1.0 + beta_qsgd(k, P.s)));
        const uint32_t* w_idx = wire + payload;
        const uint32_t* w_sgn = w_idx + words_for(n, bi);
        const uint32_t* w_lvl = w_sgn + words_for(n, 1);
        for (int64_t j = 0; j < n; ++j) {
            const int64_t i = lo + (int64_t)get_bits(w_idx, j * bi, bi);
            const int neg = (plain || minmax) ? 0 : (int)get_bits(w_sgn, j, 1);
            float gval;
            if (plain) {
                std::memcpy(&gval, &w_sgn[j], 4);
            } else if (minmax) {
                gval = value_minmax(vlo, N, P.s, (int)get_bits(w_sgn, j * bl, bl) + 1);
            } else if (has_levels) {
                const int level = (int)get_bits(w_lvl, j * bl, bl) + 1;
                gval = value_qsgd(N, level, P.s, P.quantizer == QZ_QSGD_SCALED, c, neg);
            } else {
                gval = value_sign(N, k, neg);
            }
            acc[i] = acc[i] + gval;
        }
        payload += payload_words(n, bi, bl, P.quantizer);
    }
}

// ---------------------------------------------------------------- gap-coded record
// The paper counts what the workers transmit in bits (Section 5, the x-axes of the figures) and
// leaves the coding of the k indices open.  [gap coding] A second form of the record sends, per
// segment, the first index and then the gaps between successive indices (ascending, so every gap
// g_j = i_j - i_(j-1) - 1 >= 0) in fields of w bits.  For w >= 1 the field value E = 2^w - 1 is an
// escape: a gap >= E is sent as E and the gap itself follows, in order, in a stream of exceptions
// of b_idx bits each.  w = 0 means no fields at all and needs every gap to be 0.  The sender takes
// the w in 0 .. b_idx that makes (n - 1) w + x(w) b_idx smallest (x(w): gaps >= 2^w - 1), the
// smallest such w on a tie; w = b_idx has no exceptions, so the code is never longer than the
// plain one.  Row of one worker:
//   directory: nseg entries of five words (n, norm bits, w, first index, x); the min/max
//              quantizer keeps (min, max) in the first two, n = k.  x could be recounted from the
//              fields; it is kept as a word so that the streams' places are known at once, and is
//              not counted as transmitted;
//   per segment: n - 1 gap fields of w bits, LSB first, padded to a word; x exception fields of
//              b_idx bits, padded to a word; then the streams that follow the indices in the
//              plain record (signs, levels or values), word for word.
// bits per segment: 64 + 6 + [n >= 1] (b_idx + (n - 1) w + x b_idx) + n (entry bits - b_idx).
int bit_length(uint32_t v) { int b = 0; while (v) { ++b; v >>= 1; } return b; }

int64_t gap_words(const Plan& P) {
    int64_t w = 5 * (int64_t)P.nseg;
    const int bl = bits_lvl(P.s);
    for (int g = 0; g < P.nseg; ++g) {
        const int bi = bits_idx(P.off[g + 1] - P.off[g]);
        const int64_t k = P.kseg[g];
        // fields and exceptions together never exceed (k - 1) b_idx bits; two streams, each padded
        w += words_for(k - 1, bi) + 1 + payload_words(k, bi, bl, P.quantizer) - words_for(k, bi);
    }
    return w;
}

// the field width a segment's gaps are sent with, and the exceptions it leaves
void choose_width(const std::vector<uint32_t>& gaps, int bi, int* w_out, int64_t* x_out) {
    const int64_t m = (int64_t)gaps.size();
    int best_w = bi;
    int64_t best_x = 0, best_cost = m * bi;
    for (int w = bi - 1; w >= 0; --w) {
        int64_t x = 0;
        bool all_zero = true;
        for (int64_t j = 0; j < m; ++j) {
            if (gaps[j]) all_zero = false;
            if (w >= 1 && (uint64_t)gaps[j] >= (1ull << w) - 1ull) ++x;
        }
        if (w == 0 && !all_zero) continue;
        const int64_t cost = m * w + x * bi;
        if (cost <= best_cost) { best_cost = cost; best_w = w; best_x = x; }
    }
    *w_out = best_w;
    *x_out = best_x;
}

// plain record -> gap-coded record; returns its size in bits
int64_t recode_gaps_row(const Plan& P, const uint32_t* wire, uint32_t* out) {
    const int bl = bits_lvl(P.s);
    const int minmax = P.quantizer == QZ_MINMAX;
    int64_t in_at = 2 * (int64_t)P.nseg, out_at = 5 * (int64_t)P.nseg, bits = 0;
    for (int g = 0; g < P.nseg; ++g) {
        const int64_t n_el = P.off[g + 1] - P.off[g];
        const int64_t n = minmax ? P.kseg[g] : (int64_t)wire[2 * g];
        const int bi = bits_idx(n_el);
        const uint32_t* w_idx = wire + in_at;
        std::vector<uint32_t> idx(n), gaps;
        for (int64_t j = 0; j < n; ++j) idx[j] = get_bits(w_idx, j * bi, bi);
        for (int64_t j = 1; j < n; ++j) gaps.push_back(idx[j] - idx[j - 1] - 1u);
        int w = 0;
        int64_t x = 0;
        if (n >= 2) choose_width(gaps, bi, &w, &x);
        const uint32_t escape = w ? (uint32_t)((1ull << w) - 1ull) : 0u;
        out[5 * g] = wire[2 * g];
        out[5 * g + 1] = wire[2 * g + 1];
        out[5 * g + 2] = (uint32_t)w;
        out[5 * g + 3] = n ? idx[0] : 0u;
        out[5 * g + 4] = (uint32_t)x;
        const int64_t gw = n ? words_for(n - 1, w) : 0, ew = words_for(x, bi), iw = words_for(n, bi);
        int64_t e = 0;
        for (int64_t j = 0; j + 1 < n; ++j) {
            if (w == 0) continue;
            if (gaps[j] >= escape) {
                put_bits(out + out_at, j * w, w, escape);
                put_bits(out + out_at + gw, e * bi, bi, gaps[j]);
                ++e;
            } else {
                put_bits(out + out_at, j * w, w, gaps[j]);
            }
        }
        const int64_t rest = payload_words(n, bi, bl, P.quantizer) - iw;
        for (int64_t q = 0; q < rest; ++q) out[out_at + gw + ew + q] = wire[in_at + iw + q];
        bits += 64 + 6 + (n ? bi + (n - 1) * w + x * bi : 0) + n * (entry_bits(bi, bl, P.quantizer) - bi);
        in_at += iw + rest;
        out_at += gw + ew + rest;
    }
    return bits;
}

// gap-coded record -> plain record (the words of `wire` must be zero on entry)
void decode_gaps_row(const Plan& P, const uint32_t* packed, uint32_t* wire) {
    const int bl = bits_lvl(P.s);
    const int minmax = P.quantizer == QZ_MINMAX;
    int64_t in_at = 5 * (int64_t)P.nseg, out_at = 2 * (int64_t)P.nseg;
    for (int g = 0; g < P.nseg; ++g) {
        const int64_t n_el = P.off[g + 1] - P.off[g];
        const int64_t n = minmax ? P.kseg[g] : (int64_t)packed[5 * g];
        const int bi = bits_idx(n_el);
        const int w = (int)packed[5 * g + 2];
        const int64_t x = (int64_t)packed[5 * g + 4];
        const uint32_t escape = w ? (uint32_t)((1ull << w) - 1ull) : 0u;
        wire[2 * g] = packed[5 * g];
        wire[2 * g + 1] = packed[5 * g + 1];
        const int64_t gw = n ? words_for(n - 1, w) : 0, ew = words_for(x, bi), iw = words_for(n, bi);
        uint32_t at = packed[5 * g + 3];
        int64_t e = 0;
        for (int64_t j = 0; j < n; ++j) {
            if (j) {
                uint32_t gap = get_bits(packed + in_at, (j - 1) * w, w);
                if (w && gap == escape) gap = get_bits(packed + in_at + gw, (e++) * bi, bi);
                at = at + gap + 1u;
            }
            put_bits(wire + out_at, j * bi, bi, at);
        }
        const int64_t rest = payload_words(n, bi, bl, P.quantizer) - iw;
        for (int64_t q = 0; q < rest; ++q) wire[out_at + iw + q] = packed[in_at + gw + ew + q];
        in_at += gw + ew + rest;
        out_at += iw + rest;
    }
}

bool valid_plan(const Plan& P) {
    if (P.R < 1 || P.d < 1 || P.nseg < 1 || P.s < 1 || P.s > 65535) return false;
    if (P.quantizer == QZ_MINMAX && P.s < 2) return false;
    if (P.off[0] != 0 || P.off[P.nseg] != P.d) return false;
    for (int g = 0; g < P.nseg; ++g) {
        int64_t n = P.off[g + 1] - P.off[g];
        if (n < 1 || P.kseg[g] < 1 || P.kseg[g] > n) return false;
    }
    return true;
}

}  // namespace

extern "C" {

void qso_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}
uint32_t qso_philox_word(uint64_t seed, uint64_t round, uint32_t worker, uint64_t element,
                         uint32_t stream) {
    return philox_word(seed, round, worker, element, stream);
}
float qso_norm_l2(const float* v, int64_t n) { return norm_l2_exact(v, n); }
float qso_norm_l1(const float* v, int64_t n) { return norm_l1_exact(v, n); }
void qso_select_topk(const float* u, int64_t n, int64_t k, int mode, int64_t* idx_out) {
    select_topk(u, n, k, mode, idx_out);
}
void qso_select_randk(uint64_t seed, uint64_t round, uint32_t worker, int64_t lo, int64_t n,
                      int64_t k, int mode, int64_t* idx_out) {
    select_randk(seed, round, worker, lo, n, k, mode, idx_out);
}
int qso_qsgd_level(float u, float N, int s, uint32_t w) { return qsgd_level(u, N, s, w); }
int qso_minmax_level(float v, float lo, float hi, int s, uint32_t w) { return minmax_level(v, lo, hi, s, w); }
float qso_value_minmax(float lo, float hi, int s, int level) { return value_minmax(lo, hi, s, level); }
double qso_beta_qsgd(int64_t k, int s) { return beta_qsgd(k, s); }

int64_t qso_wire_words(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s,
                       int quantizer) {
    Plan P = {R, d, nseg, off, kseg, s, SP_TOPK, quantizer, 0};
    return valid_plan(P) ? wire_words(P) : (int64_t)ERR_ARG;
}

// Local step of Algorithm 1: xhat_r <- xhat_r - eta * grad_r (multiply, then
// subtract, each rounded to fp32).
void qso_local_step(int R, int64_t d, float* xw, const float* grad, float eta,
                    const uint8_t* mask) {
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        for (int64_t i = 0; i < d; ++i) {
            float step = eta * grad[(int64_t)r * d + i];
            xw[(int64_t)r * d + i] = xw[(int64_t)r * d + i] - step;
        }
    }
}

// Local step with momentum (Section 5.1: momentum 0.9 applied on the local
// iterations; the paper prints no formula, the heavy-ball form is taken):
//   v_r <- mu * v_r + grad_r ;  xhat_r <- xhat_r - eta * v_r
// every product and sum rounded to fp32 on its own.  mu = 0 is the plain step.
void qso_local_step_momentum(int R, int64_t d, float* xw, float* vel, const float* grad,
                             float eta, float mu, const uint8_t* mask) {
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        for (int64_t i = 0; i < d; ++i) {
            const int64_t p = (int64_t)r * d + i;
            float carried = mu * vel[p];
            float v = carried + grad[p];
            vel[p] = v;
            float step = eta * v;
            xw[p] = xw[p] - step;
        }
    }
}

// Worker half of a round for every worker in mask (NULL = all).  anchors NULL
// means the synchronous algorithm (anchor = x).  Optional outputs are laid out
// per worker: sel/lvl/sgn R x sum(kseg), norm/n R x nseg.
int qso_compress_feedback(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg,
                          int s, int sparsifier, int quantizer, uint64_t seed, uint64_t round,
                          const float* x, const float* xw, float* mem, const float* anchors,
                          const uint8_t* mask, uint32_t* wire, int64_t stride_words,
                          int64_t* bits_out, int mode, int nthreads, int64_t* sel_out,
                          int32_t* lvl_out, uint8_t* sgn_out, float* norm_out, int64_t* n_out) {
    Plan P = {R, d, nseg, off, kseg, s, sparsifier, quantizer, seed};
    if (!valid_plan(P)) return ERR_ARG;
    if (stride_words < wire_words(P)) return ERR_CAPACITY;
    int64_t K = 0;
    for (int g = 0; g < nseg; ++g) K += kseg[g];
    std::vector<int> status(R, ERR_OK);
    auto work = [&](int r) {
        if (mask && !mask[r]) return;
        const float* anchor = anchors ? anchors + (int64_t)r * d : x;
        status[r] = worker_compress(P, round, r, anchor, xw + (int64_t)r * d, mem + (int64_t)r * d,
                                    wire + (int64_t)r * stride_words, bits_out ? bits_out + r : 0,
                                    mode, sel_out ? sel_out + (int64_t)r * K : 0,
                                    lvl_out ? lvl_out + (int64_t)r * K : 0,
                                    sgn_out ? sgn_out + (int64_t)r * K : 0,
                                    norm_out ? norm_out + (int64_t)r * nseg : 0,
                                    n_out ? n_out + (int64_t)r * nseg : 0);
    };
    if (nthreads <= 1) {
        for (int r = 0; r < R; ++r) work(r);
    } else {
        for (int base = 0; base < R; base += nthreads) {
            std::vector<std::thread> pool;
            for (int r = base; r < R && r < base + nthreads; ++r) pool.emplace_back(work, r);
            for (auto& t : pool) t.join();
        }
    }
    for (int r = 0; r < R; ++r) if (status[r] != ERR_OK) return status[r];
    return ERR_OK;
}

// Worker half for one worker given by its id (the id enters the Philox counter), on that
// worker's own rows: used where only some workers of a large configuration are replayed.
int qso_compress_worker(int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s, int sparsifier,
                        int quantizer, uint64_t seed, uint64_t round, int worker, const float* anchor,
                        const float* xw_r, float* mem_r, uint32_t* wire, int64_t stride_words,
                        int64_t* bits_out, int mode) {
    Plan P = {worker + 1, d, nseg, off, kseg, s, sparsifier, quantizer, seed};
    if (worker < 0 || !valid_plan(P)) return ERR_ARG;
    if (stride_words < wire_words(P)) return ERR_CAPACITY;
    return worker_compress(P, round, worker, anchor, xw_r, mem_r, wire, bits_out, mode, 0, 0, 0, 0, 0);
}

// Master half: decode the records of the workers in mask from the wire words,
// accumulate in worker order, update x; the divisor is R whatever the mask.
int qso_unpack_accumulate(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg,
                          int s, int quantizer, float* x, const uint32_t* wire,
                          int64_t stride_words, const uint8_t* mask) {
    Plan P = {R, d, nseg, off, kseg, s, SP_TOPK, quantizer, 0};
    if (!valid_plan(P)) return ERR_ARG;
    std::vector<float> acc(d, 0.0f);
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        master_add_record(P, wire + (int64_t)r * stride_words, acc.data());
    }
    for (int64_t i = 0; i < d; ++i) x[i] = x[i] - acc[i] / (float)R;
    return ERR_OK;
}

int64_t qso_gap_words(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s,
                      int quantizer) {
    Plan P = {R, d, nseg, off, kseg, s, SP_TOPK, quantizer, 0};
    return valid_plan(P) ? gap_words(P) : (int64_t)ERR_ARG;
}

// Plain records -> gap-coded records for the workers in mask; rows of `out` must be zero.
int qso_recode_gaps(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s,
                    int quantizer, const uint32_t* wire, int64_t stride_words, const uint8_t* mask,
                    uint32_t* out, int64_t out_stride, int64_t* bits_out) {
    Plan P = {R, d, nseg, off, kseg, s, SP_TOPK, quantizer, 0};
    if (!valid_plan(P)) return ERR_ARG;
    if (stride_words < wire_words(P) || out_stride < gap_words(P)) return ERR_CAPACITY;
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        const int64_t bits = recode_gaps_row(P, wire + (int64_t)r * stride_words, out + (int64_t)r * out_stride);
        if (bits_out) bits_out[r] = bits;
    }
    return ERR_OK;
}

// Gap-coded records -> plain records; rows of `wire` must be zero.
int qso_decode_gaps(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s,
                    int quantizer, const uint32_t* packed, int64_t packed_stride, const uint8_t* mask,
                    uint32_t* wire, int64_t stride_words) {
    Plan P = {R, d, nseg, off, kseg, s, SP_TOPK, quantizer, 0};
    if (!valid_plan(P)) return ERR_ARG;
    if (stride_words < wire_words(P) || packed_stride < gap_words(P)) return ERR_CAPACITY;
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        decode_gaps_row(P, packed + (int64_t)r * packed_stride, wire + (int64_t)r * stride_words);
    }
    return ERR_OK;
}

// Broadcast: xhat_r <- x (and the anchor in the asynchronous algorithm) for the
// workers in mask.
void qso_broadcast(int R, int64_t d, const float* x, float* xw, float* anchors,
                   const uint8_t* mask) {
    for (int r = 0; r < R; ++r) {
        if (mask && !mask[r]) continue;
        for (int64_t i = 0; i < d; ++i) {
            xw[(int64_t)r * d + i] = x[i];
            if (anchors) anchors[(int64_t)r * d + i] = x[i];
        }
    }
}

// Whole round = the three calls above in order.
int qso_sync_round(int R, int64_t d, int nseg, const int64_t* off, const int64_t* kseg, int s,
                   int sparsifier, int quantizer, uint64_t seed, uint64_t round, float* x,
                   float* xw, float* mem, float* anchors, const uint8_t* mask, uint32_t* wire,
                   int64_t stride_words, int64_t* bits_out, int mode, int nthreads) {
    int rc = qso_compress_feedback(R, d, nseg, off, kseg, s, sparsifier, quantizer, seed, round, x,
                                   xw, mem, anchors, mask, wire, stride_words, bits_out, mode,
                                   nthreads, 0, 0, 0, 0, 0);
    if (rc != ERR_OK) return rc;
    rc = qso_unpack_accumulate(R, d, nseg, off, kseg, s, quantizer, x, wire, stride_words, mask);
    if (rc != ERR_OK) return rc;
    qso_broadcast(R, d, x, xw, anchors, mask);
    return ERR_OK;
}

}  // extern "C"
