// Gap-coded records: a second form of a worker's record in which a segment's k indices travel as
// the first index and the gaps between successive indices in short fields; the few gaps too large
// for a field travel in a stream of exceptions.  The paper counts what the workers transmit in bits
// (Section 5) and leaves the coding of the indices open; with k indices spread over d coordinates a
// gap takes about log2(d/k) + 1 bits against log2(d) for the index itself.
//
// Row of one worker:
//   directory: nseg entries of five words (n, norm bits, w, first index, x); the min/max quantizer
//              keeps (min, max) in the first two words, n = k;
//   per segment: n - 1 gap fields (i_j - i_(j-1) - 1) of w bits, LSB first, padded to a word; for
//              w >= 1 the value E = 2^w - 1 is an escape: the gap is the next of the x exception
//              fields of b_idx bits that follow, padded to a word; then the streams that follow the
//              indices in the plain record, word for word.
// w is the width in 0 .. b_idx that makes (n - 1) w + x(w) b_idx smallest (the smallest on a tie;
// w = 0 only when every gap is 0).
//
// Both directions are a handful of small launches over (worker, segment) units; nothing here is on
// the path of a fused round.
#include "qs_kernels.h"

namespace qs {

namespace {

constexpr int GT = 256;                  // threads per block
constexpr uint32_t GCH = 1024;           // gap fields per chunk of the decoder's two-level sums

struct GapArgs {
    Plan P;
    Active act;
    const uint32_t* in;
    long long in_stride;
    uint32_t* out;
    long long out_stride;
    long long* bits_out;
    uint32_t row_chunks;                 // chunk sums reserved per worker
    int which;                           // the array of chunk sums a scan works on; the direction of a count
};

constexpr int GBINS = 33;                // gaps by the bit length of gap + 1 (1 .. 32)

// per-unit table: seven arrays of MAX_R * nseg words, then GBINS counts per unit
struct UnitTab {
    uint32_t *n, *plain_off, *packed_off, *w, *first, *cbase, *x, *hist;
};
__device__ __forceinline__ UnitTab unit_tab(const Plan& P) {
    const size_t m = (size_t)MAX_R * P.nseg;
    UnitTab t = {P.gap_unit,         P.gap_unit + m,     P.gap_unit + 2 * m, P.gap_unit + 3 * m,
                 P.gap_unit + 4 * m, P.gap_unit + 5 * m, P.gap_unit + 6 * m, P.gap_unit + 7 * m};
    return t;
}
// the two arrays of chunk sums: escapes in front of a chunk, index distance in front of a chunk
__device__ __forceinline__ uint32_t* chunk_sums(const GapArgs& a, int which) {
    return a.P.gap_csum + (size_t)which * MAX_R * a.row_chunks;
}
__device__ __forceinline__ uint32_t escape_of(uint32_t w) { return w >= 32u ? 0xffffffffu : (1u << w) - 1u; }

// field of `width` bits (0 .. 32) at bit `pos` of a stream; never reads a word the field does not touch
__device__ __forceinline__ uint32_t get_field(const uint32_t* s, uint64_t pos, uint32_t width) {
    if (width == 0u) return 0u;
    const uint64_t q = pos >> 5;
    const uint32_t sh = (uint32_t)(pos & 31u);
    uint64_t v = s[q] >> sh;
    if (sh + width > 32u) v |= (uint64_t)s[q + 1] << (32u - sh);
    return (uint32_t)(v & ((width >= 32u) ? 0xffffffffull : ((1ull << width) - 1ull)));
}

__device__ __forceinline__ void or_field(uint32_t* s, uint64_t pos, uint32_t width, uint32_t val) {
    const uint64_t q = pos >> 5;
    const uint32_t sh = (uint32_t)(pos & 31u);
    atomicOr(s + q, val << sh);
    if (sh + width > 32u) atomicOr(s + q + 1, val >> (32u - sh));
}

// exclusive scan of one value per thread over the block; *total gets the sum
__device__ uint32_t block_scan(uint32_t v, uint32_t* sh, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    __syncthreads();
    if (lane == 31) sh[warp] = inc;
    __syncthreads();
    uint32_t before = 0, all = 0;
    for (int k = 0; k < GT / 32; ++k) {
        if (k < warp) before += sh[k];
        all += sh[k];
    }
    *total = all;
    return before + inc - v;
}

// Per worker: three running sums over its segments at once (a, b, c per segment), written as
// exclusive prefixes.  Threads take contiguous ranges of segments.
template <class F, class G>
__device__ void row_prefixes(uint32_t nseg, uint32_t* sh, F item, G store) {
    const uint32_t per = (nseg + GT - 1) / GT;
    const uint32_t g0 = threadIdx.x * per, g1 = g0 + per < nseg ? g0 + per : nseg;
    uint32_t a = 0, b = 0, c = 0;
    for (uint32_t g = g0; g < g1; ++g) {
        uint32_t x, y, z;
        item(g, &x, &y, &z);
        a += x; b += y; c += z;
    }
    uint32_t ta, tb, tc;
    uint32_t pa = block_scan(a, sh, &ta);
    uint32_t pb = block_scan(b, sh, &tb);
    uint32_t pc = block_scan(c, sh, &tc);
    for (uint32_t g = g0; g < g1; ++g) {
        uint32_t x, y, z;
        item(g, &x, &y, &z);
        store(g, pa, pb, pc);
        pa += x; pb += y; pc += z;
    }
}

__device__ __forceinline__ uint32_t count_of(const Plan& P, const uint32_t* dir_word, uint32_t g) {
    const uint32_t k = P.kseg[g];
    if (P.qz == QS_MINMAX) return k;
    const uint32_t n = *dir_word;
    return n < k ? n : k;                 // (a count above k cannot come from a worker: clipped, the words stay in bounds)
}


// ---- plain -> gap-coded

// where each segment's streams start in the plain row; the counts of gaps start at 0
__global__ void __launch_bounds__(GT) gap_plain_layout(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t slot = blockIdx.x, nseg = (uint32_t)P.nseg;
    const uint32_t* row = a.in + (size_t)a.act.r[slot] * a.in_stride;
    const UnitTab t = unit_tab(P);
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        const uint32_t n = count_of(P, row + 2 * g, g);
        *x = streams_words(n, P.bidx[g], (uint32_t)P.bl, P.qz);
        *y = n >= 2u ? (n - 1u + GCH - 1u) / GCH : 0u;
        *z = 0;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t pb, uint32_t) {
        const size_t u = (size_t)slot * nseg + g;
        t.n[u] = count_of(P, row + 2 * g, g);
        t.plain_off[u] = 2u * nseg + pa;
        t.cbase[u] = slot * a.row_chunks + pb;
        for (int b = 0; b < GBINS; ++b) t.hist[u * GBINS + b] = 0u;
    };
    row_prefixes(nseg, sh, item, store);
}

// gaps of every unit counted by the bit length of gap + 1
__global__ void __launch_bounds__(GT) gap_histogram(const GapArgs a) {
    __shared__ uint32_t bins[GBINS];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], bi = P.bidx[g];
    if ((uint64_t)blockIdx.y * GT + 1u >= n) return;                 // nothing for this block (uniform)
    const uint32_t* idx = a.in + (size_t)a.act.r[slot] * a.in_stride + t.plain_off[u];
    if (threadIdx.x < GBINS) bins[threadIdx.x] = 0u;
    __syncthreads();
    for (uint64_t j = 1 + (uint64_t)blockIdx.y * GT + threadIdx.x; j < n; j += (uint64_t)gridDim.y * GT) {
        const uint32_t gap = get_field(idx, j * bi, bi) - get_field(idx, (j - 1) * bi, bi) - 1u;
        atomicAdd(&bins[32 - __clz(gap + 1u)], 1u);                  // (gap + 1 < 2^32: a gap is shorter than its segment)
    }
    __syncthreads();
    if (threadIdx.x < GBINS && bins[threadIdx.x]) atomicAdd(&t.hist[(size_t)u * GBINS + threadIdx.x], bins[threadIdx.x]);
}

// the width that makes a segment's fields and exceptions smallest: cost (n - 1) w + x(w) b_idx with
// x(w) = gaps >= 2^w - 1 = gaps whose gap + 1 is longer than w bits
__device__ void choose_width(const uint32_t* hist, uint32_t n, uint32_t bi, uint32_t* w_out, uint32_t* x_out) {
    uint32_t best_w = bi, best_x = 0;
    uint64_t best = (uint64_t)(n - 1u) * bi;
    uint32_t longer = 0;                                             // gaps with gap + 1 longer than w bits
    for (int w = 32; w >= 0; --w) {
        const uint32_t above_one_bit = longer;                       // (read at w = 0: gaps other than 0)
        if (w < 32) longer += hist[w + 1];
        if ((uint32_t)w >= bi) continue;
        if (w == 0 && above_one_bit != 0u) continue;                 // no fields at all needs every gap to be 0
        const uint64_t cost = (uint64_t)(n - 1u) * (uint32_t)w + (uint64_t)(w ? longer : 0u) * bi;
        if (cost <= best) { best = cost; best_w = (uint32_t)w; best_x = w ? longer : 0u; }
    }
    *w_out = best_w;
    *x_out = best_x;
}

// widths, exceptions, places in the packed row, its directory and its size in bits
__global__ void __launch_bounds__(GT) gap_packed_layout(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    __shared__ unsigned long long sh_bits;
    const Plan& P = a.P;
    const uint32_t slot = blockIdx.x, nseg = (uint32_t)P.nseg;
    const uint32_t* row = a.in + (size_t)a.act.r[slot] * a.in_stride;
    uint32_t* out = a.out + (size_t)a.act.r[slot] * a.out_stride;
    const UnitTab t = unit_tab(P);
    if (threadIdx.x == 0) sh_bits = 0ull;
    __syncthreads();
    unsigned long long bits = 0;
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        const size_t u = (size_t)slot * nseg + g;
        const uint32_t n = t.n[u], bi = P.bidx[g];
        uint32_t w = 0, xc = 0;
        if (n >= 2u) choose_width(t.hist + u * GBINS, n, bi, &w, &xc);
        *x = (n ? words_for(n - 1u, w) : 0u) + words_for(xc, bi) + streams_words(n, bi, (uint32_t)P.bl, P.qz) - words_for(n, bi);
        *y = 0; *z = 0;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t, uint32_t) {
        const size_t u = (size_t)slot * nseg + g;
        const uint32_t n = t.n[u], bi = P.bidx[g];
        uint32_t w = 0, xc = 0;
        if (n >= 2u) choose_width(t.hist + u * GBINS, n, bi, &w, &xc);
        const uint32_t first = n ? get_field(row + t.plain_off[u], 0, bi) : 0u;
        t.packed_off[u] = 5u * nseg + pa;
        t.w[u] = w;
        t.x[u] = xc;
        out[5 * g] = row[2 * g];
        out[5 * g + 1] = row[2 * g + 1];
        out[5 * g + 2] = w;
        out[5 * g + 3] = first;
        out[5 * g + 4] = xc;
        bits += 64ull + 6ull + (n ? (unsigned long long)bi + (unsigned long long)(n - 1u) * w + (unsigned long long)xc * bi : 0ull) +
                (unsigned long long)n * (entry_bits(bi, (uint32_t)P.bl, P.qz) - bi);
    };
    row_prefixes(nseg, sh, item, store);
    atomicAdd(&sh_bits, bits);
    __syncthreads();
    if (threadIdx.x == 0 && a.bits_out) a.bits_out[a.act.r[slot]] = (long long)sh_bits;
}

// Escapes per chunk of GCH fields.  which = 0: counted from the plain record's indices (a gap at or
// above the escape value); which = 1: counted from the packed fields (a field equal to it).
__global__ void __launch_bounds__(GT) gap_escape_counts(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], w = t.w[u], bi = P.bidx[g];
    if (n < 2u) return;
    const uint32_t esc = escape_of(w);
    const uint32_t* src = a.in + (size_t)a.act.r[slot] * a.in_stride + (a.which ? t.packed_off[u] : t.plain_off[u]);
    uint32_t* cs = chunk_sums(a, 0) + t.cbase[u];
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        uint32_t s = 0;
        for (uint32_t f = c * GCH + threadIdx.x; f < n - 1u && f < (c + 1u) * GCH && w; f += GT) {
            if (a.which) s += get_field(src, (uint64_t)f * w, w) == esc;
            else s += get_field(src, (uint64_t)(f + 1u) * bi, bi) - get_field(src, (uint64_t)f * bi, bi) - 1u >= esc;
        }
        uint32_t total;
        block_scan(s, sh, &total);
        if (threadIdx.x == 0) cs[c] = total;
        __syncthreads();
    }
}

// the chunk sums of a unit become the offsets of its chunks (array a.which)
__global__ void __launch_bounds__(GT) gap_chunk_scan(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u];
    if (n < 2u) return;
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    uint32_t* cs = chunk_sums(a, a.which) + t.cbase[u];
    uint32_t carry = 0;
    for (uint32_t c0 = 0; c0 < nchunk; c0 += GT) {
        const uint32_t c = c0 + threadIdx.x;
        const uint32_t v = c < nchunk ? cs[c] : 0u;
        uint32_t total;
        const uint32_t ex = block_scan(v, sh, &total);
        if (c < nchunk) cs[c] = carry + ex;
        carry += total;
        __syncthreads();
    }
}

// the gap fields (one output word per thread), the other streams copied, then the exceptions
__global__ void __launch_bounds__(GT) gap_write(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], bi = P.bidx[g], w = t.w[u], xc = t.x[u];
    const uint32_t esc = escape_of(w);
    const uint32_t* src = a.in + (size_t)a.act.r[slot] * a.in_stride + t.plain_off[u];
    uint32_t* dst = a.out + (size_t)a.act.r[slot] * a.out_stride + t.packed_off[u];
    const uint32_t gw = n ? words_for(n - 1u, w) : 0u, ew = words_for(xc, bi), iw = words_for(n, bi);
    const uint32_t rest = streams_words(n, bi, (uint32_t)P.bl, P.qz) - iw;
    for (uint64_t q = (uint64_t)blockIdx.y * GT + threadIdx.x; q < (uint64_t)gw + rest; q += (uint64_t)gridDim.y * GT) {
        if (q >= gw) { dst[ew + q] = src[iw + (q - gw)]; continue; }
        // fields that touch bits 32 q .. 32 q + 31 (w >= 1 here: no gap words otherwise)
        const uint64_t b0 = q * 32ull;
        uint64_t f = b0 / w;
        uint32_t word = 0;
        for (; f + 1 < n && f * w < b0 + 32ull; ++f) {
            uint64_t gap = get_field(src, (f + 1) * bi, bi) - get_field(src, f * bi, bi) - 1u;
            if (gap > esc) gap = esc;
            const long long p = (long long)(f * w) - (long long)b0;
            word |= (uint32_t)(p >= 0 ? gap << p : gap >> (-p));
        }
        dst[q] = word;
    }
    if (xc == 0u || n < 2u) return;
    // exceptions, in the order of their fields: rank = escapes in front of the chunk + those in front inside it
    // (the exception words are zero before this kernel)
    const uint32_t* before = chunk_sums(a, 0) + t.cbase[u];
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    constexpr uint32_t PER = GCH / GT;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        const uint32_t f0 = c * GCH + threadIdx.x * PER;
        uint32_t gap[PER], mine = 0;
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) {
            gap[i] = f0 + i < n - 1u ? get_field(src, (uint64_t)(f0 + i + 1u) * bi, bi) - get_field(src, (uint64_t)(f0 + i) * bi, bi) - 1u : 0u;
            mine += (f0 + i < n - 1u && gap[i] >= esc) ? 1u : 0u;
        }
        uint32_t total;
        uint32_t rank = before[c] + block_scan(mine, sh, &total);
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i)
            if (f0 + i < n - 1u && gap[i] >= esc) or_field(dst + gw, (uint64_t)(rank++) * bi, bi, gap[i]);
        __syncthreads();
    }
}

// ---- gap-coded -> plain

// places of every segment in both rows, the plain directory, where its chunk sums live
__global__ void __launch_bounds__(GT) gap_decode_layout(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t slot = blockIdx.x, nseg = (uint32_t)P.nseg;
    const uint32_t* row = a.in + (size_t)a.act.r[slot] * a.in_stride;          // packed
    uint32_t* out = a.out + (size_t)a.act.r[slot] * a.out_stride;              // plain
    const UnitTab t = unit_tab(P);
    // what a sender can have written: a width up to b_idx, no more exceptions than fields; clipped otherwise
    auto width = [&](uint32_t g) { const uint32_t w = row[5 * g + 2]; return w < P.bidx[g] ? w : (uint32_t)P.bidx[g]; };
    auto exceptions = [&](uint32_t g, uint32_t n) {
        const uint32_t x = row[5 * g + 4], most = (n >= 2u && width(g)) ? n - 1u : 0u;
        return x < most ? x : most;
    };
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        const uint32_t n = count_of(P, row + 5 * g, g), bi = P.bidx[g];
        const uint32_t all = streams_words(n, bi, (uint32_t)P.bl, P.qz);
        *x = (n ? words_for(n - 1u, width(g)) : 0u) + words_for(exceptions(g, n), bi) + all - words_for(n, bi);
        *y = all;
        *z = n >= 2u ? (n - 1u + GCH - 1u) / GCH : 0u;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t pb, uint32_t pc) {
        const size_t u = (size_t)slot * nseg + g;
        const uint32_t n = count_of(P, row + 5 * g, g);
        t.n[u] = n;
        t.packed_off[u] = 5u * nseg + pa;
        t.plain_off[u] = 2u * nseg + pb;
        t.cbase[u] = slot * a.row_chunks + pc;
        t.w[u] = width(g);
        t.x[u] = exceptions(g, n);
        const uint32_t span = P.seg_off[g + 1] - P.seg_off[g];
        t.first[u] = row[5 * g + 3] < span ? row[5 * g + 3] : span - 1u;
        out[2 * g] = row[5 * g];
        out[2 * g + 1] = row[5 * g + 1];
    };
    row_prefixes(nseg, sh, item, store);
}

// The PER consecutive gaps (+ 1) a thread holds of chunk c: fields, with the escapes replaced by
// their exceptions (rank = escapes in front of the chunk + in front inside it; a rank beyond the
// exceptions the directory announces reads the last one: the words stay in bounds).
template <uint32_t PER>
__device__ __forceinline__ void chunk_steps(const uint32_t* fields, const uint32_t* exc, uint32_t escapes_before, uint32_t n,
                                            uint32_t w, uint32_t bi, uint32_t xc, uint32_t c, uint32_t* sh, uint32_t step[PER]) {
    const uint32_t esc = escape_of(w);
    const uint32_t f0 = c * GCH + threadIdx.x * PER;
    uint32_t mine = 0;
#pragma unroll
    for (uint32_t i = 0; i < PER; ++i) {
        step[i] = f0 + i < n - 1u ? get_field(fields, (uint64_t)(f0 + i) * w, w) : 0u;
        mine += (f0 + i < n - 1u && w && xc && step[i] == esc) ? 1u : 0u;
    }
    uint32_t total;
    uint32_t rank = escapes_before + block_scan(mine, sh, &total);
#pragma unroll
    for (uint32_t i = 0; i < PER; ++i) {
        if (f0 + i >= n - 1u) { step[i] = 0u; continue; }
        if (w && xc && step[i] == esc) {
            const uint32_t at = rank < xc ? rank : xc - 1u;
            step[i] = get_field(exc, (uint64_t)at * bi, bi);
            ++rank;
        }
        step[i] += 1u;
    }
}

// index distance covered by each chunk of GCH fields
__global__ void __launch_bounds__(GT) gap_chunk_sums(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], w = t.w[u], bi = P.bidx[g], xc = t.x[u];
    if (n < 2u) return;
    const uint32_t* fields = a.in + (size_t)a.act.r[slot] * a.in_stride + t.packed_off[u];
    const uint32_t* exc = fields + words_for(n - 1u, w);
    const uint32_t* before = chunk_sums(a, 0) + t.cbase[u];
    uint32_t* cs = chunk_sums(a, 1) + t.cbase[u];
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    constexpr uint32_t PER = GCH / GT;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        uint32_t step[PER], s = 0;
        chunk_steps<PER>(fields, exc, before[c], n, w, bi, xc, c, sh, step);
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) s += step[i];
        uint32_t total;
        block_scan(s, sh, &total);
        if (threadIdx.x == 0) cs[c] = total;
        __syncthreads();
    }
}

// indices from the gaps (sums inside the chunk on top of the chunk's offset), the other streams
// copied; the plain row is zero before this kernel
__global__ void __launch_bounds__(GT) gap_expand(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], w = t.w[u], bi = P.bidx[g], xc = t.x[u];
    if (n == 0u) return;
    const uint32_t* fields = a.in + (size_t)a.act.r[slot] * a.in_stride + t.packed_off[u];
    uint32_t* dst = a.out + (size_t)a.act.r[slot] * a.out_stride + t.plain_off[u];
    const uint32_t gw = words_for(n - 1u, w), ew = words_for(xc, bi), iw = words_for(n, bi);
    const uint32_t* exc = fields + gw;
    const uint32_t rest = streams_words(n, bi, (uint32_t)P.bl, P.qz) - iw;
    const uint32_t mask = bi >= 32u ? 0xffffffffu : (1u << bi) - 1u;
    for (uint64_t q = (uint64_t)blockIdx.y * GT + threadIdx.x; q < rest; q += (uint64_t)gridDim.y * GT) dst[iw + q] = fields[gw + ew + q];
    if (blockIdx.y == 0 && threadIdx.x == 0) or_field(dst, 0, bi, t.first[u] & mask);
    if (n < 2u) return;
    const uint32_t* before = chunk_sums(a, 0) + t.cbase[u];
    const uint32_t* offset = chunk_sums(a, 1) + t.cbase[u];
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    constexpr uint32_t PER = GCH / GT;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        const uint32_t f0 = c * GCH + threadIdx.x * PER;
        uint32_t step[PER], s = 0;
        chunk_steps<PER>(fields, exc, before[c], n, w, bi, xc, c, sh, step);
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) s += step[i];
        uint32_t total;
        uint32_t at = t.first[u] + offset[c] + block_scan(s, sh, &total);
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) {
            at += step[i];
            if (f0 + i < n - 1u) or_field(dst, (uint64_t)(f0 + i + 1u) * bi, bi, at & mask);   // field f is the gap in front of entry f + 1
        }
        __syncthreads();
    }
}

uint32_t y_blocks(uint64_t items) {
    const uint64_t y = (items + GT - 1) / GT;
    return (uint32_t)(y < 1 ? 1 : (y > 4096 ? 4096 : y));
}
uint32_t y_chunks(uint32_t longest_k) {
    const uint32_t c = (longest_k + GCH - 1) / GCH;
    return c < 1 ? 1 : (c > 4096 ? 4096 : c);
}

}  // namespace

uint32_t gap_chunk(void) { return GCH; }
uint32_t gap_unit_words(void) { return 7u + (uint32_t)GBINS; }

cudaError_t launch_recode_gaps(const Plan& P, const Active& act, const uint32_t* wire, long long stride, uint32_t* out,
                               long long out_stride, long long* bits_out, uint32_t longest_k, uint32_t most_words,
                               uint32_t row_chunks, cudaStream_t st) {
    GapArgs a = {P, act, wire, stride, out, out_stride, bits_out, row_chunks, 0};
    const uint32_t units = (uint32_t)act.n * (uint32_t)P.nseg;
    gap_plain_layout<<<act.n, GT, 0, st>>>(a);
    gap_histogram<<<dim3(units, y_blocks(longest_k)), GT, 0, st>>>(a);
    gap_packed_layout<<<act.n, GT, 0, st>>>(a);
    gap_escape_counts<<<dim3(units, y_chunks(longest_k)), GT, 0, st>>>(a);
    gap_chunk_scan<<<units, GT, 0, st>>>(a);
    gap_write<<<dim3(units, y_blocks(most_words)), GT, 0, st>>>(a);
    return cudaPeekAtLastError();
}

cudaError_t launch_decode_gaps(const Plan& P, const Active& act, const uint32_t* packed, long long packed_stride,
                               uint32_t* wire, long long stride, uint32_t longest_k, uint32_t most_words,
                               uint32_t row_chunks, cudaStream_t st) {
    GapArgs a = {P, act, packed, packed_stride, wire, stride, nullptr, row_chunks, 1};
    const uint32_t units = (uint32_t)act.n * (uint32_t)P.nseg;
    gap_decode_layout<<<act.n, GT, 0, st>>>(a);
    gap_escape_counts<<<dim3(units, y_chunks(longest_k)), GT, 0, st>>>(a);      // which = 1: from the packed fields
    a.which = 0;
    gap_chunk_scan<<<units, GT, 0, st>>>(a);
    gap_chunk_sums<<<dim3(units, y_chunks(longest_k)), GT, 0, st>>>(a);
    a.which = 1;
    gap_chunk_scan<<<units, GT, 0, st>>>(a);
    gap_expand<<<dim3(units, y_blocks(most_words > longest_k / 4 ? most_words : longest_k / 4)), GT, 0, st>>>(a);
    return cudaPeekAtLastError();
}

}  // namespace qs
