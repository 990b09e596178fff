// Gap-coded records: a second form of a worker's record in which a segment's k indices travel as
// the first index and the gaps between successive indices, in fields as wide as the segment's
// largest gap needs.  The paper counts what the workers transmit in bits (Section 5) and leaves the
// coding of the indices open; with k indices spread over d coordinates a gap takes about
// log2(d/k) + log2(ln k) bits against log2(d) for the index itself.
//
// Row of one worker:
//   directory: nseg entries of four words (n, norm bits, w, first index); the min/max quantizer
//              keeps (min, max) in the first two words, n = k;
//   per segment: n - 1 gap fields (i_j - i_(j-1) - 1) of w bits, LSB first, padded to a word; then
//              the streams that follow the indices in the plain record, word for word.
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
};

// per-unit table: six arrays of MAX_R * nseg words
struct UnitTab {
    uint32_t *n, *plain_off, *packed_off, *w, *first, *cbase;
};
__device__ __forceinline__ UnitTab unit_tab(const Plan& P) {
    const size_t m = (size_t)MAX_R * P.nseg;
    UnitTab t = {P.gap_unit, P.gap_unit + m, P.gap_unit + 2 * m, P.gap_unit + 3 * m, P.gap_unit + 4 * m, P.gap_unit + 5 * m};
    return t;
}

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

// where each segment's streams start in the plain row; the widest gap starts at 0
__global__ void __launch_bounds__(GT) gap_plain_layout(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t slot = blockIdx.x, nseg = (uint32_t)P.nseg;
    const uint32_t* row = a.in + (size_t)a.act.r[slot] * a.in_stride;
    const UnitTab t = unit_tab(P);
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        *x = streams_words(count_of(P, row + 2 * g, g), P.bidx[g], (uint32_t)P.bl, P.qz);
        *y = 0; *z = 0;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t, uint32_t) {
        const size_t u = (size_t)slot * nseg + g;
        t.n[u] = count_of(P, row + 2 * g, g);
        t.plain_off[u] = 2u * nseg + pa;
        t.w[u] = 0u;
    };
    row_prefixes(nseg, sh, item, store);
}

// the widest gap of every unit
__global__ void __launch_bounds__(GT) gap_widest(const GapArgs a) {
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], bi = P.bidx[g];
    const uint32_t* idx = a.in + (size_t)a.act.r[slot] * a.in_stride + t.plain_off[u];
    uint32_t widest = 0;
    for (uint64_t j = 1 + (uint64_t)blockIdx.y * GT + threadIdx.x; j < n; j += (uint64_t)gridDim.y * GT) {
        const uint32_t gap = get_field(idx, j * bi, bi) - get_field(idx, (j - 1) * bi, bi) - 1u;
        widest = gap > widest ? gap : widest;
    }
    widest = __reduce_max_sync(0xffffffffu, widest);
    if ((threadIdx.x & 31) == 0 && widest) atomicMax(&t.w[u], widest);
}

// widths, places in the packed row, its directory and its size in bits
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
    auto width = [&](size_t u) { return 32u - (uint32_t)__clz(t.w[u]); };      // t.w still holds the widest gap
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        const size_t u = (size_t)slot * nseg + g;
        const uint32_t n = t.n[u], bi = P.bidx[g];
        *x = (n ? words_for(n - 1u, width(u)) : 0u) + streams_words(n, bi, (uint32_t)P.bl, P.qz) - words_for(n, bi);
        *y = 0; *z = 0;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t, uint32_t) {
        const size_t u = (size_t)slot * nseg + g;
        const uint32_t n = t.n[u], bi = P.bidx[g], w = width(u);
        const uint32_t first = n ? get_field(row + t.plain_off[u], 0, bi) : 0u;
        t.packed_off[u] = 4u * nseg + pa;
        t.first[u] = w;                   // (the width, kept beside the widest gap until every thread is done with it)
        out[4 * g] = row[2 * g];
        out[4 * g + 1] = row[2 * g + 1];
        out[4 * g + 2] = w;
        out[4 * g + 3] = first;
        bits += 64ull + 6ull + (n ? (unsigned long long)bi + (unsigned long long)(n - 1u) * w : 0ull) +
                (unsigned long long)n * (entry_bits(bi, (uint32_t)P.bl, P.qz) - bi);
    };
    row_prefixes(nseg, sh, item, store);
    atomicAdd(&sh_bits, bits);
    __syncthreads();
    // the widths take the place of the widest gaps
    for (uint32_t g = threadIdx.x; g < nseg; g += GT) t.w[(size_t)slot * nseg + g] = t.first[(size_t)slot * nseg + g];
    if (threadIdx.x == 0 && a.bits_out) a.bits_out[a.act.r[slot]] = (long long)sh_bits;
}

// the gap stream, one output word per thread, and the other streams copied
__global__ void __launch_bounds__(GT) gap_write(const GapArgs a) {
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], bi = P.bidx[g], w = t.w[u];
    const uint32_t* src = a.in + (size_t)a.act.r[slot] * a.in_stride + t.plain_off[u];
    uint32_t* dst = a.out + (size_t)a.act.r[slot] * a.out_stride + t.packed_off[u];
    const uint32_t gw = n ? words_for(n - 1u, w) : 0u, iw = words_for(n, bi);
    const uint32_t rest = streams_words(n, bi, (uint32_t)P.bl, P.qz) - iw;
    for (uint64_t q = (uint64_t)blockIdx.y * GT + threadIdx.x; q < (uint64_t)gw + rest; q += (uint64_t)gridDim.y * GT) {
        if (q >= gw) { dst[q] = src[iw + (q - gw)]; continue; }
        // fields that touch bits 32 q .. 32 q + 31 (w >= 1 here: no gap words otherwise)
        const uint64_t b0 = q * 32ull;
        uint64_t f = b0 / w;
        uint32_t word = 0;
        for (; f + 1 < n && f * w < b0 + 32ull; ++f) {
            const uint64_t gap = get_field(src, (f + 1) * bi, bi) - get_field(src, f * bi, bi) - 1u;
            const long long p = (long long)(f * w) - (long long)b0;
            word |= (uint32_t)(p >= 0 ? gap << p : gap >> (-p));
        }
        dst[q] = word;
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
    auto width = [&](uint32_t g) { const uint32_t w = row[4 * g + 2]; return w < P.bidx[g] ? w : (uint32_t)P.bidx[g]; };   // (a gap is shorter than its segment)
    auto item = [&](uint32_t g, uint32_t* x, uint32_t* y, uint32_t* z) {
        const uint32_t n = count_of(P, row + 4 * g, g), bi = P.bidx[g];
        const uint32_t all = streams_words(n, bi, (uint32_t)P.bl, P.qz);
        *x = (n ? words_for(n - 1u, width(g)) : 0u) + all - words_for(n, bi);
        *y = all;
        *z = n ? (n - 1u + GCH - 1u) / GCH : 0u;
    };
    auto store = [&](uint32_t g, uint32_t pa, uint32_t pb, uint32_t pc) {
        const size_t u = (size_t)slot * nseg + g;
        t.n[u] = count_of(P, row + 4 * g, g);
        t.packed_off[u] = 4u * nseg + pa;
        t.plain_off[u] = 2u * nseg + pb;
        t.cbase[u] = slot * a.row_chunks + pc;
        t.w[u] = width(g);
        const uint32_t span = P.seg_off[g + 1] - P.seg_off[g];
        t.first[u] = row[4 * g + 3] < span ? row[4 * g + 3] : span - 1u;
        out[2 * g] = row[4 * g];
        out[2 * g + 1] = row[4 * g + 1];
    };
    row_prefixes(nseg, sh, item, store);
}

// sum of (gap + 1) over each chunk of GCH fields
__global__ void __launch_bounds__(GT) gap_chunk_sums(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], w = t.w[u];
    if (n < 2u) return;
    const uint32_t* gaps = a.in + (size_t)a.act.r[slot] * a.in_stride + t.packed_off[u];
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        uint32_t s = 0;
        for (uint32_t f = c * GCH + threadIdx.x; f < n - 1u && f < (c + 1u) * GCH; f += GT) s += get_field(gaps, (uint64_t)f * w, w) + 1u;
        uint32_t total;
        block_scan(s, sh, &total);
        if (threadIdx.x == 0) P.gap_csum[t.cbase[u] + c] = total;
        __syncthreads();
    }
}

// the chunk sums of a unit become the offsets of its chunks
__global__ void __launch_bounds__(GT) gap_chunk_scan(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u];
    if (n < 2u) return;
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    uint32_t* cs = P.gap_csum + t.cbase[u];
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

// indices from the gaps (four fields a thread, sums inside the chunk), the other streams copied;
// the plain row is zero before this kernel
__global__ void __launch_bounds__(GT) gap_expand(const GapArgs a) {
    __shared__ uint32_t sh[GT / 32];
    const Plan& P = a.P;
    const uint32_t u = blockIdx.x, slot = u / (uint32_t)P.nseg, g = u % (uint32_t)P.nseg;
    const UnitTab t = unit_tab(P);
    const uint32_t n = t.n[u], w = t.w[u], bi = P.bidx[g];
    if (n == 0u) return;
    const uint32_t* src = a.in + (size_t)a.act.r[slot] * a.in_stride + t.packed_off[u];
    uint32_t* dst = a.out + (size_t)a.act.r[slot] * a.out_stride + t.plain_off[u];
    const uint32_t gw = words_for(n - 1u, w), iw = words_for(n, bi);
    const uint32_t rest = streams_words(n, bi, (uint32_t)P.bl, P.qz) - iw;
    const uint32_t mask = bi >= 32u ? 0xffffffffu : (1u << bi) - 1u;
    for (uint64_t q = (uint64_t)blockIdx.y * GT + threadIdx.x; q < rest; q += (uint64_t)gridDim.y * GT) dst[iw + q] = src[gw + q];
    if (blockIdx.y == 0 && threadIdx.x == 0) or_field(dst, 0, bi, t.first[u] & mask);
    const uint32_t nchunk = (n - 1u + GCH - 1u) / GCH;
    constexpr uint32_t PER = GCH / GT;
    for (uint32_t c = blockIdx.y; c < nchunk; c += gridDim.y) {
        const uint32_t f0 = c * GCH + threadIdx.x * PER;
        uint32_t step[PER], s = 0;
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) {
            step[i] = f0 + i < n - 1u ? get_field(src, (uint64_t)(f0 + i) * w, w) + 1u : 0u;
            s += step[i];
        }
        uint32_t total;
        uint32_t at = t.first[u] + P.gap_csum[t.cbase[u] + c] + block_scan(s, sh, &total);
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

}  // namespace

uint32_t gap_chunk(void) { return GCH; }

cudaError_t launch_recode_gaps(const Plan& P, const Active& act, const uint32_t* wire, long long stride, uint32_t* out,
                               long long out_stride, long long* bits_out, uint32_t longest_k, uint32_t most_words,
                               cudaStream_t st) {
    GapArgs a = {P, act, wire, stride, out, out_stride, bits_out, 0u};
    const uint32_t units = (uint32_t)act.n * (uint32_t)P.nseg;
    gap_plain_layout<<<act.n, GT, 0, st>>>(a);
    gap_widest<<<dim3(units, y_blocks(longest_k)), GT, 0, st>>>(a);
    gap_packed_layout<<<act.n, GT, 0, st>>>(a);
    gap_write<<<dim3(units, y_blocks(most_words)), GT, 0, st>>>(a);
    return cudaPeekAtLastError();
}

cudaError_t launch_decode_gaps(const Plan& P, const Active& act, const uint32_t* packed, long long packed_stride,
                               uint32_t* wire, long long stride, uint32_t longest_k, uint32_t most_words,
                               uint32_t row_chunks, cudaStream_t st) {
    GapArgs a = {P, act, packed, packed_stride, wire, stride, nullptr, row_chunks};
    const uint32_t units = (uint32_t)act.n * (uint32_t)P.nseg;
    const uint32_t chunks = (longest_k + GCH - 1) / GCH;
    gap_decode_layout<<<act.n, GT, 0, st>>>(a);
    gap_chunk_sums<<<dim3(units, chunks < 1 ? 1 : (chunks > 4096 ? 4096 : chunks)), GT, 0, st>>>(a);
    gap_chunk_scan<<<units, GT, 0, st>>>(a);
    gap_expand<<<dim3(units, y_blocks(most_words > longest_k / 4 ? most_words : longest_k / 4)), GT, 0, st>>>(a);
    return cudaPeekAtLastError();
}

}  // namespace qs
