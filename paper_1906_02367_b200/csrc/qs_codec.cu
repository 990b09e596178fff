// Quantizer, memory update, wire codec and master update: all O(kept coordinates).
//
//   norm_accum / norm_final   exact sum of squares (or magnitudes) of the kept values, as
//        integer sums per fp32 exponent, rounded once to fp64; sqrt; fp32
//   quant            level and sign per kept coordinate (Philox stream 0), m <- u - g
//   chunk_scan       ordered positions: kept rank, sent rank, stream offsets, bit counts
//   pack_dir / pack  directory and the three bit streams of every segment
//   dec_prep / dec_mark / dec_apply   master: which workers sent each index, then one owner
//        per index adds the values in worker order and updates x (and, in the fused round,
//        the workers' copies)
#include "qs_kernels.h"

namespace qs {

template <bool RANDK>
__device__ __forceinline__ bool is_kept(const Plan& P, const Unit& un, size_t pos) {
    const uint32_t sk = RANDK ? P.cand_key[pos] : topk_key(P.cand_val[pos]);
    return sk > un.tau || (sk == un.tau && P.cand_idx[pos] <= un.tie_max);
}

__device__ __forceinline__ void chunk_context(const Plan& P, uint32_t chunk, uint32_t* sh_u) {
    if (threadIdx.x == 0) {
        uint32_t lo = 0, hi = P.U;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (P.units[mid].chunk_base <= chunk) lo = mid; else hi = mid;
        }
        *sh_u = lo;
    }
    __syncthreads();
}

// Per-exponent integer sums of the kept values of each chunk: for exponent e the squares'
// 48-bit mantissa products are summed as two 24-bit halves (QSGD), or the 24-bit mantissas
// themselves (Sign).  A 64-bit sum cannot overflow below 2^32 terms.
template <bool RANDK>
__global__ void __launch_bounds__(256) norm_accum_kernel(const Plan P) {
    __shared__ unsigned long long acc[256][2];
    __shared__ uint32_t sh_u;
    const int lane = threadIdx.x & 31;
    const uint32_t total = *P.total_chunks;
    const bool l1 = P.qz == QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        chunk_context(P, chunk, &sh_u);
        acc[threadIdx.x][0] = 0ull;
        acc[threadIdx.x][1] = 0ull;
        __syncthreads();
        const uint32_t u = sh_u;
        const Unit un = P.units[u];
        const size_t base = (size_t)(u / P.nseg) * P.cap + un.start;
        const uint32_t first = (chunk - un.chunk_base) * CHUNK;
#pragma unroll 1
        for (int i = 0; i < CHUNK / 256; ++i) {
            const uint32_t off = first + i * 256 + threadIdx.x;
            const bool kept = off < un.c && is_kept<RANDK>(P, un, base + off);
            const uint32_t live = __ballot_sync(0xffffffffu, kept);
            if (kept) {
                const uint32_t b = __float_as_uint(P.cand_val[base + off]);
                const uint32_t e = (b >> 23) & 255u;
                const uint32_t m = e ? ((b & 0x7fffffu) | 0x800000u) : (b & 0x7fffffu);
                uint32_t lo, hi;
                if (l1) { lo = m; hi = 0; }
                else { const unsigned long long sq = (unsigned long long)m * m; lo = (uint32_t)(sq & 0xffffffu); hi = (uint32_t)(sq >> 24); }
                const uint32_t peers = __match_any_sync(live, e);
                // peers hold at most 32 values below 2^24: the 32-bit sums are exact
                const uint32_t slo = __reduce_add_sync(peers, lo);
                const uint32_t shi = __reduce_add_sync(peers, hi);
                if (lane == __ffs(peers) - 1) {
                    atomicAdd(&acc[e][0], (unsigned long long)slo);
                    if (!l1) atomicAdd(&acc[e][1], (unsigned long long)shi);
                }
            }
        }
        __syncthreads();
        const unsigned long long a0 = acc[threadIdx.x][0], a1 = acc[threadIdx.x][1];
        if (a0 | a1) {
            unsigned long long* g = P.eacc + ((size_t)u * 256 + threadIdx.x) * 2;
            if (a0) atomicAdd(g, a0);
            if (a1) atomicAdd(g + 1, a1);
            atomicMin(&P.units[u].emin, threadIdx.x);
            atomicMax(&P.units[u].emax, threadIdx.x);
        }
        __syncthreads();
    }
}

// Adds v (< 2^96, given as three 32-bit digits) * 2^bitpos into a little-endian base-2^32 integer.
__device__ void big_add(uint32_t* dig, int ndig, unsigned long long v_lo, uint32_t v_hi, int bitpos) {
    const int q = bitpos >> 5, o = bitpos & 31;
    // v << o as four digits
    uint32_t part[4];
    const uint32_t d0 = (uint32_t)v_lo, d1 = (uint32_t)(v_lo >> 32), d2 = v_hi;
    part[0] = d0 << o;
    part[1] = o ? ((d1 << o) | (d0 >> (32 - o))) : d1;
    part[2] = o ? ((d2 << o) | (d1 >> (32 - o))) : d2;
    part[3] = o ? (d2 >> (32 - o)) : 0u;
    unsigned long long carry = 0;
    for (int j = 0; q + j < ndig; ++j) {
        if (j >= 4 && carry == 0) break;
        const unsigned long long t = (unsigned long long)dig[q + j] + (j < 4 ? part[j] : 0u) + carry;
        dig[q + j] = (uint32_t)t;
        carry = t >> 32;
    }
}

// one thread per unit: exact sum -> fp64 (round to nearest even) -> norm in fp32
__global__ void __launch_bounds__(64) norm_final_kernel(const Plan P) {
    const uint32_t u = blockIdx.x * 64u + threadIdx.x;
    if (u >= P.U) return;
    Unit& un = P.units[u];
    if (un.c == 0 || un.emin > un.emax) return;   // no kept value seen: norm stays 0
    constexpr int ND = 24;                        // 768 bits
    uint32_t dig[ND];
    for (int j = 0; j < ND; ++j) dig[j] = 0;
    const bool l1 = P.qz == QS_SIGN_L1;
    // bit 0 of the integer stands for 2^-298 (squares) or 2^-149 (magnitudes)
    for (uint32_t e = un.emin; e <= un.emax; ++e) {
        unsigned long long* g = P.eacc + ((size_t)u * 256 + e) * 2;
        const unsigned long long a0 = g[0], a1 = g[1];
        if (!(a0 | a1)) continue;
        g[0] = 0ull; g[1] = 0ull;
        const int ee = e ? (int)e : 1;            // subnormals share the exponent of e = 1
        if (l1) {
            big_add(dig, ND, a0, 0u, ee - 1);
        } else {
            big_add(dig, ND, a0, 0u, 2 * (ee - 1));
            big_add(dig, ND, a1, 0u, 2 * (ee - 1) + 24);
        }
    }
    int top = -1;
    for (int j = ND - 1; j >= 0 && top < 0; --j)
        if (dig[j]) top = j * 32 + 31 - __clz(dig[j]);
    double sum = 0.0;
    if (top >= 0) {
        unsigned long long mant = 0;
        for (int p = top; p > top - 53; --p)
            mant = (mant << 1) | (p >= 0 ? (dig[p >> 5] >> (p & 31)) & 1u : 0u);
        const int gp = top - 53;
        const uint32_t guard = gp >= 0 ? (dig[gp >> 5] >> (gp & 31)) & 1u : 0u;
        uint32_t sticky = 0;
        for (int p = gp - 1; p >= 0 && !sticky; --p) sticky = (dig[p >> 5] >> (p & 31)) & 1u;
        if (guard && (sticky || (mant & 1ull))) mant += 1ull;
        sum = ldexp((double)mant, top - 52 - (l1 ? 149 : 298));
    }
    un.norm = l1 ? __double2float_rn(sum) : __double2float_rn(sqrt(sum));
}

// Levels, signs, memory update; counts kept and sent per chunk.
template <bool RANDK>
__global__ void __launch_bounds__(256) quant_kernel(const Plan P) {
    __shared__ uint32_t sh_u;
    __shared__ uint32_t sh_w[8];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t total = *P.total_chunks;
    const bool sign_op = P.qz == QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        chunk_context(P, chunk, &sh_u);
        const uint32_t u = sh_u;
        const Unit un = P.units[u];
        const uint32_t r = u / P.nseg, seg = u % P.nseg;
        const size_t base = (size_t)r * P.cap + un.start;
        const uint32_t first = (chunk - un.chunk_base) * CHUNK;
        const float N = un.norm, c = P.cscale[seg];
        const uint32_t k = P.kseg[seg];
        float* mem = P.mem + (size_t)r * P.d;
        uint32_t cnt = 0;                        // kept | sent << 16
#pragma unroll 1
        for (int i = 0; i < CHUNK / 256; ++i) {
            const uint32_t off = first + i * 256 + threadIdx.x;
            if (off >= un.c) continue;
            uint32_t q = 0;
            if (is_kept<RANDK>(P, un, base + off)) {
                const float v = P.cand_val[base + off];
                const uint32_t e = P.cand_idx[base + off];
                const bool neg = v < 0.0f;
                int level = 1;
                if (!sign_op) level = qsgd_level(v, N, P.s, philox_word(P, r, e, 0u));
                q = Q_SEL | (neg ? Q_NEG : 0u) | (uint32_t)level;
                cnt += 1u;
                if (level) {
                    mem[e] = v - coord_value(P, N, level, neg, c, k);
                    cnt += 1u << 16;
                }
            }
            P.cand_q[base + off] = q;
        }
        cnt = warp_sum(cnt);
        if (lane == 0) sh_w[wid] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t t = 0;
            for (int w = 0; w < 8; ++w) t += sh_w[w];
            P.chunk_cnt[chunk] = t;
        }
        __syncthreads();
    }
}

// single block: exclusive sums of kept / sent over the chunks, entries per unit, stream
// offsets and bit counts per worker
__global__ void __launch_bounds__(1024) chunk_scan_kernel(const Plan P, const Active act) {
    __shared__ uint32_t sh[33];
    const uint32_t total = *P.total_chunks;
    uint32_t carry_k = 0, carry_s = 0;
    for (uint32_t base = 0; base <= total; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < total ? P.chunk_cnt[i] : 0u;
        uint32_t tk, ts;
        const uint32_t ek = block_excl_scan(v & 0xffffu, sh, &tk);
        const uint32_t es = block_excl_scan(v >> 16, sh, &ts);
        if (i <= total) { P.chunk_sel[i] = carry_k + ek; P.chunk_nz[i] = carry_s + es; }
        carry_k += tk; carry_s += ts;
    }
    __syncthreads();
    for (uint32_t u = threadIdx.x; u < P.U; u += 1024) {
        Unit& un = P.units[u];
        if (!((act.bits >> (u / P.nseg)) & 1u)) continue;
        const uint32_t kept = P.chunk_sel[un.chunk_base + un.nchunks] - P.chunk_sel[un.chunk_base];
        un.n = P.chunk_nz[un.chunk_base + un.nchunks] - P.chunk_nz[un.chunk_base];
        if (kept != P.kseg[u % P.nseg]) set_status(P, QS_STATE);
    }
    __syncthreads();
    const bool has_lvl = P.qz != QS_SIGN_L1;
    for (int w = threadIdx.x; w < act.n; w += 1024) {
        const int r = act.r[w];
        uint32_t pay = 2u * P.nseg;
        long long bits = 0;
        for (int g = 0; g < P.nseg; ++g) {
            const uint32_t n = P.units[(size_t)r * P.nseg + g].n;
            const uint32_t bi = P.bidx[g];
            P.pay_off[(size_t)r * P.nseg + g] = pay;
            pay += words_for(n, bi) + words_for(n, 1) + (has_lvl ? words_for(n, P.bl) : 0u);
            bits += 64 + (long long)n * (bi + 1 + (has_lvl ? P.bl : 0));
        }
        P.bits[r] = bits;
    }
}

__device__ __forceinline__ void or_bits(uint32_t* w, uint64_t bitpos, uint32_t width, uint32_t val) {
    const uint64_t q = bitpos >> 5;
    const uint32_t o = (uint32_t)(bitpos & 31u);
    atomicOr(&w[q], val << o);
    if (o + width > 32u) atomicOr(&w[q + 1], val >> (32u - o));
}

__device__ __forceinline__ uint32_t get_bits(const uint32_t* w, uint64_t bitpos, uint32_t width) {
    const uint64_t q = bitpos >> 5;
    const uint32_t o = (uint32_t)(bitpos & 31u);
    uint32_t v = w[q] >> o;
    if (o + width > 32u) v |= w[q + 1] << (32u - o);
    return width >= 32u ? v : (v & ((1u << width) - 1u));
}

// directory words and bit counts
__global__ void __launch_bounds__(256) pack_dir_kernel(const Plan P, const Active act, uint32_t* wire,
                                                       const long long stride, long long* bits_out) {
    const uint32_t i = blockIdx.x * 256u + threadIdx.x;
    if (i >= (uint32_t)act.n * P.nseg) return;
    const int r = act.r[i / P.nseg];
    const uint32_t g = i % P.nseg;
    const Unit& un = P.units[(size_t)r * P.nseg + g];
    uint32_t* row = wire + (size_t)r * stride;
    row[2 * g] = un.n;
    row[2 * g + 1] = __float_as_uint(un.norm);
    if (g == 0 && bits_out) bits_out[r] = P.bits[r];
}

// streams of every segment, and the ordered kept list kept for inspection
__global__ void __launch_bounds__(256) pack_kernel(const Plan P, uint32_t* wire, const long long stride) {
    __shared__ uint32_t sh_u;
    __shared__ uint32_t sh[33];
    const uint32_t total = *P.total_chunks;
    const bool has_lvl = P.qz != QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        chunk_context(P, chunk, &sh_u);
        const uint32_t u = sh_u;
        const Unit un = P.units[u];
        const uint32_t r = u / P.nseg, seg = u % P.nseg;
        const size_t base = (size_t)r * P.cap + un.start;
        const uint32_t first = (chunk - un.chunk_base) * CHUNK;
        uint32_t run_k = P.chunk_sel[chunk] - P.chunk_sel[un.chunk_base];
        uint32_t run_s = P.chunk_nz[chunk] - P.chunk_nz[un.chunk_base];
        const uint32_t bi = P.bidx[seg], lo = P.seg_off[seg];
        uint32_t* w_idx = wire + (size_t)r * stride + P.pay_off[u];
        uint32_t* w_sgn = w_idx + words_for(un.n, bi);
        uint32_t* w_lvl = w_sgn + words_for(un.n, 1);
        uint32_t* o_idx = P.sel_idx + (size_t)r * P.K + P.kprefix[seg];
        uint32_t* o_q = P.sel_q + (size_t)r * P.K + P.kprefix[seg];
#pragma unroll 1
        for (int i = 0; i < CHUNK / 256; ++i) {
            const uint32_t off = first + i * 256 + threadIdx.x;
            const uint32_t q = off < un.c ? P.cand_q[base + off] : 0u;
            const uint32_t kept = (q & Q_SEL) ? 1u : 0u, sent = (kept && (q & 0xffffu)) ? 1u : 0u;
            uint32_t tot;
            const uint32_t ex = block_excl_scan(kept | (sent << 16), sh, &tot);
            if (kept) {
                const uint32_t e = P.cand_idx[base + off];
                const uint32_t jk = run_k + (ex & 0xffffu);
                o_idx[jk] = e;
                o_q[jk] = q;
                if (sent) {
                    const uint64_t js = run_s + (ex >> 16);
                    or_bits(w_idx, js * bi, bi, e - lo);
                    if (q & Q_NEG) atomicOr(&w_sgn[js >> 5], 1u << (js & 31u));
                    if (has_lvl) or_bits(w_lvl, js * P.bl, P.bl, (q & 0xffffu) - 1u);
                }
            }
            run_k += tot & 0xffffu;
            run_s += tot >> 16;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ master
// grid nact: entry and stream offsets of each segment, read from the directory
__global__ void __launch_bounds__(256) dec_prep_kernel(const Plan P, const Active act, const uint32_t* wire,
                                                       const long long stride) {
    __shared__ uint32_t sh[33];
    const int r = act.r[blockIdx.x];
    const uint32_t* row = wire + (size_t)r * stride;
    const bool has_lvl = P.qz != QS_SIGN_L1;
    uint32_t carry_e = 0, carry_w = 2u * P.nseg;
    for (uint32_t base = 0; base < (uint32_t)P.nseg; base += 256) {
        const uint32_t g = base + threadIdx.x;
        uint32_t n = 0, words = 0;
        if (g < (uint32_t)P.nseg) {
            n = row[2 * g];
            if (n > P.kseg[g]) { n = 0; set_status(P, QS_INVALID_ARG); }   // not a record of this plan
            words = words_for(n, P.bidx[g]) + words_for(n, 1) + (has_lvl ? words_for(n, P.bl) : 0u);
        }
        uint32_t te, tw;
        const uint32_t ee = block_excl_scan(n, sh, &te);
        const uint32_t ew = block_excl_scan(words, sh, &tw);
        if (g < (uint32_t)P.nseg) {
            P.dec_ent[(size_t)r * (P.nseg + 1) + g] = carry_e + ee;
            P.dec_pay[(size_t)r * P.nseg + g] = carry_w + ew;
        }
        carry_e += te; carry_w += tw;
    }
    if (threadIdx.x == 0) P.dec_ent[(size_t)r * (P.nseg + 1) + P.nseg] = carry_e;
}

struct Entry { uint32_t seg, j, n, coord; const uint32_t* w_idx; };

// entry `ent` of worker r's record
__device__ __forceinline__ bool locate_entry(const Plan& P, const uint32_t* wire, long long stride, int r,
                                             uint32_t ent, Entry* out) {
    const uint32_t* eb = P.dec_ent + (size_t)r * (P.nseg + 1);
    if (ent >= eb[P.nseg]) return false;
    uint32_t lo = 0, hi = P.nseg;               // eb[lo] <= ent < eb[hi]
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (eb[mid] <= ent) lo = mid; else hi = mid;
    }
    out->seg = lo;
    out->j = ent - eb[lo];
    out->n = eb[lo + 1] - eb[lo];
    out->w_idx = wire + (size_t)r * stride + P.dec_pay[(size_t)r * P.nseg + lo];
    out->coord = P.seg_off[lo] + get_bits(out->w_idx, (uint64_t)out->j * P.bidx[lo], P.bidx[lo]);
    return true;
}

__device__ __forceinline__ float entry_value(const Plan& P, const uint32_t* row, const Entry& en) {
    const uint32_t bi = P.bidx[en.seg];
    const uint32_t* w_sgn = en.w_idx + words_for(en.n, bi);
    const uint32_t* w_lvl = w_sgn + words_for(en.n, 1);
    const bool neg = (w_sgn[en.j >> 5] >> (en.j & 31u)) & 1u;
    const int level = P.qz == QS_SIGN_L1 ? 1 : (int)get_bits(w_lvl, (uint64_t)en.j * P.bl, P.bl) + 1;
    return coord_value(P, __uint_as_float(row[2 * en.seg + 1]), level, neg, P.cscale[en.seg], P.kseg[en.seg]);
}

__global__ void __launch_bounds__(256) dec_mark_kernel(const Plan P, const Active act, const uint32_t* wire,
                                                       const long long stride) {
    const uint64_t total = (uint64_t)act.n * P.K;
    for (uint64_t id = (uint64_t)blockIdx.x * 256u + threadIdx.x; id < total; id += (uint64_t)gridDim.x * 256u) {
        const int r = act.r[id / P.K];
        Entry en;
        if (!locate_entry(P, wire, stride, r, (uint32_t)(id % P.K), &en)) continue;
        if (en.coord < P.d) atomicOr(&P.touch[en.coord], 1u << r);
        else set_status(P, QS_INVALID_ARG);
    }
}

// The lowest worker that sent an index owns it: it adds the values of all senders in
// increasing worker order, updates x, and in the fused round patches the workers' copies.
__global__ void __launch_bounds__(256) dec_apply_kernel(const Plan P, const Active act, const uint32_t* wire,
                                                        const long long stride, const int patch) {
    const uint64_t total = (uint64_t)act.n * P.K;
    for (uint64_t id = (uint64_t)blockIdx.x * 256u + threadIdx.x; id < total; id += (uint64_t)gridDim.x * 256u) {
        const int r = act.r[id / P.K];
        Entry en;
        if (!locate_entry(P, wire, stride, r, (uint32_t)(id % P.K), &en)) continue;
        if (en.coord >= P.d) continue;
        const uint32_t senders = P.touch[en.coord];
        if (!senders || (__ffs(senders) - 1) != r) continue;
        float acc = 0.0f;
        acc = acc + entry_value(P, wire + (size_t)r * stride, en);
        uint32_t rest = senders & (senders - 1u);
        const uint32_t local = en.coord - P.seg_off[en.seg], bi = P.bidx[en.seg];
        while (rest) {
            const int r2 = __ffs(rest) - 1;
            rest &= rest - 1u;
            // find the index in r2's ascending list of this segment
            const uint32_t* eb = P.dec_ent + (size_t)r2 * (P.nseg + 1);
            Entry e2;
            e2.seg = en.seg;
            e2.n = eb[en.seg + 1] - eb[en.seg];
            e2.w_idx = wire + (size_t)r2 * stride + P.dec_pay[(size_t)r2 * P.nseg + en.seg];
            uint32_t lo = 0, hi = e2.n;          // first position with index >= local
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (get_bits(e2.w_idx, (uint64_t)mid * bi, bi) < local) lo = mid + 1; else hi = mid;
            }
            e2.j = lo;
            e2.coord = en.coord;
            acc = acc + entry_value(P, wire + (size_t)r2 * stride, e2);
        }
        const float xn = P.x[en.coord] - acc / (float)P.R;
        P.x[en.coord] = xn;
        if (patch) {
            for (int w = 0; w < act.n; ++w) {
                P.xw[(size_t)act.r[w] * P.d + en.coord] = xn;
                if (P.anchors) P.anchors[(size_t)act.r[w] * P.d + en.coord] = xn;
            }
        }
        P.touch[en.coord] = 0u;
    }
}

__global__ void __launch_bounds__(256) export_kernel(const Plan P, long long* sel_idx, int* level, uint8_t* sign,
                                                     float* norm, long long* n) {
    const uint64_t total = (uint64_t)P.R * P.K;
    for (uint64_t i = (uint64_t)blockIdx.x * 256u + threadIdx.x; i < total; i += (uint64_t)gridDim.x * 256u) {
        const uint32_t q = P.sel_q[i];
        if (sel_idx) sel_idx[i] = P.sel_idx[i];
        if (level) level[i] = (int)(q & 0xffffu);
        if (sign) sign[i] = (q & Q_NEG) ? 1 : 0;
    }
    for (uint32_t u = blockIdx.x * 256u + threadIdx.x; u < P.U; u += gridDim.x * 256u) {
        if (norm) norm[u] = P.units[u].norm;
        if (n) n[u] = P.units[u].n;
    }
}

// ------------------------------------------------------------------ launchers
void launch_quantize(const Plan& P, const Active& act, int sms, cudaStream_t st) {
    const bool rk = P.sp == QS_RANDK;
    const int grid = chunk_grid(P, sms);
    if (rk) norm_accum_kernel<true><<<grid, 256, 0, st>>>(P);
    else norm_accum_kernel<false><<<grid, 256, 0, st>>>(P);
    norm_final_kernel<<<(P.U + 63) / 64, 64, 0, st>>>(P);
    if (rk) quant_kernel<true><<<grid, 256, 0, st>>>(P);
    else quant_kernel<false><<<grid, 256, 0, st>>>(P);
    chunk_scan_kernel<<<1, 1024, 0, st>>>(P, act);
}

void launch_pack(const Plan& P, const Active& act, uint32_t* wire, long long stride, long long* bits_out,
                 int sms, cudaStream_t st) {
    const uint32_t items = (uint32_t)act.n * P.nseg;
    pack_dir_kernel<<<(items + 255) / 256, 256, 0, st>>>(P, act, wire, stride, bits_out);
    pack_kernel<<<chunk_grid(P, sms), 256, 0, st>>>(P, wire, stride);
}

void launch_decode(const Plan& P, const Active& act, const uint32_t* wire, long long stride, int patch,
                   int sms, cudaStream_t st) {
    dec_prep_kernel<<<act.n, 256, 0, st>>>(P, act, wire, stride);
    const uint64_t total = (uint64_t)act.n * P.K;
    uint64_t blocks = (total + 255) / 256;
    const uint64_t cap = (uint64_t)sms * 16;
    const int grid = (int)(blocks < cap ? (blocks ? blocks : 1) : cap);
    dec_mark_kernel<<<grid, 256, 0, st>>>(P, act, wire, stride);
    dec_apply_kernel<<<grid, 256, 0, st>>>(P, act, wire, stride, patch);
}

void launch_export(const Plan& P, long long* sel_idx, int* level, uint8_t* sign, float* norm, long long* n,
                   int sms, cudaStream_t st) {
    export_kernel<<<sms * 4, 256, 0, st>>>(P, sel_idx, level, sign, norm, n);
}

}  // namespace qs
