// Everything between the dense pass and the end of the round, as ONE persistent kernel.
//
// The work after the dense pass is O(candidates): small, and made of a dozen steps that each
// need the previous one finished everywhere.  Launched separately they cost more in launch
// gaps and cold starts than in work, so they run here as stages of one cooperative launch
// (every block resident), separated by grid-wide barriers with a bounded wait:
//
//   candidates  scan of the per-block candidate counts left by the dense pass, candidate
//               range of every (worker, segment) unit, the exact fallback for workers whose
//               predicted threshold left a unit short (histogram of the top key bits, new
//               threshold, bitmap rebuilt from the stored u), ordered emission (index, value)
//   select      radix select over the 32-bit sort key (4 levels of 8 bits), tie cut by lower
//               index, next round's prediction
//   quantize    exact norm of the kept values, levels and signs (Philox stream 0), m <- u - g,
//               ordered positions of kept and sent entries
//   pack        directory and the three bit streams of every segment
//   decode      senders of every index, then one owner per index adds the values in worker
//               order, updates x and (fused round) patches the workers' copies
//
// Order-dependent results come only from ordered scans, never from the order of atomics.
#include "qs_kernels.h"

namespace qs {

constexpr int BT = 256;                    // threads per block of the persistent kernel
constexpr int PER = CHUNK / BT;            // candidates per thread and chunk
constexpr uint32_t SPIN_LIMIT = 1u << 22;  // barrier polls before giving up (about a second)

struct MidArgs {
    Plan P;
    Active act;
    int do_compress, do_pack, do_decode, patch, do_broadcast, aligned;
    uint32_t* wire;
    long long stride;
    long long* bits_out;
};

// ------------------------------------------------------------------ grid barrier
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// All blocks of the cooperative launch meet here.  The wait is bounded: a block that gives up
// records QS_TIMEOUT and every block leaves the kernel at its next barrier.
__device__ __forceinline__ bool grid_barrier(const Plan& P, uint32_t& target, int* sh_abort) {
    target += gridDim.x;
    __syncthreads();
    if (P.trace && blockIdx.x == 0 && threadIdx.x == 0) {     // stage boundaries as block 0 sees them
        const uint32_t slot = target / gridDim.x;
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (slot < TRACE_SLOTS) P.trace[slot] = t;
    }
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(P.bar, 1u);
        uint32_t spins = 0;
        while (ld_acquire(P.bar) < target) {
            if (++spins > SPIN_LIMIT) {
                atomicCAS(P.status, 0, QS_TIMEOUT);
                *sh_abort = 1;
                break;
            }
            __nanosleep(32);
        }
        __threadfence();
    }
    __syncthreads();
    return *sh_abort == 0;
}

__device__ __forceinline__ uint32_t popc4(const uint4 w) {
    return __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
}

template <bool RANDK>
__device__ __forceinline__ uint32_t sort_key(const Plan& P, size_t pos) {
    return RANDK ? P.cand_key[pos] : topk_key(P.cand_val[pos]);
}

// ------------------------------------------------------------------ candidates
// exclusive prefix of the per-block candidate counts of each worker; clears the counts
__device__ void stage_scan(const Plan& P, const Active& act, bool only_failed, uint32_t* sh) {
    for (int w = blockIdx.x; w < act.n; w += gridDim.x) {
        const int r = act.r[w];
        if (only_failed && !P.fail[r]) continue;
        uint32_t carry = 0;
        for (uint32_t base = 0; base < P.nblk; base += BT) {
            const uint32_t i = base + threadIdx.x;
            uint32_t v = 0;
            if (i < P.nblk) {
                v = P.blk_count[(size_t)r * P.nblk + i];
                P.blk_count[(size_t)r * P.nblk + i] = 0;
            }
            uint32_t total;
            const uint32_t ex = block_excl_scan(v, sh, &total);
            if (i < P.nblk) P.blk_base[(size_t)r * P.nblk + i] = carry + ex;
            carry += total;
        }
        if (threadIdx.x == 0) P.ncand[r] = carry;
    }
}

// candidates of worker r among coordinates below p (warp-cooperative, every lane gets it)
__device__ uint32_t cand_prefix(const Plan& P, int r, uint32_t p, int lane) {
    if (p >= P.d) return P.ncand[r];
    const uint32_t g = p >> 7, blk = g / EMIT_GROUPS;
    const uint4* bm = reinterpret_cast<const uint4*>(P.bitmap) + (size_t)r * P.ngroups;
    uint32_t c = 0;
    for (uint32_t gg = blk * EMIT_GROUPS + lane; gg < g; gg += 32) c += popc4(bm[gg]);
    if (lane == 0) {
        const uint4 w = bm[g];
        const uint32_t pl = p & 127u;
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) {
            const uint32_t nl = pl > j ? (pl - j + 3u) >> 2 : 0u;      // lanes l with 4 l + j < pl
            const uint32_t mask = nl >= 32u ? 0xffffffffu : ((1u << nl) - 1u);
            c += __popc(ws[j] & mask);
        }
        c += P.blk_base[(size_t)r * P.nblk + blk];
    }
    return warp_sum(c);
}

// one warp per unit: its candidate range; a unit with fewer candidates than k marks its worker
__device__ void stage_bounds(const Plan& P, const Active& act, bool only_failed) {
    const int lane = threadIdx.x & 31;
    const uint32_t nunits = (uint32_t)act.n * P.nseg;
    for (uint32_t wu = blockIdx.x * (BT / 32) + (threadIdx.x >> 5); wu < nunits; wu += gridDim.x * (BT / 32)) {
        const int r = act.r[wu / P.nseg];
        const uint32_t seg = wu % P.nseg;
        if (only_failed && !P.fail[r]) continue;
        const uint32_t lo = cand_prefix(P, r, P.seg_off[seg], lane);
        const uint32_t hi = cand_prefix(P, r, P.seg_off[seg + 1], lane);
        if (lane == 0) {
            Unit& un = P.units[(size_t)r * P.nseg + seg];
            un.start = lo;
            un.c = hi - lo;
            if (hi - lo < P.kseg[seg]) {
                if (only_failed) set_status(P, QS_STATE);      // the exact pass cannot miss
                else atomicExch(&P.fail[r], 1u);
            }
        }
    }
}

// histogram of the top 11 key bits of one stretch of one segment, for missed workers
template <bool RANDK>
__device__ void stage_fb_hist(const Plan& P, const Active& act, uint32_t* sh_bins) {
    const uint32_t items = P.nfb * (uint32_t)act.n;
    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int r = act.r[item / P.nfb];
        if (!P.fail[r]) continue;
        const FbBlock blk = P.fb_tab[item % P.nfb];
        for (int i = threadIdx.x; i < FB_BINS; i += BT) sh_bins[i] = 0;
        __syncthreads();
        const size_t row = (size_t)r * P.d;
        for (uint32_t base = 0; base < blk.len; base += BT) {
            const uint32_t i = base + threadIdx.x;
            const bool valid = i < blk.len;
            const uint32_t live = __ballot_sync(0xffffffffu, valid);
            if (valid) {
                const uint32_t e = blk.start + i;
                const uint32_t sk = RANDK ? ~philox_word(P, (uint32_t)r, e, 1u) : topk_key(P.mem[row + e]);
                const uint32_t bin = sk >> FB_SHIFT;
                const uint32_t peers = __match_any_sync(live, bin);
                if ((threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&sh_bins[bin], __popc(peers));
            }
        }
        __syncthreads();
        uint32_t* out = P.fb_hist + ((size_t)r * P.nseg + blk.seg) * FB_BINS;
        for (int i = threadIdx.x; i < FB_BINS; i += BT)
            if (sh_bins[i]) atomicAdd(&out[i], sh_bins[i]);
        __syncthreads();
    }
}

// new threshold of each segment of a missed worker: the lowest bin edge that still leaves
// `target` coordinates at or above it; clears the histogram
__device__ void stage_fb_guess(const Plan& P, const Active& act, uint32_t* sh, uint32_t* sh_best) {
    const uint32_t items = (uint32_t)P.nseg * act.n;
    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int r = act.r[item / P.nseg];
        if (!P.fail[r]) continue;
        const uint32_t seg = item % P.nseg;
        uint32_t* hist = P.fb_hist + ((size_t)r * P.nseg + seg) * FB_BINS;
        uint32_t v[8], s = 0;                    // thread t owns bins 2047 - 8t .. 2040 - 8t
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int bin = FB_BINS - 1 - 8 * (int)threadIdx.x - i;
            v[i] = hist[bin];
            hist[bin] = 0;
            s += v[i];
        }
        if (threadIdx.x == 0) *sh_best = 0;
        uint32_t total;
        const uint32_t excl = block_excl_scan(s, sh, &total);
        const uint32_t target = P.target[seg];
        if (excl < target && excl + s >= target) {
            uint32_t run = excl;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                run += v[i];
                if (run >= target) { *sh_best = (uint32_t)(FB_BINS - 1 - 8 * (int)threadIdx.x - i); break; }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) P.guess[(size_t)r * P.nseg + seg] = *sh_best << FB_SHIFT;
        __syncthreads();
    }
}

// segment of each coordinate of a quad
__device__ __forceinline__ void quad_segments(const Plan& P, uint32_t g, uint32_t e0, int sg[4]) {
    if (P.nseg == 1) { sg[0] = sg[1] = sg[2] = sg[3] = 0; return; }
    int sq = (int)P.grp_seg[g];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        while (sq + 1 < P.nseg && e0 + j >= P.seg_off[sq + 1]) ++sq;
        sg[j] = sq;
    }
}

// bitmap and block counts of the missed workers rebuilt from the stored u
template <bool RANDK>
__device__ void stage_reflag(const Plan& P, const Active& act) {
    const int lane = threadIdx.x & 31;
    for (int w = 0; w < act.n; ++w) {
        const int r = act.r[w];
        if (!P.fail[r]) continue;
        const size_t row = (size_t)r * P.d;
        const uint32_t* gs = P.guess + (size_t)r * P.nseg;
        for (uint32_t g = blockIdx.x * (BT / 32) + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * (BT / 32)) {
            const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
            int sg[4];
            quad_segments(P, g, e0, sg);
            uint4 h = make_uint4(0, 0, 0, 0);
            if (RANDK) h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
            const uint32_t hh[4] = {h.x, h.y, h.z, h.w};
            uint32_t fl[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                fl[j] = 0;
                if (e0 + j < P.d) {
                    const uint32_t sk = RANDK ? ~hh[j] : topk_key(P.mem[row + e0 + j]);
                    fl[j] = sk >= gs[sg[j]];
                }
            }
            const uint32_t b0 = __ballot_sync(0xffffffffu, fl[0]);
            const uint32_t b1 = __ballot_sync(0xffffffffu, fl[1]);
            const uint32_t b2 = __ballot_sync(0xffffffffu, fl[2]);
            const uint32_t b3 = __ballot_sync(0xffffffffu, fl[3]);
            if (lane == 0) {
                reinterpret_cast<uint4*>(P.bitmap)[(size_t)r * P.ngroups + g] = make_uint4(b0, b1, b2, b3);
                const uint32_t cnt = __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
                if (cnt) atomicAdd(&P.blk_count[(size_t)r * P.nblk + g / EMIT_GROUPS], cnt);
            }
        }
    }
}

// candidates of one emission block, in ascending coordinate order
template <bool RANDK>
__device__ void stage_emit(const Plan& P, const Active& act, uint32_t* sh) {
    const uint32_t items = P.nblk * (uint32_t)act.n;
    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int r = act.r[item / P.nblk];
        const uint32_t blk = item % P.nblk;
        const uint32_t g = blk * (uint32_t)EMIT_GROUPS + threadIdx.x;
        uint4 w = make_uint4(0, 0, 0, 0);
        if (g < P.ngroups) w = reinterpret_cast<const uint4*>(P.bitmap)[(size_t)r * P.ngroups + g];
        uint32_t total;
        const uint32_t ex = block_excl_scan(popc4(w), sh, &total);
        if (total == 0) continue;
        size_t pos = (size_t)r * P.cap + P.blk_base[(size_t)r * P.nblk + blk] + ex;
        const float* mem = P.mem + (size_t)r * P.d;
        while (w.x | w.y | w.z | w.w) {
            uint32_t best = 0xffffffffu;               // lowest coordinate 4 l + j still set
            if (w.x) best = min(best, (uint32_t)(__ffs(w.x) - 1) * 4u + 0u);
            if (w.y) best = min(best, (uint32_t)(__ffs(w.y) - 1) * 4u + 1u);
            if (w.z) best = min(best, (uint32_t)(__ffs(w.z) - 1) * 4u + 2u);
            if (w.w) best = min(best, (uint32_t)(__ffs(w.w) - 1) * 4u + 3u);
            const uint32_t j = best & 3u;
            if (j == 0) w.x &= w.x - 1u; else if (j == 1) w.y &= w.y - 1u;
            else if (j == 2) w.z &= w.z - 1u; else w.w &= w.w - 1u;
            const uint32_t e = g * (uint32_t)GROUP + best;
            P.cand_idx[pos] = e;
            P.cand_val[pos] = mem[e];
            if (RANDK) P.cand_key[pos] = ~philox_word(P, (uint32_t)r, e, 1u);
            ++pos;
        }
    }
}

// block 0: chunk numbering over the units of the active workers, in (worker, segment) order
__device__ void stage_setup(const Plan& P, const Active& act, uint32_t* sh) {
    if (blockIdx.x != 0) return;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < P.U; base += BT) {
        const uint32_t u = base + threadIdx.x;
        uint32_t nch = 0, cands = 0;
        if (u < P.U) {
            Unit& un = P.units[u];
            if (!((act.bits >> (u / P.nseg)) & 1u)) un.c = 0;
            cands = un.c;
            nch = (cands + CHUNK - 1) / CHUNK;
        }
        uint32_t total;
        const uint32_t ex = block_excl_scan(nch, sh, &total);
        if (u < P.U) {
            Unit& un = P.units[u];
            un.chunk_base = carry + ex;
            un.nchunks = nch;
            un.n = 0;
            un.emin = 255u;
            un.emax = 0u;
            un.norm = 0.0f;
            if (cands) atomicAdd((unsigned long long*)&P.stats[1], (unsigned long long)cands);
        }
        carry += total;
    }
    if (threadIdx.x == 0) {
        *P.total_chunks = carry;
        uint32_t nf = 0;
        for (int w = 0; w < act.n; ++w) { nf += P.fail[act.r[w]] ? 1u : 0u; P.fail[act.r[w]] = 0; }
        if (nf) atomicAdd((unsigned long long*)&P.stats[0], (unsigned long long)nf);
    }
}

// ------------------------------------------------------------------ select
// unit owning a chunk: the last unit whose first chunk is not after it
__device__ __forceinline__ uint32_t unit_of_chunk(const Plan& P, uint32_t chunk) {
    uint32_t lo = 0, hi = P.U;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (P.units[mid].chunk_base <= chunk) lo = mid; else hi = mid;
    }
    return lo;
}

// Within 256 bins counted from the top, the bin holding rank kk (1-based) and the number of
// keys in higher bins.  Warp-cooperative.
__device__ __forceinline__ void find_bin(const uint32_t* h, uint32_t kk, int lane, uint32_t* bin, uint32_t* above) {
    uint32_t v[8], s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[i] = h[255 - 8 * lane - i]; s += v[i]; }
    const uint32_t incl = warp_incl_scan(s, lane);
    const uint32_t hit = __ballot_sync(0xffffffffu, incl >= kk);
    const int owner = hit ? __ffs(hit) - 1 : 31;
    uint32_t b = 0, a = 0;
    if (lane == owner) {
        uint32_t run = incl - s;
        b = 255u - 8u * lane - 7u; a = run;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (run + v[i] >= kk) { b = 255u - 8u * lane - i; a = run; break; }
            run += v[i];
        }
    }
    *bin = __shfl_sync(0xffffffffu, b, owner);
    *above = __shfl_sync(0xffffffffu, a, owner);
}

// key prefix fixed by levels 0 .. level-1 and the number of keys above it (one warp)
__device__ void derive_prefix(const Plan& P, uint32_t u, uint32_t k, int level, int lane, uint32_t* prefix,
                              uint32_t* above_total) {
    uint32_t pf = 0, kk = k, at = 0;
    for (int L = 0; L < level; ++L) {
        uint32_t bin, above;
        find_bin(P.hist + ((size_t)L * P.U + u) * 256, kk, lane, &bin, &above);
        pf = (pf << 8) | bin;
        kk -= above;
        at += above;
    }
    *prefix = pf;
    *above_total = at;
}

struct ChunkCtx { uint32_t u, r, seg, first; Unit un; size_t base; };

// which unit a chunk belongs to (one search per block, shared through sh_u)
__device__ __forceinline__ ChunkCtx chunk_context(const Plan& P, uint32_t chunk, uint32_t* sh_u) {
    __syncthreads();
    if (threadIdx.x == 0) *sh_u = unit_of_chunk(P, chunk);
    __syncthreads();
    ChunkCtx c;
    c.u = *sh_u;
    c.un = P.units[c.u];
    c.r = c.u / P.nseg;
    c.seg = c.u % P.nseg;
    c.first = (chunk - c.un.chunk_base) * CHUNK;
    c.base = (size_t)c.r * P.cap + c.un.start;
    return c;
}

// one level of the radix select: histogram of the level's digit among keys matching the prefix
template <bool RANDK>
__device__ void stage_hist(const Plan& P, int level, uint32_t* sh_hist, uint32_t* sh_u, uint32_t* sh_prefix) {
    const int lane = threadIdx.x & 31;
    const uint32_t total = *P.total_chunks;
    const int shift = 24 - 8 * level;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        const ChunkCtx c = chunk_context(P, chunk, sh_u);
        uint32_t sk[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            sk[i] = off < c.un.c ? sort_key<RANDK>(P, c.base + off) : 0u;
        }
        if (threadIdx.x < 32) {
            uint32_t prefix, at;
            derive_prefix(P, c.u, P.kseg[c.seg], level, lane, &prefix, &at);
            if (lane == 0) *sh_prefix = prefix;
        }
        sh_hist[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t prefix = *sh_prefix;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool valid = off < c.un.c && (level == 0 || (sk[i] >> (32 - 8 * level)) == prefix);
            const uint32_t digit = (sk[i] >> shift) & 255u;
            const uint32_t live = __ballot_sync(0xffffffffu, valid);
            if (valid) {
                const uint32_t peers = __match_any_sync(live, digit);
                if (lane == __ffs(peers) - 1) atomicAdd(&sh_hist[digit], __popc(peers));
            }
        }
        __syncthreads();
        const uint32_t v = sh_hist[threadIdx.x];
        if (v) atomicAdd(&P.hist[((size_t)level * P.U + c.u) * 256 + threadIdx.x], v);
    }
}

// threshold key, tie cut and next prediction of each unit; clears its histograms
template <bool RANDK>
__device__ void stage_final(const Plan& P, uint32_t* sh4, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (uint32_t u = blockIdx.x; u < P.U; u += gridDim.x) {
        const Unit un = P.units[u];
        if (un.c == 0) continue;
        const uint32_t seg = u % P.nseg, r = u / P.nseg, k = P.kseg[seg];
        __syncthreads();
        if (wid == 0) {
            uint32_t prefix, above;
            derive_prefix(P, u, k, 4, lane, &prefix, &above);
            if (lane == 0) {
                sh4[0] = prefix;                                   // tau
                sh4[1] = k - above;                                // kept among keys equal to tau
                sh4[2] = P.hist[((size_t)3 * P.U + u) * 256 + (prefix & 255u)];
                sh4[3] = 0xffffffffu;                              // index of the last kept tie
                sh4[4] = 0;                                        // ties seen so far
            }
        }
        __syncthreads();
        for (int L = 0; L < 4; ++L) P.hist[((size_t)L * P.U + u) * 256 + threadIdx.x] = 0;
        const uint32_t tau = sh4[0], t = sh4[1], ceq = sh4[2];
        uint32_t tie_max = 0xffffffffu;
        if (ceq > t) {
            // more equal keys than slots: the t lowest coordinates win; walk the list in order
            const size_t base = (size_t)r * P.cap + un.start;
            for (uint32_t first = 0; first < un.c; first += BT) {
                const uint32_t off = first + threadIdx.x;
                const bool eq = off < un.c && sort_key<RANDK>(P, base + off) == tau;
                const uint32_t bal = __ballot_sync(0xffffffffu, eq);
                if (lane == 0) sh_w[wid] = __popc(bal);
                __syncthreads();
                uint32_t before = sh4[4];
                for (int w = 0; w < wid; ++w) before += sh_w[w];
                const uint32_t mine = before + __popc(bal & ((1u << lane) - 1u));
                if (eq && mine == t - 1) sh4[3] = P.cand_idx[base + off];
                __syncthreads();
                if (threadIdx.x == 0) { uint32_t s = 0; for (int w = 0; w < BT / 32; ++w) s += sh_w[w]; sh4[4] += s; }
                __syncthreads();
                if (sh4[3] != 0xffffffffu) break;
            }
            tie_max = sh4[3];
        }
        if (threadIdx.x == 0) {
            Unit& out = P.units[u];
            out.tau = tau;
            out.tie_max = tie_max;
            if (!RANDK) {
                // prediction for the next round: move the candidate floor so that about `target`
                // coordinates pass it, assuming the tail keeps its shape (log-linear in the count)
                uint32_t* gp = &P.guess[(size_t)r * P.nseg + seg];
                const float tk = __uint_as_float(tau >> 1), tg = __uint_as_float(*gp >> 1);
                const float target = (float)P.target[seg];
                float tn = tg;
                if (un.c > k && tk > tg) {
                    float ratio = __logf(target / (float)k) / __logf((float)un.c / (float)k);
                    ratio = fminf(fmaxf(ratio, 0.25f), 4.0f);
                    tn = tk - (tk - tg) * ratio;
                } else if (un.c <= k) {
                    tn = tk * 0.75f;
                }
                tn = fminf(fmaxf(tn, tk * 0.25f), tk);
                *gp = __float_as_uint(tn) << 1;
            }
        }
    }
}

// ------------------------------------------------------------------ quantize
template <bool RANDK>
__device__ __forceinline__ bool is_kept(const Unit& un, uint32_t sk, uint32_t idx) {
    return sk > un.tau || (sk == un.tau && idx <= un.tie_max);
}

// Per-exponent integer sums of the kept values: for exponent e the squares' 48-bit mantissa
// products are summed as two 24-bit halves (QSGD), or the 24-bit mantissas themselves (Sign).
// A 64-bit sum cannot overflow below 2^32 terms.
template <bool RANDK>
__device__ void stage_norm_accum(const Plan& P, unsigned long long (*acc)[2], uint32_t* sh_u) {
    const int lane = threadIdx.x & 31;
    const uint32_t total = *P.total_chunks;
    const bool l1 = P.qz == QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        const ChunkCtx c = chunk_context(P, chunk, sh_u);
        float val[PER];
        uint32_t idx[PER], key[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool in = off < c.un.c;
            val[i] = in ? P.cand_val[c.base + off] : 0.0f;
            idx[i] = in ? P.cand_idx[c.base + off] : 0xffffffffu;
            key[i] = RANDK ? (in ? P.cand_key[c.base + off] : 0u) : topk_key(val[i]);
        }
        acc[threadIdx.x][0] = 0ull;
        acc[threadIdx.x][1] = 0ull;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool kept = off < c.un.c && is_kept<RANDK>(c.un, key[i], idx[i]);
            const uint32_t live = __ballot_sync(0xffffffffu, kept);
            if (kept) {
                const uint32_t b = __float_as_uint(val[i]);
                const uint32_t e = (b >> 23) & 255u;
                const uint32_t m = e ? ((b & 0x7fffffu) | 0x800000u) : (b & 0x7fffffu);
                uint32_t lo, hi;
                if (l1) { lo = m; hi = 0; }
                else { const unsigned long long sq = (unsigned long long)m * m; lo = (uint32_t)(sq & 0xffffffu); hi = (uint32_t)(sq >> 24); }
                const uint32_t peers = __match_any_sync(live, e);
                // at most 32 values below 2^24: the 32-bit sums are exact
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
            unsigned long long* g = P.eacc + ((size_t)c.u * 256 + threadIdx.x) * 2;
            if (a0) atomicAdd(g, a0);
            if (a1) atomicAdd(g + 1, a1);
            atomicMin(&P.units[c.u].emin, threadIdx.x);
            atomicMax(&P.units[c.u].emax, threadIdx.x);
        }
    }
}

// adds v * 2^bitpos into a little-endian base-2^32 integer
__device__ void big_add(uint32_t* dig, int ndig, unsigned long long v, int bitpos) {
    const int q = bitpos >> 5, o = bitpos & 31;
    const uint32_t d0 = (uint32_t)v, d1 = (uint32_t)(v >> 32);
    uint32_t part[3];
    part[0] = d0 << o;
    part[1] = o ? ((d1 << o) | (d0 >> (32 - o))) : d1;
    part[2] = o ? (d1 >> (32 - o)) : 0u;
    unsigned long long carry = 0;
    for (int j = 0; q + j < ndig; ++j) {
        if (j >= 3 && carry == 0) break;
        const unsigned long long t = (unsigned long long)dig[q + j] + (j < 3 ? part[j] : 0u) + carry;
        dig[q + j] = (uint32_t)t;
        carry = t >> 32;
    }
}

// one thread per unit: exact sum -> fp64 (round to nearest even) -> norm in fp32
__device__ void stage_norm_final(const Plan& P) {
    for (uint32_t u = blockIdx.x * BT + threadIdx.x; u < P.U; u += gridDim.x * BT) {
        Unit& un = P.units[u];
        if (un.c == 0 || un.emin > un.emax) continue;
        constexpr int ND = 24;                      // 768 bits
        uint32_t dig[ND];
        for (int j = 0; j < ND; ++j) dig[j] = 0;
        const bool l1 = P.qz == QS_SIGN_L1;
        // bit 0 stands for 2^-298 (squares) or 2^-149 (magnitudes)
        for (uint32_t e = un.emin; e <= un.emax; ++e) {
            unsigned long long* g = P.eacc + ((size_t)u * 256 + e) * 2;
            const unsigned long long a0 = g[0], a1 = g[1];
            if (!(a0 | a1)) continue;
            g[0] = 0ull; g[1] = 0ull;
            const int ee = e ? (int)e : 1;          // subnormals share the exponent of e = 1
            if (l1) {
                big_add(dig, ND, a0, ee - 1);
            } else {
                big_add(dig, ND, a0, 2 * (ee - 1));
                big_add(dig, ND, a1, 2 * (ee - 1) + 24);
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
}

// levels, signs, memory update; kept and sent counts per chunk
template <bool RANDK>
__device__ void stage_quant(const Plan& P, uint32_t* sh_u, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t total = *P.total_chunks;
    const bool sign_op = P.qz == QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        const ChunkCtx c = chunk_context(P, chunk, sh_u);
        const float N = c.un.norm, cs = P.cscale[c.seg];
        const uint32_t k = P.kseg[c.seg];
        float* mem = P.mem + (size_t)c.r * P.d;
        float val[PER];
        uint32_t idx[PER], key[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool in = off < c.un.c;
            val[i] = in ? P.cand_val[c.base + off] : 0.0f;
            idx[i] = in ? P.cand_idx[c.base + off] : 0xffffffffu;
            key[i] = RANDK ? (in ? P.cand_key[c.base + off] : 0u) : topk_key(val[i]);
        }
        uint32_t cnt = 0;                            // kept | sent << 16
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            if (off >= c.un.c) continue;
            uint32_t q = 0;
            if (is_kept<RANDK>(c.un, key[i], idx[i])) {
                const bool neg = val[i] < 0.0f;
                int level = 1;
                if (!sign_op) level = qsgd_level(val[i], N, P.s, philox_word(P, c.r, idx[i], 0u));
                q = Q_SEL | (neg ? Q_NEG : 0u) | (uint32_t)level;
                cnt += 1u;
                if (level) {
                    mem[idx[i]] = val[i] - coord_value(P, N, level, neg, cs, k);
                    cnt += 1u << 16;
                }
            }
            P.cand_q[c.base + off] = q;
        }
        cnt = warp_sum(cnt);
        if (lane == 0) sh_w[wid] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t t = 0;
            for (int w = 0; w < BT / 32; ++w) t += sh_w[w];
            P.chunk_cnt[chunk] = t;
        }
    }
}

// block 0: exclusive sums of kept / sent over the chunks, entries per unit, stream offsets,
// bit counts; writes the directory when a wire is given
__device__ void stage_chunk_scan(const Plan& P, const Active& act, uint32_t* sh) {
    if (blockIdx.x != 0) return;
    const uint32_t total = *P.total_chunks;
    uint32_t carry_k = 0, carry_s = 0;
    for (uint32_t base = 0; base <= total; base += BT) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < total ? P.chunk_cnt[i] : 0u;
        uint32_t tk, ts;
        const uint32_t ek = block_excl_scan(v & 0xffffu, sh, &tk);
        const uint32_t es = block_excl_scan(v >> 16, sh, &ts);
        if (i <= total) { P.chunk_sel[i] = carry_k + ek; P.chunk_nz[i] = carry_s + es; }
        carry_k += tk; carry_s += ts;
    }
    __syncthreads();
    for (uint32_t u = threadIdx.x; u < P.U; u += BT) {
        Unit& un = P.units[u];
        if (!((act.bits >> (u / P.nseg)) & 1u)) continue;
        const uint32_t kept = P.chunk_sel[un.chunk_base + un.nchunks] - P.chunk_sel[un.chunk_base];
        un.n = P.chunk_nz[un.chunk_base + un.nchunks] - P.chunk_nz[un.chunk_base];
        if (kept != P.kseg[u % P.nseg]) set_status(P, QS_STATE);
    }
    __syncthreads();
    const bool has_lvl = P.qz != QS_SIGN_L1;
    for (int w = threadIdx.x; w < act.n; w += BT) {
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

// ------------------------------------------------------------------ pack
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

__device__ void stage_pack_dir(const Plan& P, const Active& act, uint32_t* wire, long long stride, long long* bits_out) {
    const uint32_t items = (uint32_t)act.n * P.nseg;
    for (uint32_t i = blockIdx.x * BT + threadIdx.x; i < items; i += gridDim.x * BT) {
        const int r = act.r[i / P.nseg];
        const uint32_t g = i % P.nseg;
        const Unit& un = P.units[(size_t)r * P.nseg + g];
        uint32_t* row = wire + (size_t)r * stride;
        row[2 * g] = un.n;
        row[2 * g + 1] = __float_as_uint(un.norm);
        if (g == 0 && bits_out) bits_out[r] = P.bits[r];
    }
}

// streams of every segment, and the ordered kept list kept for inspection
__device__ void stage_pack(const Plan& P, uint32_t* wire, long long stride, uint32_t* sh_u, uint32_t* sh) {
    const uint32_t total = *P.total_chunks;
    const bool has_lvl = P.qz != QS_SIGN_L1;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        const ChunkCtx c = chunk_context(P, chunk, sh_u);
        uint32_t run_k = P.chunk_sel[chunk] - P.chunk_sel[c.un.chunk_base];
        uint32_t run_s = P.chunk_nz[chunk] - P.chunk_nz[c.un.chunk_base];
        const uint32_t bi = P.bidx[c.seg], lo = P.seg_off[c.seg];
        uint32_t* w_idx = wire + (size_t)c.r * stride + P.pay_off[c.u];
        uint32_t* w_sgn = w_idx + words_for(c.un.n, bi);
        uint32_t* w_lvl = w_sgn + words_for(c.un.n, 1);
        uint32_t* o_idx = P.sel_idx + (size_t)c.r * P.K + P.kprefix[c.seg];
        uint32_t* o_q = P.sel_q + (size_t)c.r * P.K + P.kprefix[c.seg];
        uint32_t q[PER], e[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            q[i] = off < c.un.c ? P.cand_q[c.base + off] : 0u;
            e[i] = off < c.un.c ? P.cand_idx[c.base + off] : 0u;
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t kept = (q[i] & Q_SEL) ? 1u : 0u, sent = (kept && (q[i] & 0xffffu)) ? 1u : 0u;
            uint32_t tot;
            const uint32_t ex = block_excl_scan(kept | (sent << 16), sh, &tot);
            if (kept) {
                const uint32_t jk = run_k + (ex & 0xffffu);
                o_idx[jk] = e[i];
                o_q[jk] = q[i];
                if (sent) {
                    const uint64_t js = run_s + (ex >> 16);
                    or_bits(w_idx, js * bi, bi, e[i] - lo);
                    if (q[i] & Q_NEG) atomicOr(&w_sgn[js >> 5], 1u << (js & 31u));
                    if (has_lvl) or_bits(w_lvl, js * P.bl, P.bl, (q[i] & 0xffffu) - 1u);
                }
            }
            run_k += tot & 0xffffu;
            run_s += tot >> 16;
        }
    }
}

// ------------------------------------------------------------------ master
// entry and stream offsets of each segment, read from the directory
__device__ void stage_dec_prep(const Plan& P, const Active& act, const uint32_t* wire, long long stride, uint32_t* sh) {
    const bool has_lvl = P.qz != QS_SIGN_L1;
    for (int w = blockIdx.x; w < act.n; w += gridDim.x) {
        const int r = act.r[w];
        const uint32_t* row = wire + (size_t)r * stride;
        uint32_t carry_e = 0, carry_w = 2u * P.nseg;
        for (uint32_t base = 0; base < (uint32_t)P.nseg; base += BT) {
            const uint32_t g = base + threadIdx.x;
            uint32_t n = 0, words = 0;
            if (g < (uint32_t)P.nseg) {
                n = row[2 * g];
                if (n > P.kseg[g]) { n = 0; set_status(P, QS_INVALID_ARG); }     // not a record of this plan
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
}

struct Entry { uint32_t seg, j, n, coord; const uint32_t* w_idx; };

__device__ __forceinline__ bool locate_entry(const Plan& P, const uint32_t* wire, long long stride, int r,
                                             uint32_t ent, Entry* out) {
    const uint32_t* eb = P.dec_ent + (size_t)r * (P.nseg + 1);
    if (ent >= eb[P.nseg]) return false;
    uint32_t lo = 0, hi = P.nseg;                // eb[lo] <= ent < eb[hi]
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

__device__ void stage_dec_mark(const Plan& P, const Active& act, const uint32_t* wire, long long stride) {
    const uint64_t total = (uint64_t)act.n * P.K;
    for (uint64_t id = (uint64_t)blockIdx.x * BT + threadIdx.x; id < total; id += (uint64_t)gridDim.x * BT) {
        const int r = act.r[id / P.K];
        Entry en;
        if (!locate_entry(P, wire, stride, r, (uint32_t)(id % P.K), &en)) continue;
        if (en.coord < P.d) atomicOr(&P.touch[en.coord], 1u << r);
        else set_status(P, QS_INVALID_ARG);
    }
}

// The lowest worker that sent an index owns it: it adds the values of all senders in increasing
// worker order, updates x, and in the fused round patches the workers' copies.
__device__ void stage_dec_apply(const Plan& P, const Active& act, const uint32_t* wire, long long stride, int patch) {
    const uint64_t total = (uint64_t)act.n * P.K;
    for (uint64_t id = (uint64_t)blockIdx.x * BT + threadIdx.x; id < total; id += (uint64_t)gridDim.x * BT) {
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
            const uint32_t* eb = P.dec_ent + (size_t)r2 * (P.nseg + 1);
            Entry e2;
            e2.seg = en.seg;
            e2.n = eb[en.seg + 1] - eb[en.seg];
            e2.w_idx = wire + (size_t)r2 * stride + P.dec_pay[(size_t)r2 * P.nseg + en.seg];
            uint32_t lo = 0, hi = e2.n;              // first position with index >= local
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

// xw_r <- x (and the anchors) for the active workers: the closing dense stage of a fused round
template <bool ALIGNED>
__device__ void stage_broadcast(const Plan& P, const Active& act) {
    const int lane = threadIdx.x & 31;
    for (uint32_t g = blockIdx.x * (BT / 32) + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * (BT / 32)) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        if (e0 >= P.d) continue;
        if (ALIGNED) {
            const float4 v = *reinterpret_cast<const float4*>(P.x + e0);
            for (int w = 0; w < act.n; ++w) {
                __stcs(reinterpret_cast<float4*>(P.xw + (size_t)act.r[w] * P.d + e0), v);
                if (P.anchors) __stcs(reinterpret_cast<float4*>(P.anchors + (size_t)act.r[w] * P.d + e0), v);
            }
        } else {
            for (uint32_t j = 0; j < 4 && e0 + j < P.d; ++j) {
                const float v = P.x[e0 + j];
                for (int w = 0; w < act.n; ++w) {
                    P.xw[(size_t)act.r[w] * P.d + e0 + j] = v;
                    if (P.anchors) P.anchors[(size_t)act.r[w] * P.d + e0 + j] = v;
                }
            }
        }
    }
}

// ------------------------------------------------------------------ the persistent kernel
template <bool RANDK>
__global__ void __launch_bounds__(BT) mid_kernel(const MidArgs a) {
    __shared__ uint32_t sh_scan[33];
    __shared__ uint32_t sh_small[8];              // unit id, prefix, select scratch
    __shared__ uint32_t sh_w[BT / 32];
    __shared__ int sh_abort;
    __shared__ __align__(16) unsigned char sh_big[FB_BINS * 4];   // fallback bins / radix bins / exponent sums
    const Plan& P = a.P;
    const Active& act = a.act;
    uint32_t* bins = reinterpret_cast<uint32_t*>(sh_big);
    if (threadIdx.x == 0) sh_abort = 0;
    uint32_t target = 0;
    if (P.trace && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        P.trace[0] = t;
        for (int i = 1; i < TRACE_SLOTS; ++i) P.trace[i] = 0;
    }
#define QS_BARRIER() do { if (!grid_barrier(P, target, &sh_abort)) return; } while (0)

    if (a.do_compress) {
        stage_scan(P, act, false, sh_scan);
        QS_BARRIER();
        stage_bounds(P, act, false);
        QS_BARRIER();
        int missed = 0;
        for (int w = 0; w < act.n; ++w) missed |= (int)P.fail[act.r[w]];
        if (missed) {                              // same value in every block
            QS_BARRIER();                          // nobody may clear a flag before all have read it
            stage_fb_hist<RANDK>(P, act, bins);
            QS_BARRIER();
            stage_fb_guess(P, act, sh_scan, &sh_small[0]);
            QS_BARRIER();
            stage_reflag<RANDK>(P, act);
            QS_BARRIER();
            stage_scan(P, act, true, sh_scan);
            QS_BARRIER();
            stage_bounds(P, act, true);
            QS_BARRIER();
        }
        stage_emit<RANDK>(P, act, sh_scan);
        stage_setup(P, act, sh_scan);
        QS_BARRIER();
        for (int level = 0; level < 4; ++level) {
            stage_hist<RANDK>(P, level, bins, &sh_small[0], &sh_small[1]);
            QS_BARRIER();
        }
        stage_final<RANDK>(P, &sh_small[2], sh_w);
        QS_BARRIER();
        stage_norm_accum<RANDK>(P, reinterpret_cast<unsigned long long(*)[2]>(sh_big), &sh_small[0]);
        QS_BARRIER();
        stage_norm_final(P);
        QS_BARRIER();
        stage_quant<RANDK>(P, &sh_small[0], sh_w);
        QS_BARRIER();
        stage_chunk_scan(P, act, sh_scan);
        QS_BARRIER();
    }
    if (a.do_pack) {
        stage_pack_dir(P, act, a.wire, a.stride, a.bits_out);
        stage_pack(P, a.wire, a.stride, &sh_small[0], sh_scan);
        if (a.do_decode) QS_BARRIER();
    }
    if (a.do_decode) {
        stage_dec_prep(P, act, a.wire, a.stride, sh_scan);
        QS_BARRIER();
        stage_dec_mark(P, act, a.wire, a.stride);
        QS_BARRIER();
        stage_dec_apply(P, act, a.wire, a.stride, a.patch);
    }
    if (a.do_broadcast) {
        QS_BARRIER();
        if (a.aligned) stage_broadcast<true>(P, act);
        else stage_broadcast<false>(P, act);
    }
#undef QS_BARRIER
    // the last block to leave resets the barrier for the next launch
    __syncthreads();
    if (P.trace && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        P.trace[TRACE_SLOTS - 1] = t;
    }
    if (threadIdx.x == 0) {
        if (atomicAdd(P.bar + 1, 1u) == gridDim.x - 1) {
            P.bar[0] = 0;
            P.bar[1] = 0;
        }
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
int mid_blocks_per_sm(bool randk) {
    int per_sm = 0;
    const cudaError_t e = randk ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mid_kernel<true>, BT, 0)
                                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mid_kernel<false>, BT, 0);
    return e == cudaSuccess ? per_sm : 0;
}

cudaError_t launch_mid(const Plan& P, const Active& act, int do_compress, int do_pack, int do_decode, int patch,
                       int do_broadcast, int aligned, uint32_t* wire, long long stride, long long* bits_out, int grid,
                       cudaStream_t st) {
    MidArgs a;
    a.P = P; a.act = act;
    a.do_compress = do_compress; a.do_pack = do_pack; a.do_decode = do_decode; a.patch = patch;
    a.do_broadcast = do_broadcast; a.aligned = aligned;
    a.wire = wire; a.stride = stride; a.bits_out = bits_out;
    void* params[] = {&a};
    const void* fn = P.sp == QS_RANDK ? (const void*)mid_kernel<true> : (const void*)mid_kernel<false>;
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(BT), params, 0, st);
}

void launch_export(const Plan& P, long long* sel_idx, int* level, uint8_t* sign, float* norm, long long* n,
                   int sms, cudaStream_t st) {
    export_kernel<<<sms * 4, 256, 0, st>>>(P, sel_idx, level, sign, norm, n);
}

}  // namespace qs
