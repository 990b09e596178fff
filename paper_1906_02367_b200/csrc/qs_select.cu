// Selection of the kept set from the candidate bitmap.
//
//   cand_count / cand_scan / unit_bounds   candidates per emission block, their prefix
//        sums, and the candidate range of every (worker, segment) unit; a unit with fewer
//        candidates than k marks its worker for the exact fallback
//   cand_emit        candidates written out in ascending coordinate order (index, value)
//   unit_setup       chunk numbering over all units
//   sel_hist x4      radix select over the 32-bit sort key, 8 bits per level
//   sel_final        threshold key, number above it, tie cut by lower index, and the
//                    prediction for the next round
//
// Everything here is O(candidates); order-dependent results come only from ordered scans.
#include "qs_kernels.h"

namespace qs {

__device__ __forceinline__ uint32_t popc4(const uint4 w) {
    return __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
}

// grid (nblk, nact): candidates of each emission block
__global__ void __launch_bounds__(256) cand_count_kernel(const Plan P, const Active act, const int only_failed) {
    __shared__ uint32_t sh[8];
    const int r = act.r[blockIdx.y];
    if (only_failed && !P.fail[r]) return;
    const uint32_t g = blockIdx.x * (uint32_t)EMIT_GROUPS + threadIdx.x;
    uint32_t c = 0;
    if (g < P.ngroups) c = popc4(reinterpret_cast<const uint4*>(P.bitmap)[(size_t)r * P.ngroups + g]);
    c = warp_sum(c);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int i = 0; i < 8; ++i) t += sh[i];
        P.blk_count[(size_t)r * P.nblk + blockIdx.x] = t;
    }
}

// grid (nact), 1024 threads: exclusive prefix of the block counts of one worker
__global__ void __launch_bounds__(1024) cand_scan_kernel(const Plan P, const Active act, const int only_failed) {
    __shared__ uint32_t sh[33];
    const int r = act.r[blockIdx.x];
    if (only_failed && !P.fail[r]) return;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < P.nblk; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < P.nblk ? P.blk_count[(size_t)r * P.nblk + i] : 0u;
        uint32_t total;
        const uint32_t ex = block_excl_scan(v, sh, &total);
        if (i < P.nblk) P.blk_base[(size_t)r * P.nblk + i] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) P.ncand[r] = carry;
}

// candidates of worker r among coordinates below p (warp-cooperative, all lanes get it)
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
            // lanes l with 4 l + j < pl
            const uint32_t nl = pl > j ? (pl - j + 3u) >> 2 : 0u;
            const uint32_t mask = nl >= 32u ? 0xffffffffu : ((1u << nl) - 1u);
            c += __popc(ws[j] & mask);
        }
        c += P.blk_base[(size_t)r * P.nblk + blk];
    }
    return warp_sum(c);
}

// one warp per unit: candidate range; marks the worker when a unit has too few
__global__ void __launch_bounds__(256) unit_bounds_kernel(const Plan P, const Active act, const int only_failed) {
    const int lane = threadIdx.x & 31;
    const uint32_t wid = blockIdx.x * 8u + (threadIdx.x >> 5);
    if (wid >= (uint32_t)act.n * P.nseg) return;
    const int r = act.r[wid / P.nseg];
    const uint32_t seg = wid % P.nseg;
    if (only_failed && !P.fail[r]) return;
    const uint32_t lo = cand_prefix(P, r, P.seg_off[seg], lane);
    const uint32_t hi = cand_prefix(P, r, P.seg_off[seg + 1], lane);
    if (lane == 0) {
        Unit& un = P.units[(size_t)r * P.nseg + seg];
        un.start = lo;
        un.c = hi - lo;
        if (hi - lo < P.kseg[seg]) {
            if (only_failed) set_status(P, QS_STATE);   // the exact pass cannot miss
            else atomicExch(&P.fail[r], 1u);
        }
    }
}

// grid (nblk, nact): candidates in ascending coordinate order
template <bool RANDK>
__global__ void __launch_bounds__(256) cand_emit_kernel(const Plan P, const Active act) {
    __shared__ uint32_t sh[33];
    const int r = act.r[blockIdx.y];
    const uint32_t g = blockIdx.x * (uint32_t)EMIT_GROUPS + threadIdx.x;
    uint4 w = make_uint4(0, 0, 0, 0);
    if (g < P.ngroups) w = reinterpret_cast<const uint4*>(P.bitmap)[(size_t)r * P.ngroups + g];
    uint32_t total;
    const uint32_t ex = block_excl_scan(popc4(w), sh, &total);
    if (total == 0) return;
    size_t pos = (size_t)r * P.cap + P.blk_base[(size_t)r * P.nblk + blockIdx.x] + ex;
    const float* mem = P.mem + (size_t)r * P.d;
    while (w.x | w.y | w.z | w.w) {
        // lowest coordinate 4 l + j still set
        uint32_t best = 0xffffffffu;
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

// single block: chunk numbering over the units of the active workers, in (worker, segment) order
__global__ void __launch_bounds__(1024) unit_setup_kernel(const Plan P, const Active act) {
    __shared__ uint32_t sh[33];
    uint32_t carry = 0, cands = 0;
    for (uint32_t base = 0; base < P.U; base += 1024) {
        const uint32_t u = base + threadIdx.x;
        uint32_t nch = 0;
        if (u < P.U) {
            const uint32_t r = u / P.nseg;
            Unit& un = P.units[u];
            if (!((act.bits >> r) & 1u)) un.c = 0;
            nch = (un.c + CHUNK - 1) / CHUNK;
            cands = un.c;
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

// unit owning a chunk: last unit with chunk_base <= chunk and nchunks > 0 (binary search)
__device__ uint32_t unit_of_chunk(const Plan& P, uint32_t chunk) {
    uint32_t lo = 0, hi = P.U;             // invariant: units[lo].chunk_base <= chunk
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (P.units[mid].chunk_base <= chunk) lo = mid; else hi = mid;
    }
    return lo;
}

// Within 256 bins (counted top-down) finds the bin holding rank kk (1-based): `bin`, and the
// number of keys in higher bins `above`.  Warp-cooperative; h may be global or shared.
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
        b = 255u - 8u * lane - 7u; a = run;      // fallback: lowest bin of the lane
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (run + v[i] >= kk) { b = 255u - 8u * lane - i; a = run; break; }
            run += v[i];
        }
    }
    *bin = __shfl_sync(0xffffffffu, b, owner);
    *above = __shfl_sync(0xffffffffu, a, owner);
}

// Key prefix fixed by levels 0 .. level-1 and the rank still to find inside it (warp 0 calls this).
__device__ void derive_prefix(const Plan& P, uint32_t u, uint32_t k, int level, int lane,
                              uint32_t* prefix, uint32_t* rank, uint32_t* above_total) {
    uint32_t pf = 0, kk = k, at = 0;
    for (int L = 0; L < level; ++L) {
        uint32_t bin, above;
        find_bin(P.hist + ((size_t)L * P.U + u) * 256, kk, lane, &bin, &above);
        pf = (pf << 8) | bin;
        kk -= above;
        at += above;
    }
    *prefix = pf; *rank = kk; *above_total = at;
}

template <bool RANDK>
__device__ __forceinline__ uint32_t cand_sort_key(const Plan& P, size_t pos) {
    return RANDK ? P.cand_key[pos] : topk_key(P.cand_val[pos]);
}

// One level of the radix select: histogram of the level's digit among keys matching the prefix.
template <bool RANDK>
__global__ void __launch_bounds__(256) sel_hist_kernel(const Plan P, const int level) {
    __shared__ uint32_t sh_hist[256];
    __shared__ uint32_t sh_u, sh_prefix;
    const int lane = threadIdx.x & 31;
    const uint32_t total = *P.total_chunks;
    for (uint32_t chunk = blockIdx.x; chunk < total; chunk += gridDim.x) {
        if (threadIdx.x < 32) {
            const uint32_t u = unit_of_chunk(P, chunk);
            uint32_t prefix, rank, at;
            derive_prefix(P, u, P.kseg[u % P.nseg], level, lane, &prefix, &rank, &at);
            if (lane == 0) { sh_u = u; sh_prefix = prefix; }
        }
        sh_hist[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t u = sh_u, prefix = sh_prefix;
        const Unit un = P.units[u];
        const uint32_t r = u / P.nseg;
        const uint32_t first = (chunk - un.chunk_base) * CHUNK;
        const size_t base = (size_t)r * P.cap + un.start;
        const int shift = 24 - 8 * level;
#pragma unroll 1
        for (int i = 0; i < CHUNK / 256; ++i) {
            const uint32_t off = first + i * 256 + threadIdx.x;
            bool valid = off < un.c;
            uint32_t digit = 0;
            if (valid) {
                const uint32_t sk = cand_sort_key<RANDK>(P, base + off);
                valid = level == 0 || (sk >> (32 - 8 * level)) == prefix;
                digit = (sk >> shift) & 255u;
            }
            const uint32_t live = __ballot_sync(0xffffffffu, valid);
            if (valid) {
                const uint32_t peers = __match_any_sync(live, digit);
                if (lane == __ffs(peers) - 1) atomicAdd(&sh_hist[digit], __popc(peers));
            }
        }
        __syncthreads();
        const uint32_t v = sh_hist[threadIdx.x];
        if (v) atomicAdd(&P.hist[((size_t)level * P.U + u) * 256 + threadIdx.x], v);
        __syncthreads();
    }
}

// grid U: threshold key, tie cut and next prediction of one unit; clears its histograms.
template <bool RANDK>
__global__ void __launch_bounds__(256) sel_final_kernel(const Plan P) {
    __shared__ uint32_t sh_tau, sh_t, sh_ceq, sh_found, sh_run;
    __shared__ uint32_t sh_w[8];
    const uint32_t u = blockIdx.x;
    const Unit un = P.units[u];
    if (un.c == 0) return;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t seg = u % P.nseg, r = u / P.nseg, k = P.kseg[seg];
    if (wid == 0) {
        uint32_t prefix, rank, above;
        derive_prefix(P, u, k, 4, lane, &prefix, &rank, &above);
        if (lane == 0) {
            sh_tau = prefix;
            sh_t = k - above;                      // kept among keys equal to tau
            sh_ceq = P.hist[((size_t)3 * P.U + u) * 256 + (prefix & 255u)];
            sh_found = 0xffffffffu;
            sh_run = 0;
        }
    }
    __syncthreads();
    for (int L = 0; L < 4; ++L) P.hist[((size_t)L * P.U + u) * 256 + threadIdx.x] = 0;
    const uint32_t tau = sh_tau, t = sh_t, ceq = sh_ceq;
    uint32_t tie_max = 0xffffffffu;
    if (ceq > t) {
        // more equal keys than slots: the t lowest coordinates win; walk the list in order
        const size_t base = (size_t)r * P.cap + un.start;
        for (uint32_t first = 0; first < un.c; first += 256) {
            const uint32_t off = first + threadIdx.x;
            const bool eq = off < un.c && cand_sort_key<RANDK>(P, base + off) == tau;
            const uint32_t bal = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) sh_w[wid] = __popc(bal);
            __syncthreads();
            uint32_t before = sh_run;
            for (int w = 0; w < wid; ++w) before += sh_w[w];
            const uint32_t mine = before + __popc(bal & ((1u << lane) - 1u));
            if (eq && mine == t - 1) sh_found = P.cand_idx[base + off];
            __syncthreads();
            if (threadIdx.x == 0) { uint32_t s = 0; for (int w = 0; w < 8; ++w) s += sh_w[w]; sh_run += s; }
            __syncthreads();
            if (sh_found != 0xffffffffu) break;
        }
        tie_max = sh_found;
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

// ------------------------------------------------------------------ launchers
void launch_candidates(const Plan& P, const Active& act, int only_failed, cudaStream_t st) {
    cand_count_kernel<<<dim3(P.nblk, act.n), 256, 0, st>>>(P, act, only_failed);
    cand_scan_kernel<<<act.n, 1024, 0, st>>>(P, act, only_failed);
    const uint32_t warps = (uint32_t)act.n * P.nseg;
    unit_bounds_kernel<<<(warps + 7) / 8, 256, 0, st>>>(P, act, only_failed);
}

void launch_select(const Plan& P, const Active& act, int sms, cudaStream_t st) {
    const bool rk = P.sp == QS_RANDK;
    const dim3 ge(P.nblk, act.n);
    if (rk) cand_emit_kernel<true><<<ge, 256, 0, st>>>(P, act);
    else cand_emit_kernel<false><<<ge, 256, 0, st>>>(P, act);
    unit_setup_kernel<<<1, 1024, 0, st>>>(P, act);
    const int grid = chunk_grid(P, sms);
    for (int level = 0; level < 4; ++level) {
        if (rk) sel_hist_kernel<true><<<grid, 256, 0, st>>>(P, level);
        else sel_hist_kernel<false><<<grid, 256, 0, st>>>(P, level);
    }
    if (rk) sel_final_kernel<true><<<P.U, 256, 0, st>>>(P);
    else sel_final_kernel<false><<<P.U, 256, 0, st>>>(P);
}

}  // namespace qs
