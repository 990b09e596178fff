// Everything between the dense pass and the end of the round, as ONE persistent kernel.
//
// The work after the dense pass is O(candidates): small, and made of a dozen steps that each
// need the previous one finished everywhere.  Launched separately they cost more in launch
// gaps and cold starts than in work, so they run here as stages of one cooperative launch
// (every block resident), separated by grid-wide barriers with a bounded wait:
//
//   candidates  the per-tile candidate runs left by the dense pass are gathered into each worker's
//               ordered list (index, value) with the first select histogram and the segment
//               boundaries; the exact fallback for workers whose predicted threshold left a unit
//               short (histogram of the top key bits, new threshold, candidates found again from
//               the stored u)
//   select      radix select over the 32-bit sort key (4 levels of 8 bits), tie cut by lower
//               index, next round's prediction; units with short candidate lists are selected
//               from by one block (or warp) each, with block barriers only, beside the first level
//   quantize    exact norm of the kept values (or their smallest and largest), levels and signs
//               (Philox stream 0), m <- u - g, ordered positions of kept and sent entries
//   pack        directory and the bit streams of every segment
//   closing     whole round: the master's update and the broadcast in one pass over x (the kept
//               entries are found again in the dense pass's runs), the records written beside it
//   decode      separate master call: senders of every index from the record words, then one
//               owner per index adds the values in worker order and updates x
//
// Order-dependent results come only from ordered scans, never from the order of atomics.
#include "qs_bulk.cuh"
#include "qs_kernels.h"

namespace qs {

constexpr int BT = 256;                    // threads per block of the persistent kernel
constexpr int PER = CHUNK / BT;            // candidates per thread and chunk

struct MidArgs {
    Plan P;
    Active act;
    int do_compress, do_pack, do_decode, do_broadcast, aligned;
    uint32_t* wire;
    long long stride, wire_words;
    long long* bits_out;
};

// ------------------------------------------------------------------ grid barrier
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// All blocks of the cooperative launch meet here (every block is resident).  The wait is
// bounded: a block that gives up records QS_TIMEOUT and every block leaves the stages at its next
// barrier.
__device__ __forceinline__ bool grid_barrier(const Plan& P, uint32_t& target, int* sh_abort) {
    const bool first = target == 0;
    target += gridDim.x;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        // (test of the bounded wait: one block stays away once, the others' waits run out)
        if (!(P.test_miss_barrier && first && blockIdx.x == 0)) atomicAdd(P.bar, 1u);
        uint32_t spins = 0;
        while (ld_acquire(P.bar) < target) {
            if (++spins > P.spin_limit) {
                atomicCAS(P.status, 0, QS_TIMEOUT);
                *sh_abort = 1;
                break;
            }
            __nanosleep(32);
        }
        // (the acquiring load that saw the last arrival orders this thread behind every block's
        // writes, and the block barrier below passes that on to the other threads)
        if (P.trace && blockIdx.x == 0) {          // time at which every block has finished the stage
            const uint32_t slot = target / gridDim.x;
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            if (slot < TRACE_SLOTS - 4) P.trace[slot] = t;
        }
    }
    __syncthreads();
    return *sh_abort == 0;
}

template <bool RANDK>
__device__ __forceinline__ uint32_t sort_key(const Plan& P, size_t pos) {
    return RANDK ? P.cand_key[pos] : topk_key(P.cand_val[pos]);
}

// quantizers that send every kept entry with level 1: nothing about the record depends on the norm
__device__ __forceinline__ bool qz_early(int qz) { return qz_is_sign(qz) || qz == QS_NONE; }

// Unit table: where each (worker, segment) unit's candidates start, how many there are, and the
// number of chunks before it.  Every block builds it for itself in shared memory.
struct Tab {
    const uint32_t* start;
    const uint32_t* c;
    const uint32_t* cb;      // U + 1 entries
    const uint32_t* lb;      // U + 1 entries: chunks of long units before each unit
    uint32_t total_chunks;
    uint32_t total_long;     // chunks of the units that take the grid-wide select
    uint32_t short_c;        // a unit with at most this many candidates is selected from by one block on its own
    bool any_short;          // there is such a unit
    bool fast;               // pack finds its own positions: few chunks per unit, and the streams' places are known
};

__device__ __forceinline__ uint32_t segment_of(const Plan& P, uint32_t e) {
    if (P.nseg == 1) return 0;
    uint32_t sq = P.grp_seg[e >> 7];
    while (sq + 1 < (uint32_t)P.nseg && e >= P.seg_off[sq + 1]) ++sq;
    return sq;
}

// ------------------------------------------------------------------ candidates
// One candidate block (BLK_TILES tiles of one worker): its candidates are copied from the tiles'
// fixed places into the worker's ordered list, their top key digit is counted for the select,
// and the list positions of the segment boundaries inside the block are recorded.
template <bool RANDK>
__device__ void stage_order(const Plan& P, const Active& act, uint32_t only_mask, uint32_t* sh_bins) {
    const int lane = threadIdx.x & 31;
    // one segment and few workers: the top-byte counts, which pile up on two or three bins per
    // worker, are gathered per block in shared memory (8 workers x 256 bins) and flushed once
    const bool local_bins = P.nseg == 1 && act.n <= 8;
    if (local_bins) {
        for (int i = threadIdx.x; i < FB_BINS; i += BT) sh_bins[i] = 0;
        __syncthreads();
    }
    const uint32_t items = P.nblk * (uint32_t)act.n;
    const uint32_t nwarps = gridDim.x * (BT / 32);
    for (uint32_t item = blockIdx.x * (BT / 32) + (threadIdx.x >> 5); item < items; item += nwarps) {
        const uint32_t wslot = item / P.nblk;
        const int r = act.r[wslot];
        if (only_mask && !((only_mask >> r) & 1u)) continue;
        const uint32_t blk = item % P.nblk;
        const uint32_t sup = blk / SUP_BLOCKS;
        // candidates of this worker in earlier blocks: whole super-blocks, then blocks of this one
        uint32_t part = 0;
        for (uint32_t i = lane; i < sup; i += 32) part += P.sup_count[(size_t)r * P.nsup + i];
        for (uint32_t i = sup * SUP_BLOCKS + lane; i < blk; i += 32) part += P.blk_count[(size_t)r * P.nblk + i];
        const uint32_t base = warp_sum(part);
        const uint32_t t0 = blk * BLK_TILES;
        const uint32_t tc = lane < BLK_TILES ? P.tile_cnt[(size_t)r * P.nblk * BLK_TILES + t0 + lane] : 0u;
        const uint32_t incl = warp_incl_scan(tc, lane);          // lanes >= BLK_TILES repeat the total
        const uint32_t n = __shfl_sync(0xffffffffu, incl, 31);
        const size_t row = (size_t)r * P.cap;
        constexpr int OB = 4;                     // entries per lane whose reads are issued together
        for (uint32_t eb = 0; eb < n; eb += 32 * OB) {
            uint2 ent[OB];
#pragma unroll
            for (int q = 0; q < OB; ++q) {
                const uint32_t e = eb + q * 32 + lane;
                // tile of entry e: the number of tiles whose inclusive count is <= e
                uint32_t t = 0, before = 0;
#pragma unroll
                for (int i = 0; i < BLK_TILES; ++i) {
                    const uint32_t inc_i = __shfl_sync(0xffffffffu, incl, i);
                    if (e >= inc_i) { t = i + 1; before = inc_i; }
                }
                ent[q] = make_uint2(0u, 0u);
                if (e < n) ent[q] = P.stage[row + (size_t)(t0 + t) * STILE + (e - before)];
            }
#pragma unroll
            for (int q = 0; q < OB; ++q) {
                const uint32_t e = eb + q * 32 + lane;
                const bool valid = e < n;
                const uint32_t idx = ent[q].x;
                uint32_t sk = 0, seg = 0;
                if (valid) {
                    const float val = __uint_as_float(ent[q].y);
                    sk = RANDK ? ~philox_word(P, (uint32_t)r, idx, 1u) : topk_key(val);
                    P.cand_idx[row + base + e] = idx;
                    P.cand_val[row + base + e] = val;
                    if (RANDK) P.cand_key[row + base + e] = sk;
                    seg = segment_of(P, idx);
                }
                // level 0 of the radix select: count the top key byte per unit.  Shared memory takes
                // an add per lane as it comes (equal addresses cost nothing extra there); adds to
                // global memory are gathered per warp first
                if (local_bins) {
                    if (valid) atomicAdd(&sh_bins[wslot * 256 + (sk >> 24)], 1u);
                } else {
                    const uint32_t tag = (seg << 8) | (sk >> 24);
                    const uint32_t live = __ballot_sync(0xffffffffu, valid);
                    if (valid) {
                        const uint32_t peers = __match_any_sync(live, tag);
                        if (lane == __ffs(peers) - 1) atomicAdd(&P.hist[((size_t)r * P.nseg + seg) * 256 + (sk >> 24)], __popc(peers));
                    }
                }
            }
        }
        __syncwarp();                             // the block's part of the ordered list is written
        // segment boundaries inside this block: position of the first candidate at or after each
        const uint32_t lo = blk * (uint32_t)(BLK_TILES * STILE);
        const uint64_t hi64 = (uint64_t)lo + BLK_TILES * STILE;
        const uint32_t hi = hi64 < P.d ? (uint32_t)hi64 : P.d;
        uint32_t s_lo = 0;
        if (P.nseg > 1) {
            const uint32_t sc = P.grp_seg[lo >> 7];
            s_lo = P.seg_off[sc] == lo ? sc : sc + 1;
        } else if (blk != 0) {
            s_lo = 1;
        }
        uint32_t* ss = P.seg_start + (size_t)r * (P.nseg + 1);
        for (uint32_t sgm = s_lo + lane; sgm < (uint32_t)P.nseg && P.seg_off[sgm] < hi; sgm += 32) {
            const uint32_t bound = P.seg_off[sgm];
            uint32_t a = 0, b = n;               // first entry of the block with index >= bound
            while (a < b) {
                const uint32_t m = (a + b) >> 1;
                if (P.cand_idx[row + base + m] < bound) a = m + 1; else b = m;
            }
            ss[sgm] = base + a;
        }
        if (blk == P.nblk - 1 && lane == 0) ss[P.nseg] = base + n;
    }
    if (local_bins) {
        __syncthreads();
        for (int i = threadIdx.x; i < act.n * 256; i += BT)
            if (sh_bins[i]) atomicAdd(&P.hist[(size_t)act.r[i >> 8] * 256 + (i & 255)], sh_bins[i]);
        __syncthreads();
    }
}

constexpr uint32_t ORDER_ITEMS_MAX = 8192;    // words of shared memory the order stage may use for its sums

// Exclusive sums in place over a[0..n) in shared memory, started at `base`; a[n] receives the end.
__device__ void smem_excl_scan(uint32_t* a, uint32_t n, uint32_t base, uint32_t* sh_scan) {
    const uint32_t per = (n + BT - 1) / BT;
    const uint32_t i0 = threadIdx.x * per < n ? threadIdx.x * per : n;
    const uint32_t i1 = i0 + per < n ? i0 + per : n;
    uint32_t sum = 0;
    for (uint32_t i = i0; i < i1; ++i) sum += a[i];
    uint32_t total;
    uint32_t run = base + block_excl_scan(sum, sh_scan, &total);
    for (uint32_t i = i0; i < i1; ++i) {
        const uint32_t c = a[i];
        a[i] = run;
        run += c;
    }
    if (threadIdx.x == 0) a[n] = base + total;
    __syncthreads();
}

// largest i in [0, n) with a[i] <= g (a ascending, a[0] <= g)
__device__ __forceinline__ uint32_t last_not_above(const uint32_t* a, uint32_t n, uint32_t g) {
    uint32_t lo = 0, hi = n;
    while (hi - lo > 1) {
        const uint32_t m = (lo + hi) >> 1;
        if (a[m] <= g) lo = m; else hi = m;
    }
    return lo;
}

// The same stage with the work dealt evenly, for act.n x nsup <= ORDER_SUPS_MAX.  Candidates pile up
// where the coordinates are large (a few tensors), so a split by region leaves most warps idle.
// Here every block sums the (worker, super-block) counts in shared memory, takes an equal share of
// the worker-major candidate sequence, wherever it lies, sums the block counts of the super-blocks
// its share touches (a window at a time), and copies: entry -> block by binary search, -> tile by
// the block's sixteen tile counts, -> its place in the tile's run.  No block reads more counts
// than its share needs: a table every block reads in full is a hot spot in the L2.
constexpr uint32_t ORDER_WIN = (ORDER_ITEMS_MAX - ORDER_SUPS_MAX - 8) / SUP_BLOCKS;   // super-blocks per window

template <bool RANDK>
__device__ void stage_order_even(const Plan& P, const Active& act, uint32_t only_mask, uint32_t* sh_bins,
                                 uint32_t* sh_tab, uint32_t* sh_scan) {
    const int lane = threadIdx.x & 31;
    // one segment: the top-byte counts, which pile up on two or three bins per worker, are gathered
    // per block in shared memory for the eight workers from the first one of the block's share on
    const bool local_bins = P.nseg == 1;
    if (local_bins)
        for (int i = threadIdx.x; i < FB_BINS; i += BT) sh_bins[i] = 0;
    uint32_t ws0 = 0;                                    // first worker slot with local bins
    uint32_t* psup = sh_tab;                             // ns + 1 sums over (worker, super-block)
    uint32_t* pre = sh_tab + ORDER_SUPS_MAX + 4;         // sums over the blocks of the current window
    const uint32_t ns = P.nsup * (uint32_t)act.n;
    for (uint32_t i = threadIdx.x; i < ns; i += BT) {
        const uint32_t wslot = i / P.nsup;
        const int r = act.r[wslot];
        psup[i] = (only_mask && !((only_mask >> r) & 1u)) ? 0u : P.sup_count[(size_t)r * P.nsup + (i - wslot * P.nsup)];
    }
    __syncthreads();
    smem_excl_scan(psup, ns, 0u, sh_scan);
    const uint32_t total = psup[ns];
    const uint32_t g_lo = (uint32_t)(((uint64_t)total * blockIdx.x) / gridDim.x);
    const uint32_t g_hi = (uint32_t)(((uint64_t)total * (blockIdx.x + 1u)) / gridDim.x);
    if (g_lo < g_hi) {                                   // the same for every thread of the block
        const uint32_t s_a = last_not_above(psup, ns, g_lo), s_b = last_not_above(psup, ns, g_hi - 1u);
        ws0 = s_a / P.nsup;
        for (uint32_t sw = s_a; sw <= s_b; sw += ORDER_WIN) {
            const uint32_t se = sw + ORDER_WIN < s_b + 1u ? sw + ORDER_WIN : s_b + 1u;
            const uint32_t nbw = (se - sw) * SUP_BLOCKS;
            for (uint32_t i = threadIdx.x; i < nbw; i += BT) {
                const uint32_t sg = sw + i / SUP_BLOCKS;
                const uint32_t wslot = sg / P.nsup;
                const uint32_t blk = (sg - wslot * P.nsup) * SUP_BLOCKS + i % SUP_BLOCKS;
                const int r = act.r[wslot];
                const bool out = blk >= P.nblk || (only_mask && !((only_mask >> r) & 1u));
                pre[i] = out ? 0u : P.blk_count[(size_t)r * P.nblk + blk];
            }
            __syncthreads();
            smem_excl_scan(pre, nbw, psup[sw], sh_scan);
            if (pre[nbw] != psup[se]) set_status(P, QS_STATE);   // the two levels of counts disagree
            const uint32_t lo = g_lo > psup[sw] ? g_lo : psup[sw];
            const uint32_t hi = g_hi < psup[se] ? g_hi : psup[se];
            constexpr int OB = 4;                 // entries per thread whose reads are issued together
            for (uint32_t g0 = lo; g0 < hi; g0 += BT * OB) {
                uint2 ent[OB];
                uint32_t wsl[OB], pos[OB];
#pragma unroll
                for (int q = 0; q < OB; ++q) {
                    const uint32_t g = g0 + q * BT + threadIdx.x;
                    ent[q] = make_uint2(0u, 0u);
                    wsl[q] = 0; pos[q] = 0;
                    if (g < hi) {
                        const uint32_t a = last_not_above(pre, nbw, g);      // the block that holds entry g
                        const uint32_t sg = sw + a / SUP_BLOCKS;
                        const uint32_t wslot = sg / P.nsup;
                        const uint32_t blk = (sg - wslot * P.nsup) * SUP_BLOCKS + a % SUP_BLOCKS;
                        const int r = act.r[wslot];
                        uint32_t off = g - pre[a];
                        const uint32_t t0 = blk * BLK_TILES;
                        // the block's sixteen tile counts: 64 aligned bytes
                        const uint4* tq = reinterpret_cast<const uint4*>(P.tile_cnt + (size_t)r * P.nblk * BLK_TILES + t0);
                        const uint4 q0 = tq[0], q1 = tq[1], q2 = tq[2], q3 = tq[3];
                        const uint32_t tc[BLK_TILES] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w,
                                                        q2.x, q2.y, q2.z, q2.w, q3.x, q3.y, q3.z, q3.w};
                        uint32_t t = 0;
                        bool found = false;
#pragma unroll
                        for (int i = 0; i < BLK_TILES; ++i) {
                            if (!found) {
                                if (off < tc[i]) { t = i; found = true; }
                                else off -= tc[i];
                            }
                        }
                        wsl[q] = wslot;
                        pos[q] = g - psup[wslot * P.nsup];
                        if (found) ent[q] = P.stage[(size_t)r * P.cap + (size_t)(t0 + t) * STILE + off];
                        else set_status(P, QS_STATE);    // the counts of the dense pass disagree with each other
                    }
                }
#pragma unroll
                for (int q = 0; q < OB; ++q) {
                    const uint32_t g = g0 + q * BT + threadIdx.x;
                    const bool valid = g < hi;
                    const uint32_t idx = ent[q].x;
                    const int r = act.r[wsl[q]];
                    uint32_t sk = 0, seg = 0;
                    if (valid) {
                        const float val = __uint_as_float(ent[q].y);
                        sk = RANDK ? ~philox_word(P, (uint32_t)r, idx, 1u) : topk_key(val);
                        const size_t o = (size_t)r * P.cap + pos[q];
                        P.cand_idx[o] = idx;
                        P.cand_val[o] = val;
                        if (RANDK) P.cand_key[o] = sk;
                        seg = segment_of(P, idx);
                    }
                    // level 0 of the radix select: count the top key byte per unit (shared memory: an add
                    // per lane; global memory: gathered per warp first)
                    const bool local = local_bins && wsl[q] - ws0 < 8u;
                    if (valid && local) atomicAdd(&sh_bins[(wsl[q] - ws0) * 256 + (sk >> 24)], 1u);
                    const uint32_t tag = (wsl[q] << 24) | (seg << 8) | (sk >> 24);
                    const uint32_t live = __ballot_sync(0xffffffffu, valid && !local);
                    if (valid && !local) {
                        const uint32_t peers = __match_any_sync(live, tag);
                        if (lane == __ffs(peers) - 1) atomicAdd(&P.hist[((size_t)r * P.nseg + seg) * 256 + (sk >> 24)], __popc(peers));
                    }
                }
            }
            __syncthreads();                      // the window's sums are replaced next
        }
    }
    // where each segment's candidates begin in the worker's ordered list
    const uint32_t nb = (uint32_t)act.n * (uint32_t)(P.nseg + 1);
    for (uint32_t it = blockIdx.x * BT + threadIdx.x; it < nb; it += gridDim.x * BT) {
        const uint32_t wslot = it / (uint32_t)(P.nseg + 1), sgm = it - wslot * (uint32_t)(P.nseg + 1);
        const int r = act.r[wslot];
        if (only_mask && !((only_mask >> r) & 1u)) continue;
        uint32_t* ss = P.seg_start + (size_t)r * (P.nseg + 1);
        const uint32_t wbase = psup[wslot * P.nsup];
        if (sgm == (uint32_t)P.nseg) { ss[sgm] = psup[(wslot + 1) * P.nsup] - wbase; continue; }
        const uint32_t bound = P.seg_off[sgm];
        const uint32_t tile = bound / (uint32_t)STILE, blk = tile / (uint32_t)BLK_TILES, sup = blk / (uint32_t)SUP_BLOCKS;
        uint32_t at = psup[wslot * P.nsup + sup] - wbase;
        for (uint32_t bq = sup * SUP_BLOCKS; bq < blk; ++bq) at += P.blk_count[(size_t)r * P.nblk + bq];
        for (uint32_t t = blk * BLK_TILES; t < tile; ++t) at += P.tile_cnt[(size_t)r * P.nblk * BLK_TILES + t];
        const uint2* run = P.stage + (size_t)r * P.cap + (size_t)tile * STILE;
        uint32_t a = 0, b = P.tile_cnt[(size_t)r * P.nblk * BLK_TILES + tile];   // first entry of the tile with index >= bound
        while (a < b) {
            const uint32_t m = (a + b) >> 1;
            if (run[m].x < bound) a = m + 1; else b = m;
        }
        ss[sgm] = at + a;
    }
    if (local_bins) {
        __syncthreads();
        for (int i = threadIdx.x; i < 8 * 256; i += BT)
            if (sh_bins[i] && ws0 + (uint32_t)(i >> 8) < (uint32_t)act.n)
                atomicAdd(&P.hist[(size_t)act.r[ws0 + (uint32_t)(i >> 8)] * 256 + (i & 255)], sh_bins[i]);
        __syncthreads();
    }
}

// Builds the unit table; returns the workers (bit mask) that have a unit with fewer candidates
// than k.  Every block computes the same thing from the same data.
__device__ uint32_t build_table(const Plan& P, const Active& act, uint32_t* t_start, uint32_t* t_c, uint32_t* t_cb,
                                uint32_t* t_lb, uint32_t* sh, uint32_t* sh_flag, Tab* tab) {
    if (threadIdx.x == 0) { sh_flag[0] = 0; sh_flag[1] = 0; sh_flag[2] = 0; sh_flag[3] = 0; }   // workers that fell short; the longest list; units; any short unit
    __syncthreads();
    uint32_t carry = 0;
    for (uint32_t ub = 0; ub < P.U; ub += BT) {
        const uint32_t u = ub + threadIdx.x;
        uint32_t start = 0, c = 0;
        if (u < P.U) {
            const uint32_t r = u / P.nseg, seg = u % P.nseg;
            if ((act.bits >> r) & 1u) {
                const uint32_t* ss = P.seg_start + (size_t)r * (P.nseg + 1);
                start = ss[seg];
                c = ss[seg + 1] - start;
                if (c < P.kseg[seg]) atomicOr(sh_flag, 1u << r);
                atomicMax(sh_flag + 1, c);
                // lists that would keep a block busy for a while: weight 2, or 1 up to half the cap
                if (c > (uint32_t)BT && c <= P.unit_cap) atomicAdd(sh_flag + 2, c > P.unit_cap / 2u ? 2u : 1u);
            }
        }
        uint32_t total;
        const uint32_t ex = block_excl_scan((c + CHUNK - 1) / CHUNK, sh, &total);
        if (u < P.U) { t_start[u] = start; t_c[u] = c; t_cb[u] = carry + ex; }
        carry += total;
    }
    if (threadIdx.x == 0) t_cb[P.U] = carry;
    __syncthreads();
    tab->start = t_start; tab->c = t_c; tab->cb = t_cb; tab->lb = t_lb; tab->total_chunks = carry;
    const uint32_t longest = sh_flag[1];
    // the streams' places: one segment, or a quantizer that sends every kept entry (fixed places)
    tab->fast = (P.nseg == 1 || qz_sends_all(P.qz)) && (longest + CHUNK - 1) / CHUNK <= 1024u;
    // Which units one block selects from on its own (block barriers only), and which take the
    // grid-wide radix levels: every list up to the cap when there is a block for each list that
    // would keep one busy for a while, two lists of up to half the cap counting as one (lists are
    // dealt largest first); otherwise only the lists of at most one candidate per thread.
    uint32_t short_c = 0;
    if (P.unit_cap) {
        const bool all = sh_flag[2] <= 2u * gridDim.x;
        short_c = all ? P.unit_cap : (P.unit_cap < (uint32_t)BT ? P.unit_cap : (uint32_t)BT);
    }
    tab->short_c = short_c;
    carry = 0;
    for (uint32_t ub = 0; ub < P.U; ub += BT) {
        const uint32_t u = ub + threadIdx.x;
        const uint32_t c = u < P.U ? t_c[u] : 0u;
        if (c && c <= short_c) sh_flag[3] = 1u;            // some unit is short (same value from every writer)
        uint32_t total;
        const uint32_t ex = block_excl_scan(c > short_c ? (c + CHUNK - 1) / CHUNK : 0u, sh, &total);
        if (u < P.U) t_lb[u] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) t_lb[P.U] = carry;
    __syncthreads();
    tab->total_long = carry;
    tab->any_short = sh_flag[3] != 0u;
    return sh_flag[0];
}

// The unit table where every block can read it.  Up to UT_MAX units every block builds its own
// copy in shared memory.  More units than that: block 0 builds the table in global memory, writes
// the few numbers that go with it, and after a grid barrier every block reads it from there.
// Returns false when that barrier gave up.
__device__ bool table_step(const Plan& P, const Active& act, uint32_t* sh_tab, uint32_t* sh_scan, uint32_t* sh_flag, Tab* tab,
                           uint32_t* missed, uint32_t& target, int* sh_abort) {
    if (P.U <= (uint32_t)UT_MAX) {
        *missed = build_table(P, act, sh_tab, sh_tab + UT_MAX, sh_tab + 2 * UT_MAX, sh_tab + 3 * UT_MAX + 4, sh_scan, sh_flag, tab);
        return true;
    }
    uint32_t* g = P.gtab;
    const uint32_t n = P.U + 1u;
    if (blockIdx.x == 0) {
        const uint32_t m = build_table(P, act, g, g + n, g + 2 * n, g + 3 * n, sh_scan, sh_flag, tab);
        if (threadIdx.x == 0) {
            uint32_t* info = g + 4 * n;
            info[0] = tab->total_chunks; info[1] = tab->total_long; info[2] = tab->short_c;
            info[3] = tab->any_short ? 1u : 0u; info[4] = tab->fast ? 1u : 0u; info[5] = m;
        }
    }
    if (!grid_barrier(P, target, sh_abort)) return false;
    const uint32_t* info = g + 4 * n;
    tab->start = g; tab->c = g + n; tab->cb = g + 2 * n; tab->lb = g + 3 * n;
    tab->total_chunks = info[0]; tab->total_long = info[1]; tab->short_c = info[2];
    tab->any_short = info[3] != 0u; tab->fast = info[4] != 0u;
    *missed = info[5];
    return true;
}

// histogram of the top 11 key bits of one stretch of one segment, for missed workers
template <bool RANDK>
__device__ void stage_fb_hist(const Plan& P, const Active& act, uint32_t missed, uint32_t* sh_bins) {
    const uint32_t items = P.nfb * (uint32_t)act.n;
    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int r = act.r[item / P.nfb];
        if (!((missed >> r) & 1u)) continue;
        const FbBlock blk = P.fb_tab[item % P.nfb];
        for (int i = threadIdx.x; i < FB_BINS; i += BT) sh_bins[i] = 0;
        __syncthreads();
        const size_t row = (size_t)r * P.d;
        for (uint32_t base = 0; base < blk.len; base += BT) {
            const uint32_t i = base + threadIdx.x;
            if (i < blk.len) {
                const uint32_t e = blk.start + i;
                const uint32_t sk = RANDK ? ~philox_word(P, (uint32_t)r, e, 1u) : topk_key(P.mem[row + e]);
                atomicAdd(&sh_bins[sk >> FB_SHIFT], 1u);
            }
        }
        __syncthreads();
        uint32_t* out = P.fb_hist + ((size_t)r * P.nseg + blk.seg) * FB_BINS;
        for (int i = threadIdx.x; i < FB_BINS; i += BT)
            if (sh_bins[i]) atomicAdd(&out[i], sh_bins[i]);
        __syncthreads();
    }
}

// New threshold of each segment of a missed worker: the lowest bin edge that still leaves
// `target` coordinates at or above it.  Clears the histogram, the worker's candidate counts and
// the select histogram its first attempt filled.
__device__ void stage_fb_guess(const Plan& P, const Active& act, uint32_t missed, uint32_t* sh, uint32_t* sh_best) {
    const uint32_t items = (uint32_t)P.nseg * act.n;
    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int r = act.r[item / P.nseg];
        if (!((missed >> r) & 1u)) continue;
        const uint32_t seg = item % P.nseg;
        uint32_t* hist = P.fb_hist + ((size_t)r * P.nseg + seg) * FB_BINS;
        uint32_t v[8], sum = 0;                  // thread t owns bins 2047 - 8t .. 2040 - 8t
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int bin = FB_BINS - 1 - 8 * (int)threadIdx.x - i;
            v[i] = hist[bin];
            hist[bin] = 0;
            sum += v[i];
        }
        P.hist[((size_t)r * P.nseg + seg) * 256 + threadIdx.x] = 0;
        if (threadIdx.x == 0) *sh_best = 0;
        uint32_t total;
        const uint32_t excl = block_excl_scan(sum, sh, &total);
        const uint32_t target = P.target[seg];
        if (excl < target && excl + sum >= target) {
            uint32_t run = excl;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                run += v[i];
                if (run >= target) { *sh_best = (uint32_t)(FB_BINS - 1 - 8 * (int)threadIdx.x - i); break; }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            // rounds of wider slack after a miss (predict_floor); the first round of a context has no
            // prediction to miss
            if (P.guess[(size_t)r * P.nseg + seg] != NO_GUESS) P.wary[(size_t)r * P.nseg + seg] = 16u;
            P.guess[(size_t)r * P.nseg + seg] = *sh_best << FB_SHIFT;
        }
        __syncthreads();
    }
    for (int w = 0; w < act.n; ++w) {
        const int r = act.r[w];
        if (!((missed >> r) & 1u)) continue;
        for (uint32_t i = blockIdx.x * BT + threadIdx.x; i < P.nblk; i += gridDim.x * BT) P.blk_count[(size_t)r * P.nblk + i] = 0;
        for (uint32_t i = blockIdx.x * BT + threadIdx.x; i < P.nsup; i += gridDim.x * BT) P.sup_count[(size_t)r * P.nsup + i] = 0;
    }
}

// candidates of the missed workers found again from the stored u with the new thresholds
template <bool RANDK>
__device__ void stage_reflag(const Plan& P, const Active& act, uint32_t missed, uint32_t* sh_cnt) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t item = 0;
    for (int w = 0; w < act.n; ++w) {
        const int r = act.r[w];
        if (!((missed >> r) & 1u)) continue;
        const size_t row = (size_t)r * P.d;
        const uint32_t* gs = P.guess + (size_t)r * P.nseg;
        for (uint32_t tile = blockIdx.x; tile < P.ntile; tile += gridDim.x, ++item) {
            uint32_t bal[GPW][4];
            float u[GPW][4];
#pragma unroll
            for (int k = 0; k < GPW; ++k) {
                const uint32_t e0 = (tile * (uint32_t)(STILE / GROUP) + warp * GPW + k) * (uint32_t)GROUP + (uint32_t)lane * 4u;
                uint4 h = make_uint4(0, 0, 0, 0);
                if (RANDK) h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
                const uint32_t hh[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool in = e0 + j < P.d;
                    u[k][j] = in ? P.mem[row + e0 + j] : 0.0f;
                    const uint32_t sk = RANDK ? ~hh[j] : topk_key(u[k][j]);
                    bal[k][j] = __ballot_sync(0xffffffffu, in && sk >= gs[segment_of(P, in ? e0 + j : 0u)]);
                }
            }
            uint32_t* cnt = sh_cnt + (item & 1u) * (8 * GPW);
            tile_counts(cnt, warp, lane, bal);
            __syncthreads();
            tile_write(P, r, tile, cnt, warp, lane, bal, u);
        }
    }
}

// ------------------------------------------------------------------ select
// unit owning a chunk: the last unit whose first chunk is not after it
__device__ __forceinline__ uint32_t unit_of_chunk(const Plan& P, const Tab& tab, uint32_t chunk) {
    uint32_t lo = 0, hi = P.U;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (tab.cb[mid] <= chunk) lo = mid; else hi = mid;
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

struct ChunkCtx { uint32_t u = 0xffffffffu, r, seg, first, c, cb, chunk; Unit un; size_t base; };   // chunk: its number among all chunks

// which unit a chunk belongs to (one search per block, shared through sh_u)
// `last`: the context of the block's previous chunk in this stage; a block's consecutive chunks
// mostly lie in one unit, whose record (unchanged within a stage) is then not read again.
__device__ __forceinline__ ChunkCtx chunk_context(const Plan& P, const Tab& tab, uint32_t chunk, uint32_t* sh_u,
                                                  const ChunkCtx* last = nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) *sh_u = unit_of_chunk(P, tab, chunk);
    __syncthreads();
    ChunkCtx c;
    c.u = *sh_u;
    if (last && last->u == c.u) c.un = last->un; else c.un = P.units[c.u];
    c.r = c.u / P.nseg;
    c.seg = c.u % P.nseg;
    c.c = tab.c[c.u];
    c.cb = tab.cb[c.u];
    c.first = (chunk - c.cb) * CHUNK;
    c.chunk = chunk;
    c.base = (size_t)c.r * P.cap + tab.start[c.u];
    return c;
}

// the same for chunk q of the long units only (the stages of the grid-wide select walk these)
__device__ __forceinline__ ChunkCtx long_chunk_context(const Plan& P, const Tab& tab, uint32_t q, uint32_t* sh_u,
                                                       const ChunkCtx* last = nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t lo = 0, hi = P.U;               // the last unit with lb <= q: short units before it share its lb
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (tab.lb[mid] <= q) lo = mid; else hi = mid;
        }
        *sh_u = lo;
    }
    __syncthreads();
    ChunkCtx c;
    c.u = *sh_u;
    if (last && last->u == c.u) c.un = last->un; else c.un = P.units[c.u];
    c.r = c.u / P.nseg;
    c.seg = c.u % P.nseg;
    c.c = tab.c[c.u];
    c.cb = tab.cb[c.u];
    c.first = (q - tab.lb[c.u]) * CHUNK;
    c.chunk = c.cb + (q - tab.lb[c.u]);
    c.base = (size_t)c.r * P.cap + tab.start[c.u];
    return c;
}

// one level of the radix select: histogram of the level's digit among keys matching the prefix.
// A block takes consecutive chunks; while they lie in one unit the prefix is worked out once and
// the counts stay in shared memory, to be added to the unit's histogram in one go.
template <bool RANDK>
__device__ void final_unit(const Plan& P, const Tab& tab, uint32_t u, uint32_t* sh4, uint32_t* sh_w);

// At the last level the block whose counts complete a unit (a count of finished chunks per unit)
// goes on to the unit's threshold, tie cut and prediction at once: no stage of its own for that.
template <bool RANDK>
__device__ void stage_hist(const Plan& P, const Tab& tab, int level, uint32_t* sh_hist, uint32_t* sh_u, uint32_t* sh_prefix,
                           uint32_t* sh4, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31;
    const uint32_t total = tab.total_long;
    const int shift = 24 - 8 * level;
    const uint32_t share = (total + gridDim.x - 1) / gridDim.x;
    const uint32_t c_lo = blockIdx.x * share, c_hi = c_lo + share < total ? c_lo + share : total;
    uint32_t held = 0xffffffffu, prefix = 0, nheld = 0;
    auto flush = [&]() {
        __syncthreads();                              // every add of the held chunks has been made
        const uint32_t v = sh_hist[threadIdx.x];
        if (v) atomicAdd(&P.hist[((size_t)level * P.U + held) * 256 + threadIdx.x], v);
        if (level == 3) {
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) {
                const uint32_t nch = tab.cb[held + 1] - tab.cb[held];
                const bool last = atomicAdd(&P.units[held].done, nheld) == nch - nheld;
                if (last) __threadfence();
                *sh_prefix = last ? 1u : 0u;
            }
            __syncthreads();
            if (*sh_prefix) final_unit<RANDK>(P, tab, held, sh4, sh_w);
            __syncthreads();
        }
        nheld = 0;
    };
    ChunkCtx c;
    for (uint32_t chunk = c_lo; chunk < c_hi; ++chunk) {
        c = long_chunk_context(P, tab, chunk, sh_u, &c);
        uint32_t sk[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            sk[i] = off < c.c ? sort_key<RANDK>(P, c.base + off) : 0u;
        }
        if (c.u != held) {
            if (held != 0xffffffffu) flush();
            held = c.u;
            if (threadIdx.x < 32) {
                uint32_t pf, at;
                derive_prefix(P, c.u, P.kseg[c.seg], level, lane, &pf, &at);
                if (lane == 0) *sh_prefix = pf;
            }
            sh_hist[threadIdx.x] = 0;
            __syncthreads();
            prefix = *sh_prefix;
        }
        ++nheld;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool valid = off < c.c && (level == 0 || (sk[i] >> (32 - 8 * level)) == prefix);
            if (valid) atomicAdd(&sh_hist[(sk[i] >> shift) & 255u], 1u);
        }
    }
    if (held != 0xffffffffu) flush();
}

// Prediction for the next round (Top_k): move the candidate floor so that about `target`
// coordinates pass it, assuming the tail keeps its shape (log-linear in the count).  One thread.
__device__ void predict_floor(const Plan& P, uint32_t r, uint32_t seg, uint32_t tau, uint32_t uc, uint32_t k) {
    uint32_t* gp = &P.guess[(size_t)r * P.nseg + seg];
    const uint32_t n = P.seg_off[seg + 1] - P.seg_off[seg];
    uint32_t want = P.target[seg];
    // A unit whose prediction missed lately aims for three times the usual slack for a while: a
    // workload whose scale jumps from round to round (workers that synchronise at uneven gaps)
    // then pays with longer lists instead of with exact passes.
    uint32_t* wary = &P.wary[(size_t)r * P.nseg + seg];
    if (*wary) {
        *wary -= 1u;
        const uint64_t wide = (uint64_t)k + 3ull * (want - k);
        want = wide < n ? (uint32_t)wide : n;
    }
    if (want >= n) { *gp = 0u; return; }          // every coordinate is a candidate (k = n, or nearly)
    const float tk = __uint_as_float(tau >> 1), tg = __uint_as_float(*gp >> 1);
    const float target = (float)want;
    float tn = tg;
    if (uc > k && tk > tg) {
        float ratio = __logf(target / (float)k) / __logf((float)uc / (float)k);
        ratio = fminf(fmaxf(ratio, 0.25f), 4.0f);
        tn = tk - (tk - tg) * ratio;
    } else if (uc <= k) {
        tn = tk * 0.75f;
    }
    tn = fminf(fmaxf(tn, tk * 0.25f), tk);
    *gp = __float_as_uint(tn) << 1;
}

// threshold key, tie cut and next prediction of one long unit, by the whole block, once every
// level of its select has been counted; clears its histograms
template <bool RANDK>
__device__ void final_unit(const Plan& P, const Tab& tab, uint32_t u, uint32_t* sh4, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    {
        const uint32_t uc = tab.c[u];
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
        uint32_t tie_max = 0xffffffffu, tie_t = 0;
        if (ceq > t && uc > 16u * BT) {
            // more equal keys than slots in a long list: the cut is found by all blocks together
            tie_t = t;
            if (threadIdx.x == 0) atomicOr(&P.fail[0], 1u);
        } else if (ceq > t) {
            // more equal keys than slots: the t lowest coordinates win; walk the list in order
            const size_t base = (size_t)r * P.cap + tab.start[u];
            for (uint32_t first = 0; first < uc; first += BT) {
                const uint32_t off = first + threadIdx.x;
                const bool eq = off < uc && sort_key<RANDK>(P, base + off) == tau;
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
            out.tie_t = tie_t;
            out.n = 0;
            out.emin = P.qz == QS_MINMAX ? 0xffffffffu : 255u;    // (min/max quantizer: ordered keys of the smallest and largest kept value)
            out.emax = 0u;
            out.norm = 0.0f;
            out.done = 0;
            if (!RANDK) predict_floor(P, r, seg, tau, uc, k);
        }
    }
}

// Tie cut of long lists, step 1: keys equal to the threshold in every chunk of a waiting unit
template <bool RANDK>
__device__ void stage_tie_count(const Plan& P, const Tab& tab, uint32_t* sh_u, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    ChunkCtx c;
    for (uint32_t chunk = blockIdx.x; chunk < tab.total_long; chunk += gridDim.x) {
        c = long_chunk_context(P, tab, chunk, sh_u, &c);
        if (c.un.tie_t == 0) continue;
        uint32_t cnt = 0;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            if (off < c.c && sort_key<RANDK>(P, c.base + off) == c.un.tau) ++cnt;
        }
        cnt = warp_sum(cnt);
        if (lane == 0) sh_w[wid] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t t = 0;
            for (int w = 0; w < BT / 32; ++w) t += sh_w[w];
            P.chunk_cnt[c.chunk] = t;
        }
    }
}

// step 2: the chunk that holds the last kept tie, then the coordinate itself
template <bool RANDK>
__device__ void stage_tie_find(const Plan& P, const Tab& tab, uint32_t* sh, uint32_t* sh4, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (uint32_t u = blockIdx.x; u < P.U; u += gridDim.x) {
        const Unit un = P.units[u];
        if (un.tie_t == 0) continue;
        const uint32_t c0 = tab.cb[u], c1 = tab.cb[u + 1], t = un.tie_t;
        __syncthreads();
        if (threadIdx.x == 0) { sh4[0] = 0xffffffffu; sh4[1] = 0; sh4[3] = 0xffffffffu; sh4[4] = 0; }
        __syncthreads();
        uint32_t carry = 0;
        for (uint32_t cb = c0; cb < c1; cb += BT) {
            const uint32_t i = cb + threadIdx.x;
            const uint32_t v = i < c1 ? P.chunk_cnt[i] : 0u;
            uint32_t total;
            const uint32_t ex = block_excl_scan(v, sh, &total);
            if (carry + ex < t && carry + ex + v >= t) { sh4[0] = i; sh4[1] = carry + ex; }
            carry += total;
            __syncthreads();
            if (sh4[0] != 0xffffffffu) break;
        }
        const uint32_t chunk = sh4[0], before_chunk = sh4[1];
        uint32_t tie_max = 0xffffffffu;
        if (chunk != 0xffffffffu) {
            const uint32_t uc = tab.c[u];
            const size_t base = (size_t)(u / P.nseg) * P.cap + tab.start[u];
            const uint32_t first0 = (chunk - c0) * CHUNK;
            if (threadIdx.x == 0) sh4[4] = before_chunk;
            __syncthreads();
            for (uint32_t first = first0; first < first0 + CHUNK; first += BT) {
                const uint32_t off = first + threadIdx.x;
                const bool eq = off < uc && sort_key<RANDK>(P, base + off) == un.tau;
                const uint32_t bal = __ballot_sync(0xffffffffu, eq);
                if (lane == 0) sh_w[wid] = __popc(bal);
                __syncthreads();
                uint32_t before = sh4[4];
                for (int w = 0; w < wid; ++w) before += sh_w[w];
                const uint32_t mine = before + __popc(bal & ((1u << lane) - 1u));
                if (eq && mine == t - 1) sh4[3] = P.cand_idx[base + off];
                __syncthreads();
                if (threadIdx.x == 0) { uint32_t s2 = 0; for (int w = 0; w < BT / 32; ++w) s2 += sh_w[w]; sh4[4] += s2; }
                __syncthreads();
                if (sh4[3] != 0xffffffffu) break;
            }
            tie_max = sh4[3];
        }
        if (threadIdx.x == 0) {
            if (tie_max == 0xffffffffu) set_status(P, QS_STATE);      // the counts said it is there
            P.units[u].tie_max = tie_max;
            P.units[u].tie_t = 0;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) P.fail[0] = 0;
}

// ------------------------------------------------------------------ quantize
// The closing stage will change the worker's memory at a kept coordinate while the memory system
// is busy with its copies: ask for the sector now, while it is idle, and to keep it in the L2.
__device__ __forceinline__ void mem_ahead(const Plan& P, uint32_t r, uint32_t idx) {
    asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(P.mem + (size_t)r * P.d + idx));
}

template <bool RANDK>
__device__ __forceinline__ bool is_kept(const Unit& un, uint32_t sk, uint32_t idx) {
    return sk > un.tau || (sk == un.tau && idx <= un.tie_max);
}

__device__ void unit_norm(const Plan& P, uint32_t u, uint32_t count, uint32_t (*sh)[4]);

// Exact per-exponent sums in 32-bit words of shared memory, one add per value and word (adds to
// shared memory are single instructions on 32 bits, and equal addresses within a warp cost nothing
// extra, so nothing is gathered per warp first): a value below 2^24 is added as its low 16 bits
// and the rest; with at most 2^15 additions per word neither can overflow.  acc[e] = {lo16,
// rest} of the first sum, {lo16, rest} of the second.
__device__ __forceinline__ void sums_add(uint32_t (*acc)[4], uint32_t e, uint32_t lo, uint32_t hi, bool two) {
    atomicAdd(&acc[e][0], lo & 0xffffu);
    atomicAdd(&acc[e][1], lo >> 16);
    if (two) {
        atomicAdd(&acc[e][2], hi & 0xffffu);
        atomicAdd(&acc[e][3], hi >> 16);
    }
}

// The norm from the exact sum held as an integer: tot1 x 2^(e_lo - 1 - 149) (magnitudes) or tot2 x
// 2^(2 (e_lo - 1) - 298) (squares).  One conversion rounds it to fp64, to nearest even.
__device__ __forceinline__ float norm_of_exact_sum(bool l1, unsigned long long tot1, unsigned __int128 tot2, int e_lo) {
    double sum;
    if (l1) {
        sum = ldexp(__ull2double_rn(tot1), e_lo - 1 - 149);
    } else {
        const unsigned long long hi = (unsigned long long)(tot2 >> 64), lo = (unsigned long long)tot2;
        if (hi == 0ull) {
            sum = ldexp(__ull2double_rn(lo), 2 * (e_lo - 1) - 298);
        } else {
            // the top 64 bits with everything below folded into the lowest one: the conversion then
            // rounds as if it had seen all the bits
            const int s = 64 - __clzll(hi);
            unsigned long long top = (unsigned long long)(tot2 >> s);
            if ((lo << (64 - s)) != 0ull) top |= 1ull;
            sum = ldexp(__ull2double_rn(top), s + 2 * (e_lo - 1) - 298);
        }
    }
    return l1 ? __double2float_rn(sum) : __double2float_rn(sqrt(sum));
}

// Norm from per-exponent sums that span at most 12 exponents, each sum below 2^44: the exact sum
// fits 64 (magnitudes) or 128 (squares) bits, and one conversion rounds it to fp64 (to nearest
// even).  Other cases take norm_of_sums; both give the correctly rounded exact sum.  The sums are
// read four exponents at a time, so their reads are in flight together.
template <class Load>
__device__ float norm_of_sums_near(uint32_t emin, uint32_t emax, bool l1, Load load) {
    const int e_lo = emin ? (int)emin : 1;                 // subnormals share the exponent of e = 1
    unsigned long long tot1 = 0ull;
    unsigned __int128 tot2 = 0;
    for (uint32_t eb = emin; eb <= emax; eb += 4) {
        unsigned long long a0[4], a1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            a0[j] = 0ull; a1[j] = 0ull;
            if (eb + j <= emax) load(eb + j, &a0[j], &a1[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t e = eb + j;
            const int sh = (e ? (int)e : 1) - e_lo;
            if (l1) tot1 += a0[j] << sh;
            else tot2 += ((unsigned __int128)a0[j] + ((unsigned __int128)a1[j] << 24)) << (2 * sh);
        }
    }
    return norm_of_exact_sum(l1, tot1, tot2, e_lo);
}


// Per-exponent integer sums of the kept values: for exponent e the squares' 48-bit mantissa
// products are summed as two 24-bit halves (QSGD), or the 24-bit mantissas themselves (Sign).
// A 64-bit sum cannot overflow below 2^32 terms.
template <bool RANDK>
__device__ void stage_norm_accum(const Plan& P, const Tab& tab, bool merge, uint32_t (*acc)[4], uint32_t* sh_u,
                                 uint32_t* sh_w, uint32_t* sh_e) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t total = tab.total_long;
    const bool plain = P.qz == QS_NONE;            // the plain sparsifier sends the values: no norm
    const bool mm = P.qz == QS_MINMAX;             // smallest and largest kept value in place of a norm
    // merge: a whole round with a quantizer that sends every kept entry at level 1; the counts and
    // the kept entries are known here; the packing warps and the closing stage do the rest of the quantize stage's work
    const bool early = merge;
    const bool l1 = P.qz == QS_SIGN_L1;
    // A block takes consecutive chunks.  While they lie in one unit their sums stay in shared memory
    // and go out together (at most 32 chunks: 2^15 additions of 16 bits per word): a long list then
    // costs a block one set of atomic adds on the unit's sums, one fence and one count of finished
    // chunks, not one per chunk.  Adds from many blocks to the same few 64-bit words of a unit are
    // what this stage used to wait for.
    constexpr uint32_t HOLD = 32;
    ChunkCtx c, held;
    uint32_t pending = 0;                          // chunks whose sums are held for unit held.u
    auto flush = [&]() {
        __syncthreads();                           // every add of the held chunks has been made
        const uint4 a = *reinterpret_cast<const uint4*>(acc[threadIdx.x]);
        *reinterpret_cast<uint4*>(acc[threadIdx.x]) = make_uint4(0u, 0u, 0u, 0u);
        const unsigned long long a0 = ((unsigned long long)a.y << 16) + a.x, a1 = ((unsigned long long)a.w << 16) + a.z;
        if (a0 | a1) {
            unsigned long long* g = P.eacc + ((size_t)held.u * 256 + threadIdx.x) * 2;
            if (a0) atomicAdd(g, a0);
            if (a1) atomicAdd(g + 1, a1);
        }
        // the exponent range of the unit: one update per flush, and only when it widens the range
        // seen on entry
        const uint32_t used = __ballot_sync(0xffffffffu, (a0 | a1) != 0ull);
        if (lane == 0) sh_e[wid] = used;
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t lo_e = 256u, hi_e = 0u;
            for (int w = 0; w < BT / 32; ++w)
                if (sh_e[w]) {
                    const uint32_t first = (uint32_t)w * 32u + (uint32_t)__ffs(sh_e[w]) - 1u, last = (uint32_t)w * 32u + 31u - (uint32_t)__clz(sh_e[w]);
                    lo_e = lo_e < first ? lo_e : first;
                    hi_e = hi_e > last ? hi_e : last;
                }
            if (lo_e < held.un.emin) atomicMin(&P.units[held.u].emin, lo_e);
            if (hi_e > held.un.emax) atomicMax(&P.units[held.u].emax, hi_e);
            __threadfence();
            // the flush that completes its unit turns the sums into the norm
            const uint32_t nch = tab.cb[held.u + 1] - held.cb;
            const bool last = atomicAdd(&P.units[held.u].done, pending) == nch - pending;
            if (last) __threadfence();
            sh_e[BT / 32] = last ? 1u : 0u;
        }
        __syncthreads();
        if (sh_e[BT / 32]) unit_norm(P, held.u, held.c, acc);
        pending = 0;
    };
    *reinterpret_cast<uint4*>(acc[threadIdx.x]) = make_uint4(0u, 0u, 0u, 0u);
    const uint32_t share = (total + gridDim.x - 1) / gridDim.x;
    const uint32_t c_lo = blockIdx.x * share, c_hi = c_lo + share < total ? c_lo + share : total;
    for (uint32_t chunk = c_lo; chunk < c_hi; ++chunk) {
        c = long_chunk_context(P, tab, chunk, sh_u, &c);       // (its barriers order the zeroing above)
        if (pending && (c.u != held.u || pending == HOLD)) flush();
        held = c;
        float val[PER];
        uint32_t idx[PER], key[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool in = off < c.c;
            val[i] = in ? P.cand_val[c.base + off] : 0.0f;
            idx[i] = in ? P.cand_idx[c.base + off] : 0xffffffffu;
            key[i] = RANDK ? (in ? P.cand_key[c.base + off] : 0u) : topk_key(val[i]);
        }
        uint32_t nkept = 0;                          // lane 0 of each warp counts
        uint32_t mm_lo = 0xffffffffu, mm_hi = 0u;
        bool kept[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            kept[i] = off < c.c && is_kept<RANDK>(c.un, key[i], idx[i]);
            if (early && kept[i]) mem_ahead(P, c.r, idx[i]);
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t live = __ballot_sync(0xffffffffu, kept[i]);
            if (early && lane == 0) nkept += __popc(live);
            if (kept[i] && mm) {
                const uint32_t ok = float_order(val[i]);
                mm_lo = ok < mm_lo ? ok : mm_lo;
                mm_hi = ok > mm_hi ? ok : mm_hi;
            } else if (kept[i] && !plain) {
                const uint32_t b = __float_as_uint(val[i]);
                const uint32_t e = (b >> 23) & 255u;
                const uint32_t m = e ? ((b & 0x7fffffu) | 0x800000u) : (b & 0x7fffffu);
                uint32_t lo, hi;
                if (l1) { lo = m; hi = 0; }
                else { const unsigned long long sq = (unsigned long long)m * m; lo = (uint32_t)(sq & 0xffffffu); hi = (uint32_t)(sq >> 24); }
                sums_add(acc, e, lo, hi, !l1);
            }
        }
        if (early) {
            if (lane == 0) sh_w[wid] = nkept;
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t t = 0;
                for (int w = 0; w < BT / 32; ++w) t += sh_w[w];
                P.chunk_cnt[c.chunk] = t | (t << 16);    // kept | sent << 16
            }
        }
        if (mm) {
            mm_lo = __reduce_min_sync(0xffffffffu, mm_lo);
            mm_hi = __reduce_max_sync(0xffffffffu, mm_hi);
            if (lane == 0 && mm_lo <= mm_hi) { atomicMin(&P.units[c.u].emin, mm_lo); atomicMax(&P.units[c.u].emax, mm_hi); }
        } else if (!plain) {
            ++pending;
        }
    }
    if (pending) flush();
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

// A 768-bit integer (little-endian base 2^32; bit 0 stands for 2^-298 with squares, 2^-149 with
// magnitudes) -> fp64 (round to nearest even) -> norm in fp32.  One thread.
constexpr int NORM_DIGITS = 24;
__device__ float norm_of_digits(const uint32_t* dig, bool l1) {
    constexpr int ND = NORM_DIGITS;
    int tw = ND - 1;
    while (tw >= 0 && dig[tw] == 0) --tw;
    double sum = 0.0;
    if (tw >= 0) {
        const int top = tw * 32 + 31 - __clz(dig[tw]);
        // the 64 bits that start at the top bit (zeros below bit 0), then the 53-bit mantissa
        const int sh = 31 - (top & 31);                       // left shift that puts the top bit at bit 31
        const uint32_t w0 = dig[tw], w1 = tw >= 1 ? dig[tw - 1] : 0u, w2 = tw >= 2 ? dig[tw - 2] : 0u;
        const unsigned long long hi64 = ((unsigned long long)w0 << 32) | w1;
        const unsigned long long bits = sh ? ((hi64 << sh) | ((unsigned long long)w2 >> (32 - sh))) : hi64;
        unsigned long long mant = bits >> 11;
        const uint32_t guard = (uint32_t)(bits >> 10) & 1u;
        uint32_t sticky = (bits & 0x3ffull) != 0;
        if (sh && (w2 << sh)) sticky = 1;                     // bits of the third word not shifted in
        if (!sh && w2) sticky = 1;
        for (int j = tw - 3; j >= 0 && !sticky; --j) sticky = dig[j] != 0;
        if (guard && (sticky || (mant & 1ull))) mant += 1ull;
        sum = ldexp((double)mant, top - 52 - (l1 ? 149 : 298));
    }
    return l1 ? __double2float_rn(sum) : __double2float_rn(sqrt(sum));
}

// Exact sum of the per-exponent integer sums (exponents emin .. emax, read through `load`) ->
// norm.  One thread.
template <class Load>
__device__ float norm_of_sums(uint32_t emin, uint32_t emax, bool l1, Load load) {
    constexpr int ND = NORM_DIGITS;
    uint32_t dig[ND];
    for (int j = 0; j < ND; ++j) dig[j] = 0;
    for (uint32_t e = emin; e <= emax; ++e) {
        unsigned long long a0, a1;
        load(e, &a0, &a1);
        if (!(a0 | a1)) continue;
        const int ee = e ? (int)e : 1;          // subnormals share the exponent of e = 1
        if (l1) {
            big_add(dig, ND, a0, ee - 1);
        } else {
            big_add(dig, ND, a0, 2 * (ee - 1));
            big_add(dig, ND, a1, 2 * (ee - 1) + 24);
        }
    }
    return norm_of_digits(dig, l1);
}

// The whole block, once per unit (of `count` candidates), after every chunk has added its sums.
// The sums were built with atomics in the L2: every thread fetches those of one exponent from
// there (one round trip for all of them, where one thread reading them in turn took one each),
// leaves them zero and parks them in shared memory (sh: 256 x 16 bytes, zero on entry and on
// return); one thread then adds them up exactly.
__device__ void unit_norm(const Plan& P, uint32_t u, uint32_t count, uint32_t (*sh)[4]) {
    Unit& un = P.units[u];
    const uint32_t emin = __ldcg(&un.emin), emax = __ldcg(&un.emax);
    if (emin <= emax) {                                    // (the same in every thread)
        const uint32_t e = threadIdx.x;
        const bool mine = e >= emin && e <= emax;
        if (mine) {
            unsigned long long* g = P.eacc + ((size_t)u * 256 + e) * 2;
            const unsigned long long a0 = __ldcg(g), a1 = __ldcg(g + 1);
            g[0] = 0ull;
            g[1] = 0ull;
            *reinterpret_cast<ulonglong2*>(sh[e]) = make_ulonglong2(a0, a1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const bool l1 = P.qz == QS_SIGN_L1;
            auto sums = [&](uint32_t ee, unsigned long long* a0, unsigned long long* a1) {
                const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(sh[ee]);
                *a0 = v.x;
                *a1 = v.y;
            };
            // up to 2^20 values of 24 bits per sum: below 2^44
            un.norm = (emax - emin <= 12u && count <= (1u << 20)) ? norm_of_sums_near(emin, emax, l1, sums)
                                                                   : norm_of_sums(emin, emax, l1, sums);
        }
        __syncthreads();
        if (mine) *reinterpret_cast<uint4*>(sh[e]) = make_uint4(0u, 0u, 0u, 0u);
    }
    if (threadIdx.x == 0) un.done = 0;
}

// ------------------------------------------------------------------ short units: one block does it all
// A unit with a short candidate list is handled by ONE block from threshold to norm with block
// barriers only, in the shadow of the first grid-wide stage of the long units' select: every list
// of at most 256 candidates, and every list (up to UNIT_CAP) of a round that has a block per unit.
// The block keeps the unit's sort keys in registers (UPT per thread).  Up to 256 candidates the
// kept set comes from ranks counted directly (key descending, list position ascending: the list
// is in index order); above that from a four-level radix select over a histogram in shared
// memory.  Then the tie cut, the next prediction, the exact norm (per-exponent sums in shared
// memory) and, for the quantizers that send every kept entry at level 1, the kept counts
// per chunk.  Units are handed out by a ticket counter, largest first.
constexpr int UPT = UNIT_CAP / BT;
static_assert(UNIT_CAP % CHUNK == 0 && UNIT_CAP / CHUNK <= 16, "kept counts per chunk: sixteen slots");

struct UnitSh {                      // lives in the 8 KB scratch of the persistent kernel
    uint32_t acc[256][4];            // per-exponent sums (sums_add)
    uint32_t hist[256];
    uint32_t keys[256];              // rank path: the candidates' keys
    uint32_t ctl[8];                 // 0 ticket, 1 prefix, 2 rank wanted, 3 keys equal to tau, 4 tie_max, 5 running ties
    uint32_t kept[16];               // kept entries per chunk
};

// Calls f(row, position in the list, key, index, value bits) for the rows of BT consecutive
// candidates of a unit, in order, every thread of the block taking part in every row (f may vote
// and meet at barriers).  The reads of NB rows are issued together, so a pass costs a round trip
// to the L2 per NB rows and not per row; for the same reason what f returns (say the old value
// of an atomic it started) is handed to g only after f has run for all NB rows.  AUX: the index
// (and for Rand_k the value) is read; without it f gets zeros.
template <bool RANDK, int NB, bool AUX, class F, class G>
__device__ __forceinline__ void unit_rows(const Plan& P, size_t base, uint32_t c, const uint32_t (&key)[UPT], F f, G g) {
    static_assert(UPT % NB == 0, "whole batches of rows");
#pragma unroll
    for (int b = 0; b < UPT / NB; ++b) {
        if ((uint32_t)(b * NB * BT) < c) {
            uint32_t ix[NB], vq[NB], tok[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const uint32_t off = (uint32_t)((b * NB + j) * BT) + threadIdx.x;
                ix[j] = (AUX && off < c) ? P.cand_idx[base + off] : 0u;
                vq[j] = (AUX && (RANDK || P.qz == QS_MINMAX) && off < c) ? __float_as_uint(P.cand_val[base + off]) : 0u;
            }
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                tok[j] = 0u;
                if ((uint32_t)((b * NB + j) * BT) < c)
                    tok[j] = f((uint32_t)(b * NB + j), (uint32_t)((b * NB + j) * BT) + threadIdx.x, key[b * NB + j], ix[j], vq[j]);
            }
#pragma unroll
            for (int j = 0; j < NB; ++j)
                if ((uint32_t)((b * NB + j) * BT) < c) g(ix[j], tok[j]);
        }
    }
}

// The shortest lists (at most 64 candidates: two per lane) need no block: a warp takes such a
// unit through the same steps with shuffles only, eight units at a time per block.  Ranks by
// direct counting; the exact norm as one integer sum over the warp when the kept values' exponents
// lie within 12 of each other, otherwise value by value into the long accumulator by one lane.
constexpr uint32_t WARP_C = 64;

__device__ __forceinline__ unsigned long long warp_sum64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <bool RANDK>
__device__ void unit_by_warp(const Plan& P, const Tab& tab, uint32_t u, uint32_t r, uint32_t seg, bool early, int lane) {
    const uint32_t c = tab.c[u], k = P.kseg[seg];
    const size_t base = (size_t)r * P.cap + tab.start[u];
    const bool mm = P.qz == QS_MINMAX;
    const bool plain = P.qz == QS_NONE || mm, l1 = P.qz == QS_SIGN_L1;   // (no norm for the plain sparsifier and the min/max quantizer)
    uint32_t key[2], idx[2], vb[2];
    bool in[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint32_t j = (uint32_t)lane + 32u * q;
        in[q] = j < c;
        key[q] = in[q] ? sort_key<RANDK>(P, base + j) : 0u;
        idx[q] = in[q] ? P.cand_idx[base + j] : 0u;
        vb[q] = ((RANDK || mm) && in[q]) ? __float_as_uint(P.cand_val[base + j]) : (key[q] >> 1);
    }
    // rank of each candidate: those before it have a larger key, or an equal one earlier in the list
    uint32_t rank[2] = {0u, 0u};
    for (uint32_t j = 0; j < c; ++j) {
        const uint32_t kj = __shfl_sync(0xffffffffu, j < 32u ? key[0] : key[1], (int)(j & 31u));
        rank[0] += (kj > key[0] || (kj == key[0] && j < (uint32_t)lane)) ? 1u : 0u;
        rank[1] += (kj > key[1] || (kj == key[1] && j < (uint32_t)lane + 32u)) ? 1u : 0u;
    }
    bool kept[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) kept[q] = in[q] && rank[q] < k;
    // exponent range of the kept values
    uint32_t e[2], m[2];
    int lo_e = 255, hi_e = 0;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        e[q] = (vb[q] >> 23) & 255u;
        m[q] = e[q] ? ((vb[q] & 0x7fffffu) | 0x800000u) : (vb[q] & 0x7fffffu);
        if (kept[q] && m[q]) {
            const int ee = e[q] ? (int)e[q] : 1;
            lo_e = ee < lo_e ? ee : lo_e;
            hi_e = ee > hi_e ? ee : hi_e;
        }
    }
    lo_e = __reduce_min_sync(0xffffffffu, lo_e);
    hi_e = __reduce_max_sync(0xffffffffu, hi_e);
    float norm = 0.0f;
    if (!plain && hi_e >= lo_e && hi_e - lo_e > 12) {                      // (the same in every lane)
        uint32_t dig[NORM_DIGITS];
        for (int j = 0; j < NORM_DIGITS; ++j) dig[j] = 0;
        for (uint32_t j = 0; j < c; ++j) {
            const bool second = j >= 32u;
            const uint32_t kj = __shfl_sync(0xffffffffu, (second ? kept[1] : kept[0]) ? 1u : 0u, (int)(j & 31u));
            const uint32_t ej = __shfl_sync(0xffffffffu, second ? e[1] : e[0], (int)(j & 31u));
            const uint32_t mj = __shfl_sync(0xffffffffu, second ? m[1] : m[0], (int)(j & 31u));
            if (lane == 0 && kj && mj) {
                const int ee = ej ? (int)ej : 1;
                if (l1) big_add(dig, NORM_DIGITS, mj, ee - 1);
                else big_add(dig, NORM_DIGITS, (unsigned long long)mj * mj, 2 * (ee - 1));
            }
        }
        norm = __shfl_sync(0xffffffffu, lane == 0 ? norm_of_digits(dig, l1) : 0.0f, 0);
    } else if (!plain && hi_e >= lo_e) {
        // at most 64 terms of 24 (magnitudes) or 48 (squares) bits shifted by at most 12 (24)
        unsigned long long p1 = 0ull, p2lo = 0ull, p2hi = 0ull;
#pragma unroll
        for (int q = 0; q < 2; ++q)
            if (kept[q] && m[q]) {
                const int sh = (e[q] ? (int)e[q] : 1) - lo_e;
                if (l1) {
                    p1 += (unsigned long long)m[q] << sh;
                } else {
                    const unsigned __int128 t = (unsigned __int128)((unsigned long long)m[q] * m[q]) << (2 * sh);
                    p2lo += (unsigned long long)t & 0xffffffffffull;        // low 40 bits
                    p2hi += (unsigned long long)(t >> 40);
                }
            }
        p1 = warp_sum64(p1);
        p2lo = warp_sum64(p2lo);
        p2hi = warp_sum64(p2hi);
        norm = norm_of_exact_sum(l1, p1, ((unsigned __int128)p2hi << 40) + p2lo, lo_e);
    }
    // threshold: the candidate of rank k - 1
    const uint32_t hit0 = __ballot_sync(0xffffffffu, in[0] && rank[0] == k - 1u);
    const uint32_t hit1 = __ballot_sync(0xffffffffu, in[1] && rank[1] == k - 1u);
    const int src = hit0 ? __ffs(hit0) - 1 : __ffs(hit1) - 1;
    const uint32_t tau = __shfl_sync(0xffffffffu, hit0 ? key[0] : key[1], src);
    const uint32_t tie_max = __shfl_sync(0xffffffffu, hit0 ? idx[0] : idx[1], src);
    if (early) {
#pragma unroll
        for (int q = 0; q < 2; ++q)
            if (kept[q]) mem_ahead(P, r, idx[q]);
        const uint32_t n = __popc(__ballot_sync(0xffffffffu, kept[0])) + __popc(__ballot_sync(0xffffffffu, kept[1]));
        if (lane == 0) P.chunk_cnt[tab.cb[u]] = n | (n << 16);             // a list this short is one chunk
    }
    // the level-0 counts of the order stage are not needed on this path: leave them zero
#pragma unroll
    for (int i = 0; i < 8; ++i) P.hist[(size_t)u * 256 + (uint32_t)lane + 32u * i] = 0u;
    // min/max quantizer: ordered keys of the smallest and largest kept value
    uint32_t mm_lo = 0xffffffffu, mm_hi = 0u;
    if (mm) {
#pragma unroll
        for (int q = 0; q < 2; ++q)
            if (kept[q]) {
                const uint32_t ok = float_order(__uint_as_float(vb[q]));
                mm_lo = ok < mm_lo ? ok : mm_lo;
                mm_hi = ok > mm_hi ? ok : mm_hi;
            }
        mm_lo = __reduce_min_sync(0xffffffffu, mm_lo);
        mm_hi = __reduce_max_sync(0xffffffffu, mm_hi);
    }
    if (lane == 0) {
        Unit& out = P.units[u];
        out.tau = tau;
        out.tie_max = tie_max;
        out.tie_t = 0;
        out.n = 0;
        out.emin = mm ? mm_lo : 255u;
        out.emax = mm ? mm_hi : 0u;
        out.norm = norm;
        if (!RANDK) predict_floor(P, r, seg, tau, c, k);
    }
}

template <bool RANDK>
__device__ void stage_unit(const Plan& P, const Tab& tab, const Active& act, bool early, UnitSh& S, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t items = (uint32_t)P.nseg * (uint32_t)act.n;
    const bool mm = P.qz == QS_MINMAX;
    const bool plain = P.qz == QS_NONE || mm, l1 = P.qz == QS_SIGN_L1;   // (no norm for the plain sparsifier and the min/max quantizer)
    const uint32_t lt = (1u << lane) - 1u;
    // the shortest lists first, a warp each: eight consecutive units of the list to a block
    for (uint32_t item = blockIdx.x * (BT / 32) + wid; item < items; item += gridDim.x * (BT / 32)) {
        const uint32_t seg = P.seg_order[item / (uint32_t)act.n];
        const uint32_t r = (uint32_t)act.r[item % (uint32_t)act.n];
        const uint32_t u = r * (uint32_t)P.nseg + seg;
        const uint32_t c = tab.c[u];
        if (c && c <= WARP_C && c <= tab.short_c) unit_by_warp<RANDK>(P, tab, u, r, seg, early, lane);
    }
    if (threadIdx.x == 0) S.ctl[0] = atomicAdd(P.bar + 4, 1u);
    __syncthreads();
    for (;;) {
        const uint32_t item = S.ctl[0];
        __syncthreads();                                   // everyone has read the ticket
        if (item >= items) break;
        if (threadIdx.x == 0) S.ctl[0] = atomicAdd(P.bar + 4, 1u);     // the next one: its round trip is off the path
        const uint32_t seg = P.seg_order[item / (uint32_t)act.n];
        const uint32_t r = (uint32_t)act.r[item % (uint32_t)act.n];
        const uint32_t u = r * (uint32_t)P.nseg + seg;
        const uint32_t c = tab.c[u], k = P.kseg[seg];
        // an idle worker's, a long unit, or one that a warp has done
        if (c == 0 || c > tab.short_c || c <= WARP_C) { __syncthreads(); continue; }
        const size_t base = (size_t)r * P.cap + tab.start[u];
        uint32_t key[UPT];
#pragma unroll
        for (int i = 0; i < UPT; ++i) {
            const uint32_t off = i * BT + threadIdx.x;
            key[i] = off < c ? sort_key<RANDK>(P, base + off) : 0u;
        }
        *reinterpret_cast<uint4*>(S.acc[threadIdx.x]) = make_uint4(0u, 0u, 0u, 0u);
        if (threadIdx.x < 16) S.kept[threadIdx.x] = 0u;
        if (threadIdx.x == 0) { S.ctl[4] = 0xffffffffu; S.ctl[5] = 0u; S.ctl[6] = 0xffffffffu; S.ctl[7] = 0u; }   // (6, 7: smallest / largest kept value)
        uint32_t tau, tie_max;
        if (c <= (uint32_t)BT) {
            // ranks by direct counting: candidate j comes before this one if its key is larger, or
            // equal and earlier in the list
            const uint32_t my_idx = threadIdx.x < c ? P.cand_idx[base + threadIdx.x] : 0u;
            S.keys[threadIdx.x] = key[0];
            __syncthreads();
            uint32_t rank = 0;
            for (uint32_t j = 0; j < c; ++j) {
                const uint32_t kj = S.keys[j];
                rank += (kj > key[0] || (kj == key[0] && j < threadIdx.x)) ? 1u : 0u;
            }
            if (threadIdx.x < c && rank == k - 1u) { S.ctl[1] = key[0]; S.ctl[4] = my_idx; }
            __syncthreads();
            tau = S.ctl[1];
            tie_max = S.ctl[4];
        } else {
            // level 0 (the top key byte) was counted per unit by the order stage
            if (wid == 0) {
                uint32_t bin, above;
                find_bin(P.hist + (size_t)u * 256, k, lane, &bin, &above);
                if (lane == 0) { S.ctl[1] = bin; S.ctl[2] = k - above; S.ctl[3] = P.hist[(size_t)u * 256 + bin]; }
            }
            for (int level = 1; level < 4; ++level) {
                const int shift = 24 - 8 * level;
                S.hist[threadIdx.x] = 0u;
                __syncthreads();
                const uint32_t prefix = S.ctl[1];
                unit_rows<RANDK, 8, false>(P, base, c, key, [&](uint32_t, uint32_t off, uint32_t kv, uint32_t, uint32_t) {
                    const bool valid = off < c && (level == 0 || (kv >> (32 - 8 * level)) == prefix);
                    if (valid) atomicAdd(&S.hist[(kv >> shift) & 255u], 1u);
                    return 0u;
                }, [](uint32_t, uint32_t) {});
                __syncthreads();
                if (wid == 0) {
                    uint32_t bin, above;
                    find_bin(S.hist, S.ctl[2], lane, &bin, &above);
                    if (lane == 0) {
                        S.ctl[1] = (prefix << 8) | bin;
                        S.ctl[2] -= above;
                        S.ctl[3] = S.hist[bin];
                    }
                }
                __syncthreads();
            }
            tau = S.ctl[1];
            const uint32_t t = S.ctl[2], ceq = S.ctl[3];
            if (ceq > t) {
                // more equal keys than slots: the t earliest in the list win
                unit_rows<RANDK, 8, true>(P, base, c, key, [&](uint32_t, uint32_t off, uint32_t kv, uint32_t idx, uint32_t) {
                    const bool eq = off < c && kv == tau;
                    const uint32_t bal = __ballot_sync(0xffffffffu, eq);
                    if (lane == 0) sh_w[wid] = __popc(bal);
                    __syncthreads();
                    uint32_t before = S.ctl[5], row = 0;
                    for (int w = 0; w < BT / 32; ++w) { if (w < wid) before += sh_w[w]; row += sh_w[w]; }
                    const uint32_t mine = before + __popc(bal & lt);
                    if (eq && mine == t - 1u) S.ctl[4] = idx;
                    __syncthreads();
                    if (threadIdx.x == 0) S.ctl[5] += row;
                    return 0u;
                }, [](uint32_t, uint32_t) {});
                if (S.ctl[4] == 0xffffffffu) set_status(P, QS_STATE);     // the counts said it is there
            }
            tie_max = S.ctl[4];
        }
        // the level-0 counts of the order stage are not needed on this path: leave them zero
        P.hist[(size_t)u * 256 + threadIdx.x] = 0u;
        // kept entries: exact sums per exponent (or smallest / largest value) and kept counts per chunk
        const bool ties = tie_max != 0xffffffffu;
        auto take = [&](uint32_t i, uint32_t off, uint32_t kv, uint32_t idx, uint32_t vb) {
            const bool kept = off < c && kv >= tau && !(ties && kv == tau && idx > tie_max);
            const uint32_t live = __ballot_sync(0xffffffffu, kept);
            if (early && lane == 0 && live) atomicAdd(&S.kept[i / PER], __popc(live));
            if (early && kept) mem_ahead(P, r, idx);
            if (mm) {                                // ordered keys of the smallest and largest kept value
                const uint32_t ok = float_order(__uint_as_float(vb));
                const uint32_t w_lo = __reduce_min_sync(0xffffffffu, kept ? ok : 0xffffffffu);
                const uint32_t w_hi = __reduce_max_sync(0xffffffffu, kept ? ok : 0u);
                if (lane == 0 && live) { atomicMin(&S.ctl[6], w_lo); atomicMax(&S.ctl[7], w_hi); }
            }
            if (kept && !plain) {
                const uint32_t b = RANDK ? vb : (kv >> 1);
                const uint32_t e = (b >> 23) & 255u;
                const uint32_t m = e ? ((b & 0x7fffffu) | 0x800000u) : (b & 0x7fffffu);
                uint32_t lo, hi;
                if (l1) { lo = m; hi = 0; }
                else { const unsigned long long sq = (unsigned long long)m * m; lo = (uint32_t)(sq & 0xffffffu); hi = (uint32_t)(sq >> 24); }
                sums_add(S.acc, e, lo, hi, !l1);
            }
            return 0u;
        };
        auto none = [](uint32_t, uint32_t) {};
        // the indices are needed for a tie cut and for the request above; Rand_k and the min/max
        // quantizer read the values too
        if (early || ties || RANDK || mm) unit_rows<RANDK, 8, true>(P, base, c, key, take, none);
        else unit_rows<RANDK, 8, false>(P, base, c, key, take, none);
        __syncthreads();
        if (wid == 0) {
            // exponent range of the sums
            uint32_t lo_e = 256u, hi_e = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t e = (uint32_t)lane * 8u + j;
                const uint4 a = *reinterpret_cast<const uint4*>(S.acc[e]);
                if (a.x | a.y | a.z | a.w) { lo_e = lo_e < e ? lo_e : e; hi_e = e; }
            }
            lo_e = __reduce_min_sync(0xffffffffu, lo_e);
            hi_e = __reduce_max_sync(0xffffffffu, hi_e);
            if (lane == 0) {
                Unit& out = P.units[u];
                out.tau = tau;
                out.tie_max = tie_max;
                out.tie_t = 0;
                out.n = 0;
                out.emin = mm ? S.ctl[6] : 255u;
                out.emax = mm ? S.ctl[7] : 0u;
                auto sums = [&](uint32_t e, unsigned long long* a0, unsigned long long* a1) {
                    *a0 = ((unsigned long long)S.acc[e][1] << 16) + S.acc[e][0];
                    *a1 = ((unsigned long long)S.acc[e][3] << 16) + S.acc[e][2];
                };
                out.norm = (plain || lo_e > hi_e) ? 0.0f
                         : hi_e - lo_e <= 12u ? norm_of_sums_near(lo_e, hi_e, l1, sums) : norm_of_sums(lo_e, hi_e, l1, sums);
                if (!RANDK) predict_floor(P, r, seg, tau, c, k);
                if (early) {
                    const uint32_t c0 = tab.cb[u], nch = tab.cb[u + 1] - c0;
                    for (uint32_t j = 0; j < nch; ++j) P.chunk_cnt[c0 + j] = S.kept[j] | (S.kept[j] << 16);
                }
            }
        }
        __syncthreads();
    }
}

// levels, signs, memory update; kept and sent counts per chunk
template <bool RANDK>
__device__ void stage_quant(const Plan& P, const Tab& tab, uint32_t* sh_u, uint32_t* sh_w) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t total = tab.total_chunks;
    const bool sign_op = qz_is_sign(P.qz), plain = P.qz == QS_NONE, mm = P.qz == QS_MINMAX;
    ChunkCtx c;
    const uint32_t share = (total + gridDim.x - 1) / gridDim.x;      // consecutive chunks: mostly one unit
    const uint32_t c_lo = blockIdx.x * share, c_hi = c_lo + share < total ? c_lo + share : total;
    for (uint32_t chunk = c_lo; chunk < c_hi; ++chunk) {
        c = chunk_context(P, tab, chunk, sh_u, &c);
        const float N = c.un.norm, cs = P.cscale[c.seg];
        const uint32_t k = P.kseg[c.seg];
        float* mem = P.mem + (size_t)c.r * P.d;
        float val[PER];
        uint32_t idx[PER], key[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            const bool in = off < c.c;
            val[i] = in ? P.cand_val[c.base + off] : 0.0f;
            idx[i] = in ? P.cand_idx[c.base + off] : 0xffffffffu;
            key[i] = RANDK ? (in ? P.cand_key[c.base + off] : 0u) : topk_key(val[i]);
        }
        uint32_t cnt = 0;                            // kept | sent << 16
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const uint32_t off = c.first + i * BT + threadIdx.x;
            if (off >= c.c) continue;
            uint32_t q = 0;
            if (is_kept<RANDK>(c.un, key[i], idx[i])) {
                const bool neg = !mm && val[i] < 0.0f;       // (the min/max quantizer has no sign stream)
                int level = 1;
                float g;
                if (mm) {
                    const float lo = order_float(c.un.emin), hi = order_float(c.un.emax);
                    level = minmax_level(val[i], lo, hi, P.s, philox_word(P, c.r, idx[i], 0u));
                    g = minmax_value(lo, hi, P.s, level);
                } else {
                    if (!sign_op && !plain) level = qsgd_level(val[i], N, P.s, philox_word(P, c.r, idx[i], 0u));
                    g = plain ? val[i] : coord_value(P, N, level, neg, cs, k);
                }
                q = Q_SEL | (neg ? Q_NEG : 0u) | (uint32_t)level;
                cnt += 1u;
                if (level) {
                    mem[idx[i]] = val[i] - g;
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
__device__ void stage_chunk_scan(const Plan& P, const Tab& tab, const Active& act, uint32_t* sh) {
    if (blockIdx.x != 0) return;
    const uint32_t total = tab.total_chunks;
    uint32_t carry_k = 0, carry_s = 0;
    constexpr uint32_t SC = 16;                   // consecutive chunks per thread and step
    for (uint32_t base = 0; base <= total; base += BT * SC) {
        const uint32_t i0 = base + threadIdx.x * SC;
        uint32_t v[SC], sk = 0, ss = 0;
#pragma unroll
        for (uint32_t j = 0; j < SC; ++j) {
            v[j] = i0 + j < total ? P.chunk_cnt[i0 + j] : 0u;
            sk += v[j] & 0xffffu;
            ss += v[j] >> 16;
        }
        uint32_t tk, ts;
        uint32_t rk = carry_k + block_excl_scan(sk, sh, &tk);
        uint32_t rs = carry_s + block_excl_scan(ss, sh, &ts);
#pragma unroll
        for (uint32_t j = 0; j < SC; ++j) {
            if (i0 + j <= total) { P.chunk_sel[i0 + j] = rk; P.chunk_nz[i0 + j] = rs; }
            rk += v[j] & 0xffffu;
            rs += v[j] >> 16;
        }
        carry_k += tk; carry_s += ts;
    }
    __syncthreads();
    for (uint32_t u = threadIdx.x; u < P.U; u += BT) {
        Unit& un = P.units[u];
        if (!((act.bits >> (u / P.nseg)) & 1u)) continue;
        const uint32_t c0 = tab.cb[u], c1 = tab.cb[u + 1];
        const uint32_t kept = P.chunk_sel[c1] - P.chunk_sel[c0];
        un.n = P.chunk_nz[c1] - P.chunk_nz[c0];
        if (kept != P.kseg[u % P.nseg]) set_status(P, QS_STATE);
    }
    __syncthreads();
    for (int w = 0; w < act.n; ++w) {
        const int r = act.r[w];
        uint32_t carry = 2u * P.nseg;
        long long bits = 0;
        for (uint32_t gb = 0; gb < (uint32_t)P.nseg; gb += BT) {
            const uint32_t g = gb + threadIdx.x;
            uint32_t words = 0, n = 0, bi = 0;
            if (g < (uint32_t)P.nseg) {
                n = P.units[(size_t)r * P.nseg + g].n;
                bi = P.bidx[g];
                words = streams_words(n, bi, (uint32_t)P.bl, P.qz);
                bits += 64 + (long long)n * entry_bits(bi, (uint32_t)P.bl, P.qz);
            }
            uint32_t total;
            const uint32_t ex = block_excl_scan(words, sh, &total);
            if (g < (uint32_t)P.nseg) P.pay_off[(size_t)r * P.nseg + g] = carry + ex;
            carry += total;
        }
        // sum of the per-thread bit counts
        for (int o = 16; o; o >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, o);
        __shared__ long long sh_bits[BT / 32];
        __syncthreads();
        if ((threadIdx.x & 31) == 0) sh_bits[threadIdx.x >> 5] = bits;
        __syncthreads();
        if (threadIdx.x == 0) {
            long long t = 0;
            for (int i = 0; i < BT / 32; ++i) t += sh_bits[i];
            P.bits[r] = t;
        }
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
        const bool mm = P.qz == QS_MINMAX;           // (the pair carries (min, max), n = k)
        row[2 * g] = mm ? __float_as_uint(order_float(un.emin)) : un.n;
        row[2 * g + 1] = __float_as_uint(mm ? order_float(un.emax) : un.norm);
        if (g == 0 && bits_out) bits_out[r] = P.bits[r];
    }
}

// four sums over the block at once; every thread gets all four.  sh: 4 x (BT / 32) words
__device__ __forceinline__ void block_sum4(uint32_t v[4], uint32_t* sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    __syncthreads();                              // sh may still be read from a previous call
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t w = __reduce_add_sync(0xffffffffu, v[j]);
        if (lane == 0) sh[j * (BT / 32) + wid] = w;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t t = 0;
#pragma unroll
        for (int w = 0; w < BT / 32; ++w) t += sh[j * (BT / 32) + w];
        v[j] = t;
    }
}

// streams of every segment, and the ordered kept list kept for inspection.  A thread takes PER
// consecutive candidates, so one scan over the block places them all.  One chunk; `c` carries the
// context of the block's previous chunk in and this one's out.
template <bool RANDK>
__device__ void pack_chunk(const Plan& P, const Tab& tab, uint32_t chunk, ChunkCtx& c, bool merge, uint32_t* wire,
                           long long stride, long long* bits_out, uint32_t* sh_u, uint32_t* sh) {
    const bool plain = P.qz == QS_NONE, has_lvl = qz_has_levels(P.qz), mm = P.qz == QS_MINMAX;
    c = chunk_context(P, tab, chunk, sh_u, &c);
    // this thread's candidates first: their reads overlap the sums below
    uint32_t q[PER], e[PER];
    float val[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t off = c.first + threadIdx.x * PER + i;
        const bool in = off < c.c;
        e[i] = in ? P.cand_idx[c.base + off] : 0u;
        q[i] = (in && !merge) ? P.cand_q[c.base + off] : 0u;
        val[i] = (in && (merge || plain)) ? P.cand_val[c.base + off] : 0.0f;
        if (merge && in) {
            // the quantize stage's part for level-1 quantizers: the sign (the memory update is the closing stage's)
            const uint32_t key = RANDK ? P.cand_key[c.base + off] : topk_key(val[i]);
            if (is_kept<RANDK>(c.un, key, e[i])) {
                const bool neg = val[i] < 0.0f;
                q[i] = Q_SEL | (neg ? Q_NEG : 0u) | 1u;
            }
        }
    }
    uint32_t run_k, run_s, unit_n, pay;
    const uint32_t bi = P.bidx[c.seg], lo = P.seg_off[c.seg];
    if (tab.fast) {
        // positions from the chunk counts of the unit directly (no scan stage ran)
        const uint32_t c1 = tab.cb[c.u + 1];
        uint32_t sums[4] = {0u, 0u, 0u, 0u};          // kept before, sent before, kept in all, sent in all
        for (uint32_t i = c.cb + threadIdx.x; i < c1; i += BT) {
            const uint32_t v = P.chunk_cnt[i];
            sums[2] += v & 0xffffu; sums[3] += v >> 16;
            if (i < chunk) { sums[0] += v & 0xffffu; sums[1] += v >> 16; }
        }
        block_sum4(sums, sh);
        run_k = sums[0]; run_s = sums[1]; unit_n = sums[3];
        pay = P.nseg == 1 ? 2u : P.pay_off[c.u];          // several segments: every kept entry is sent, fixed places
        if (chunk == c.cb && threadIdx.x == 0) {          // the unit's first chunk writes its directory entry
            P.units[c.u].n = unit_n;
            if (sums[2] != P.kseg[c.seg]) set_status(P, QS_STATE);
            uint32_t* row = wire + (size_t)c.r * stride;
            row[2 * c.seg] = mm ? __float_as_uint(order_float(c.un.emin)) : unit_n;      // (min/max: the pair carries (min, max), n = k)
            row[2 * c.seg + 1] = __float_as_uint(mm ? order_float(c.un.emax) : c.un.norm);
            if (P.nseg == 1) {
                const long long bits = 64 + (long long)unit_n * entry_bits(bi, (uint32_t)P.bl, P.qz);
                P.bits[c.r] = bits;
                if (bits_out) bits_out[c.r] = bits;
            } else if (c.seg == 0 && bits_out) {
                bits_out[c.r] = P.bits[c.r];
            }
        }
    } else {
        run_k = P.chunk_sel[chunk] - P.chunk_sel[c.cb];
        run_s = P.chunk_nz[chunk] - P.chunk_nz[c.cb];
        unit_n = c.un.n;
        pay = P.pay_off[c.u];
    }
    uint32_t* w_idx = wire + (size_t)c.r * stride + pay;
    uint32_t* w_sgn = w_idx + words_for(unit_n, bi);
    uint32_t* w_lvl = mm ? w_sgn : w_sgn + words_for(unit_n, 1);          // (no sign stream in front of the min/max levels)
    uint32_t* o_idx = P.sel_idx + (size_t)c.r * P.K + P.kprefix[c.seg];
    uint32_t* o_q = P.sel_q + (size_t)c.r * P.K + P.kprefix[c.seg];
    uint32_t mine = 0;                            // kept | sent << 16 among this thread's candidates
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t kept = (q[i] & Q_SEL) ? 1u : 0u, sent = (kept && (q[i] & 0xffffu)) ? 1u : 0u;
        mine += kept | (sent << 16);
    }
    uint32_t tot;
    const uint32_t ex = block_excl_scan(mine, sh, &tot);
    uint32_t jk = run_k + (ex & 0xffffu), js0 = run_s + (ex >> 16);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t kept = (q[i] & Q_SEL) ? 1u : 0u, sent = (kept && (q[i] & 0xffffu)) ? 1u : 0u;
        if (kept && jk < P.kseg[c.seg]) {                          // (the bound holds by construction)
            o_idx[jk] = e[i];
            o_q[jk] = q[i];
            if (sent && js0 < unit_n) {
                const uint64_t js = js0;
                or_bits(w_idx, js * bi, bi, e[i] - lo);
                if (plain) {
                    w_sgn[js] = __float_as_uint(val[i]);                   // value stream
                } else {
                    if (q[i] & Q_NEG) atomicOr(&w_sgn[js >> 5], 1u << (js & 31u));
                    if (has_lvl) or_bits(w_lvl, js * P.bl, P.bl, (q[i] & 0xffffu) - 1u);
                }
            }
        }
        jk += kept;
        js0 += sent;
    }
}

// every chunk, the blocks taking equal shares of consecutive chunks (mostly one unit each)
template <bool RANDK>
__device__ void stage_pack(const Plan& P, const Tab& tab, bool merge, uint32_t* wire, long long stride,
                           long long* bits_out, uint32_t* sh_u, uint32_t* sh) {
    const uint32_t total = tab.total_chunks;
    ChunkCtx c;
    const uint32_t share = (total + gridDim.x - 1) / gridDim.x;
    const uint32_t c_lo = blockIdx.x * share, c_hi = c_lo + share < total ? c_lo + share : total;
    for (uint32_t chunk = c_lo; chunk < c_hi; ++chunk) pack_chunk<RANDK>(P, tab, chunk, c, merge, wire, stride, bits_out, sh_u, sh);
}

// The unit table as the packing warps of the closing stage need it (their block's copy in shared
// memory is gone by then): unit of every chunk, and (start, candidates, first chunk) of every unit.
__device__ void publish_table(const Plan& P, const Tab& tab) {
    for (uint32_t q = blockIdx.x * BT + threadIdx.x; q < tab.total_chunks; q += gridDim.x * BT) P.chunk_dir[q] = unit_of_chunk(P, tab, q);
    for (uint32_t u = blockIdx.x * BT + threadIdx.x; u < P.U; u += gridDim.x * BT) P.unit_tab[u] = make_uint4(tab.start[u], tab.c[u], tab.cb[u], 0u);
}

// One chunk packed by one warp: the quantizers that send every kept entry at level 1 (whole round;
// the memory update is the closing stage's).  32 rows of 32 candidates; a row's kept entries get
// consecutive places behind those of the rows and chunks before it.
template <bool RANDK>
__device__ void pack_chunk_warp(const Plan& P, uint32_t q, uint32_t* wire, long long stride, long long* bits_out, int lane) {
    const uint32_t u = P.chunk_dir[q];
    const uint4 ut = P.unit_tab[u];                   // start, candidates, first chunk
    const Unit un = P.units[u];
    const uint32_t r = u / P.nseg, seg = u % P.nseg;
    const uint32_t k = P.kseg[seg], bi = P.bidx[seg], lo = P.seg_off[seg];
    const uint32_t j = q - ut.z, first = j * (uint32_t)CHUNK;
    const size_t base = (size_t)r * P.cap + ut.x;
    const bool plain = P.qz == QS_NONE;
    uint32_t before = 0;                              // kept in the unit's earlier chunks
    for (uint32_t i = lane; i < j; i += 32) before += P.chunk_cnt[ut.z + i] & 0xffffu;
    before = warp_sum(before);
    uint32_t* row = wire + (size_t)r * stride;
    uint32_t* w_idx = row + (P.nseg == 1 ? 2u : P.pay_off[u]);
    uint32_t* w_sgn = w_idx + words_for(k, bi);
    uint32_t* o_idx = P.sel_idx + (size_t)r * P.K + P.kprefix[seg];
    uint32_t* o_q = P.sel_q + (size_t)r * P.K + P.kprefix[seg];
    if (j == 0) {                                     // the unit's first chunk writes its directory entry
        const uint32_t nch = (ut.y + CHUNK - 1) / CHUNK;
        uint32_t tot = 0;
        for (uint32_t i = lane; i < nch; i += 32) tot += P.chunk_cnt[ut.z + i] & 0xffffu;
        tot = warp_sum(tot);
        if (lane == 0) {
            if (tot != k) set_status(P, QS_STATE);
            P.units[u].n = k;
            row[2 * seg] = k;
            row[2 * seg + 1] = __float_as_uint(un.norm);
            if (P.nseg == 1) {
                const long long bits = 64 + (long long)k * entry_bits(bi, (uint32_t)P.bl, P.qz);
                P.bits[r] = bits;
                if (bits_out) bits_out[r] = bits;
            } else if (seg == 0 && bits_out) {
                bits_out[r] = P.bits[r];
            }
        }
    }
    uint32_t run = before;
    const uint32_t lt = (1u << lane) - 1u;
    constexpr int RB = 4;                             // rows whose reads are issued together
    for (uint32_t rb = 0; rb < (uint32_t)(CHUNK / 32) && first + rb * 32u < ut.y; rb += RB) {
        uint32_t idx[RB], key[RB];
        float val[RB];
        bool in[RB];
#pragma unroll
        for (int t = 0; t < RB; ++t) {
            const uint32_t off = first + (rb + t) * 32u + (uint32_t)lane;
            in[t] = off < ut.y;
            idx[t] = in[t] ? P.cand_idx[base + off] : 0u;
            val[t] = in[t] ? P.cand_val[base + off] : 0.0f;
            key[t] = RANDK ? (in[t] ? P.cand_key[base + off] : 0u) : topk_key(val[t]);
        }
#pragma unroll
        for (int t = 0; t < RB; ++t) {
            const bool kept = in[t] && is_kept<RANDK>(un, key[t], idx[t]);
            const uint32_t bal = __ballot_sync(0xffffffffu, kept);
            const uint32_t pos = run + __popc(bal & lt);
            if (kept && pos < k) {                                     // (the bound holds by construction)
                const bool neg = val[t] < 0.0f;
                o_idx[pos] = idx[t];
                o_q[pos] = Q_SEL | (neg ? Q_NEG : 0u) | 1u;
                or_bits(w_idx, (uint64_t)pos * bi, bi, idx[t] - lo);
                if (plain) w_sgn[pos] = __float_as_uint(val[t]);       // value stream
                else if (neg) atomicOr(&w_sgn[pos >> 5], 1u << (pos & 31u));
            }
            run += __popc(bal);
        }
    }
}

// chunks handed out to packing warps by a ticket counter
template <bool RANDK>
__device__ void pack_by_warps(const Plan& P, uint32_t total_chunks, uint32_t* wire, long long stride, long long* bits_out, int lane) {
    for (;;) {
        uint32_t q = 0;
        if (lane == 0) q = atomicAdd(P.bar + 6, 1u);
        q = __shfl_sync(0xffffffffu, q, 0);
        if (q >= total_chunks) break;
        pack_chunk_warp<RANDK>(P, q, wire, stride, bits_out, lane);
    }
}

// ------------------------------------------------------------------ master
// entry and stream offsets of each segment, read from the directory
__device__ void stage_dec_prep(const Plan& P, const Active& act, const uint32_t* wire, long long stride, uint32_t* sh) {
    for (int w = blockIdx.x; w < act.n; w += gridDim.x) {
        const int r = act.r[w];
        const uint32_t* row = wire + (size_t)r * stride;
        uint32_t carry_e = 0, carry_w = 2u * P.nseg;
        for (uint32_t base = 0; base < (uint32_t)P.nseg; base += BT) {
            const uint32_t g = base + threadIdx.x;
            uint32_t n = 0, words = 0;
            if (g < (uint32_t)P.nseg) {
                n = P.qz == QS_MINMAX ? P.kseg[g] : row[2 * g];                  // (min/max: every kept entry is sent)
                if (n > P.kseg[g]) { n = 0; set_status(P, QS_INVALID_ARG); }     // not a record of this plan
                words = streams_words(n, P.bidx[g], (uint32_t)P.bl, P.qz);
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

// entries and stream offset of one segment of worker r's record
__device__ __forceinline__ void record_segment(const Plan& P, const uint32_t* wire, long long stride, int r,
                                               uint32_t seg, uint32_t* n, uint32_t* pay) {
    if (P.nseg == 1) {                           // read straight from the record: no offsets to look up
        const uint32_t v = P.qz == QS_MINMAX ? P.kseg[0] : wire[(size_t)r * stride];
        *n = v <= P.kseg[0] ? v : 0u;
        *pay = 2u;
    } else {
        const uint32_t* eb = P.dec_ent + (size_t)r * (P.nseg + 1);
        *n = eb[seg + 1] - eb[seg];
        *pay = P.dec_pay[(size_t)r * P.nseg + seg];
    }
}

__device__ __forceinline__ bool locate_entry(const Plan& P, const uint32_t* wire, long long stride, int r,
                                             uint32_t ent, Entry* out) {
    if (P.nseg == 1) {
        uint32_t n, pay;
        record_segment(P, wire, stride, r, 0u, &n, &pay);
        if (ent >= n) return false;
        out->seg = 0; out->j = ent; out->n = n;
        out->w_idx = wire + (size_t)r * stride + pay;
        out->coord = get_bits(out->w_idx, (uint64_t)ent * P.bidx[0], P.bidx[0]);
        return true;
    }
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
    if (P.qz == QS_NONE) return __uint_as_float(w_sgn[en.j]);       // the value stream sits where the signs would
    if (P.qz == QS_MINMAX)                                          // so does the level stream; the header pair is (min, max)
        return minmax_value(__uint_as_float(row[2 * en.seg]), __uint_as_float(row[2 * en.seg + 1]), P.s,
                            (int)get_bits(w_sgn, (uint64_t)en.j * P.bl, P.bl) + 1);
    const int level = qz_is_sign(P.qz) ? 1 : (int)get_bits(w_lvl, (uint64_t)en.j * P.bl, P.bl) + 1;
    return coord_value(P, __uint_as_float(row[2 * en.seg + 1]), level, neg, P.cscale[en.seg], P.kseg[en.seg]);
}

__device__ void stage_dec_mark(const Plan& P, const Active& act, const uint32_t* wire, long long stride) {
    const uint64_t total = (uint64_t)act.n * P.K;
    for (uint64_t id = (uint64_t)blockIdx.x * BT + threadIdx.x; id < total; id += (uint64_t)gridDim.x * BT) {
        const int r = act.r[id / P.K];
        Entry en;
        if (P.nseg == 1 && P.qz != QS_MINMAX && id % P.K == 0 && wire[(size_t)r * stride] > P.kseg[0]) set_status(P, QS_INVALID_ARG);
        if (!locate_entry(P, wire, stride, r, (uint32_t)(id % P.K), &en)) continue;
        if (en.coord < P.d) atomicOr(&P.touch[en.coord], 1u << r);
        else set_status(P, QS_INVALID_ARG);
    }
}

// The lowest worker that sent an index owns it: it adds the values of all senders in increasing
// worker order and updates x.
__device__ void stage_dec_apply(const Plan& P, const Active& act, const uint32_t* wire, long long stride) {
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
            Entry e2;
            uint32_t pay2;
            e2.seg = en.seg;
            record_segment(P, wire, stride, r2, en.seg, &e2.n, &pay2);
            e2.w_idx = wire + (size_t)r2 * stride + pay2;
            uint32_t lo = 0, hi = e2.n;              // first position with index >= local
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (get_bits(e2.w_idx, (uint64_t)mid * bi, bi) < local) lo = mid + 1; else hi = mid;
            }
            e2.j = lo;
            e2.coord = en.coord;
            acc = acc + entry_value(P, wire + (size_t)r2 * stride, e2);
        }
        const float xn = P.x[en.coord] - acc / (float)P.rdiv;
        P.x[en.coord] = xn;
        P.touch[en.coord] = 0u;
    }
}

// ------------------------------------------------------------------ master update + broadcast
// Closing stage of a whole round: x <- x - (1/R) sum_r g_r and xw_r <- x in ONE pass over x.
//
// Tiles of x (2048 coordinates) are handed out by a ticket counter.  In every block one warp keeps
// the copies going through a ring of slots in shared memory: a tile of x comes in with one bulk
// copy and with it, one more bulk copy per active worker, the tile's candidate runs as the dense
// pass left them ((index, value) pairs; their counts were read a tile ahead); when a tile has been
// worked on it goes out to every active worker's row (and anchor row) as bulk stores.  Four
// other warps, one per slot, work on the tiles that have landed: from the unit's
// threshold, tie cut and norm a warp decides which candidates were kept and sent and what value
// g each stands for (the same expression the worker used for its memory), and applies them to
// the tile in shared memory:
//   - a coordinate with one sender: x - (0 + g) / R, on the spot;
//   - a coordinate with several senders (found with two bitmaps of the tile in shared memory):
//     the entries are listed, and the entry of the lowest worker adds the values in increasing
//     worker order before it updates x.  The list is bounded; when a tile has more such
//     coordinates than it holds, the sums are formed in the tile's own buffer worker after worker
//     and x is read again;
//   - a crowded tile (1024 candidates or more: tensors every worker keeps whole) skips the
//     bitmaps and is walked worker after worker from the start, its runs coming through a ring
//     of asynchronous copies; such tiles are handed out first (Plan::tile_order).
// Updated coordinates are also written to x in global memory.  No sender bitmaps over d, no
// scattered reads of x, no stage for shared indices: everything the update needs is in the
// tile's runs, and the copies never wait for the arithmetic as long as the working warps keep up.
// Rows that are not 16-byte aligned take the same steps with ordinary loads and stores, a warp
// per tile; so do the candidates of a tile that has more of them than the buffer holds.
constexpr int NSLOT = 4;           // tiles of a block in shared memory: coming in, worked on, going out
constexpr int NWORK = NSLOT;       // warps that work on landed tiles (warps 1 .. NWORK; warp 0 copies): one per slot, so
                                   // that each sees every phase of its slot's barrier in turn
constexpr int ML_CAP = 160;        // listed entries of coordinates with several senders
constexpr int CB = 416;            // candidates of a tile (all workers) held in shared memory
constexpr uint32_t NO_TILE = 0xffffffffu;

struct BcSlot {
    float xs[STILE];               // a tile of x
    uint2 cb[CB];                  // its candidates, worker after worker (each run padded to an even count);
                                   // once looked at, an entry holds (position | sent << 31, value)
    uint32_t cnt[32];              // candidates of each active worker (slot order)
    uint32_t pbefore[32];          // where its run starts in cb
    uint32_t gseg[STILE / GROUP];  // segment of the first coordinate of each 128-coordinate group
    uint32_t tile, staged;
    uint32_t whole;                // the working warp asks for the whole tile to be stored to x (many coordinates changed)
    uint32_t crowded;              // so many candidates that the tile is walked worker by worker
};

struct BcScratch {                 // of one working warp
    uint32_t bm1[STILE / 32];      // coordinates of the tile some worker sent
    uint32_t bm2[STILE / 32];      // coordinates several workers sent
    uint32_t pref[STILE / 32];     // such coordinates before each word of bm2
    uint32_t mpos[ML_CAP];         // listed entry: position in the tile | worker slot << 16
    float mg[ML_CAP];              // its value
    uint32_t nm, pad[3];
};

struct BcBlock {
    BcSlot slot[NSLOT];
    BcScratch scr[NWORK];
    uint64_t full[NSLOT];          // the slot's copies have landed (or the end mark is in place)
    uint64_t done[NSLOT];          // the slot's tile has been worked on
    int abort, pad[3];
};
static_assert(sizeof(BcSlot) % 16 == 0 && sizeof(BcScratch) % 16 == 0, "tile buffers are the targets of bulk copies");
constexpr size_t MID_SCRATCH_BYTES = (ORDER_ITEMS_MAX + 8) * sizeof(uint32_t) + FB_BINS * 4;
constexpr size_t MID_POOL_BYTES = sizeof(BcBlock) > MID_SCRATCH_BYTES ? sizeof(BcBlock) : MID_SCRATCH_BYTES;

// what a lane keeps about the unit (its worker, a segment) its candidates mostly belong to
struct UnitLite { uint32_t tau, tie_max, k, end; float norm, c, lo; };   // (min/max quantizer: lo = smallest, norm = largest kept value)

// Lanes to workers: the warp is cut into as many equal parts as the next power of two of the
// active workers; part j of worker slot w (lane w + j * parts) walks entries j, j + J, .. of the
// worker's run.  Everything a lane needs about its worker sits in its own registers: no shuffles
// or searches per candidate.
struct LaneMap {
    int nact, my_w;
    uint32_t J, my_j, my_r;
    bool live;
};

__device__ __forceinline__ LaneMap lane_map(const Active& act, int lane) {
    LaneMap L;
    L.nact = act.n;
    int parts = 1;
    while (parts < L.nact) parts <<= 1;               // nact <= 32
    L.J = 32u / (uint32_t)parts;
    L.my_w = lane & (parts - 1);
    L.my_j = (uint32_t)lane / (uint32_t)parts;
    L.live = L.my_w < L.nact;
    L.my_r = L.live ? (uint32_t)act.r[L.my_w] : 0u;
    return L;
}

__device__ __forceinline__ UnitLite unit_of(const Plan& P, uint32_t r, uint32_t seg) {
    UnitLite u;
    const Unit& g = P.units[(size_t)r * P.nseg + seg];
    u.tau = g.tau; u.tie_max = g.tie_max; u.norm = g.norm; u.lo = 0.0f;
    if (P.qz == QS_MINMAX) { u.lo = order_float(g.emin); u.norm = order_float(g.emax); }
    u.k = P.kseg[seg]; u.c = P.cscale[seg]; u.end = P.seg_off[seg + 1];
    return u;
}

__device__ __forceinline__ UnitLite unit_lite(const Plan& P, const LaneMap& L, uint32_t seg) {
    const UnitLite none = {0u, 0u, 0u, 0u, 0.0f, 0.0f, 0.0f};
    return L.live ? unit_of(P, L.my_r, seg) : none;
}

// First look at one entry of worker r's run in the tile that starts at e0: was it sent, and with
// what value?  un: the unit of the tile's first segment, later: the last unit looked up beyond it
// (a walk's entries come in rising order, so it serves until its segment ends).  mem_update: the
// worker's memory at a sent coordinate is written here (quantizers without a quantize stage).
template <bool RANDK>
__device__ __forceinline__ bool first_look(const Plan& P, uint32_t r, const UnitLite& un, UnitLite& later, const uint32_t* gseg,
                                           uint32_t e0, uint32_t nel, uint2 ent, bool mem_update, uint32_t* pos, float* g) {
    const uint32_t idx = ent.x;
    bool sent = idx >= e0 && idx - e0 < nel;                        // (an entry outside its tile is never written by the dense pass)
    float gv = 0.0f;
    if (sent) {
        UnitLite u = un;
        if (idx >= un.end) {                          // a later segment of the tile: look its unit up
            if (idx >= later.end) {
                uint32_t seg = gseg[(idx - e0) >> 7];
                while (seg + 1 < (uint32_t)P.nseg && idx >= P.seg_off[seg + 1]) ++seg;
                later = unit_of(P, r, seg);
            }
            u = later;
        }
        const float val = __uint_as_float(ent.y);
        const uint32_t key = RANDK ? ~philox_word(P, r, idx, 1u) : topk_key(val);
        sent = key > u.tau || (key == u.tau && idx <= u.tie_max);
        if (sent) {
            if (P.qz == QS_NONE) {
                gv = val;
            } else if (P.qz == QS_MINMAX) {
                gv = minmax_value(u.lo, u.norm, P.s, minmax_level(val, u.lo, u.norm, P.s, philox_word(P, r, idx, 0u)));
            } else {
                int level = 1;
                if (!qz_is_sign(P.qz)) level = qsgd_level(val, u.norm, P.s, philox_word(P, r, idx, 0u));
                sent = level != 0;                                 // (level 0: kept, not sent)
                if (sent) {                                        // the value as coord_value forms it
                    if (qz_is_sign(P.qz)) {
                        gv = u.norm / (float)u.k;
                    } else {
                        gv = (u.norm * (float)level) / (float)P.s;
                        if (P.qz == QS_QSGD_SCALED) gv = gv * u.c;
                    }
                    if (val < 0.0f) gv = -gv;
                }
            }
        }
        if (mem_update && sent) P.mem[(size_t)r * P.d + idx] = val - gv;
    }
    *pos = sent ? idx - e0 : 0u;
    *g = gv;
    return sent;
}

// The update of one tile by one warp.  xs: the tile in shared memory; cnt: candidates of this
// lane's worker in the tile; cb + pbefore: where they are in shared memory (staged), otherwise they
// are read from the run in global memory; gseg: the tile's group-to-segment entries.  mem_update:
// the warp also writes m <- u - g at the sent coordinates (level-1 quantizers in a whole round).
// Returns true when it leaves the tile's write-back to x to the caller (can_whole: the caller can
// store the whole tile; taken when so many coordinates changed that one sequential store is cheaper
// than their scattered sectors).
constexpr uint32_t WHOLE_TILE_MIN = 64;
constexpr uint32_t CROWDED_MIN = 1024;               // candidates of all workers from which a tile is walked worker by worker

template <bool RANDK>
__device__ bool apply_tile(const Plan& P, const LaneMap& L, int lane, uint32_t tile, uint32_t cnt, bool staged, uint2* cb,
                           uint32_t pbefore, const uint32_t* gseg, float* xs, BcScratch& W, const UnitLite& un, bool mem_update,
                           bool can_whole, bool crowded) {
    const uint32_t e0 = tile * (uint32_t)STILE;
    const uint32_t nel = P.d - e0 < (uint32_t)STILE ? P.d - e0 : (uint32_t)STILE;
    const float rdiv = (float)P.rdiv;
    const uint32_t wp = (uint32_t)(ML_CAP / (L.nact > 0 ? L.nact : 1));   // coordinates with several senders the list can take
    const uint32_t J = L.J, my_j = L.my_j, my_r = L.my_r;
    uint2* run = P.stage + (size_t)my_r * P.cap + (size_t)tile * STILE;
    // What will be read from global memory is asked for now, all of it at once (one round trip in
    // place of one per entry): the run itself when it is not in shared memory, and the units of
    // the next few segments when the tile may hold more than one.
    constexpr uint32_t AHEAD = 8;                     // lines asked for ahead of a crowded tile's walk without the ring
    if (!staged && !crowded)
        for (uint32_t line = my_j; line * 16u < cnt; line += J) asm volatile("prefetch.global.L1 [%0];" ::"l"(run + line * 16u));
    if (un.end < e0 + nel && L.live) {
        const uint32_t s0 = gseg[0];
        for (uint32_t j = 1 + my_j; j <= 4u * J && s0 + j < (uint32_t)P.nseg; j += J)
            asm volatile("prefetch.global.L1 [%0];" ::"l"(&P.units[(size_t)my_r * P.nseg + s0 + j].tau));
    }
    // Entry i of this lane's worker's run: sent?  position in the tile and value.  The first look
    // at an entry leaves the answer in its place (in shared memory, or in the run itself, which
    // nothing reads after this stage), so that the random draws and the division are made once.
    UnitLite later = {0u, 0u, 0u, 0u, 0.0f, 0.0f, 0.0f};
    auto cand = [&](uint32_t i, bool first, uint32_t* pos, float* g) -> bool {
        uint2* home = staged ? &cb[pbefore + i] : &run[i];
        const uint2 ent = *home;
        if (!first) {                                 // looked at before: the answer is in place
            *pos = ent.x & (uint32_t)(STILE - 1);
            *g = __uint_as_float(ent.y);
            return (ent.x >> 31) != 0u;
        }
        const bool sent = first_look<RANDK>(P, my_r, un, later, gseg, e0, nel, ent, mem_update, pos, g);
        *home = make_uint2(*pos | (sent ? 0x80000000u : 0u), __float_as_uint(*g));
        return sent;
    };
    // A crowded tile (small tensors that every worker sends whole, so that most coordinates have
    // several senders): one walk, worker after worker in their order with all lanes on one
    // worker's entries, the sums formed in the tile's own buffer.  A worker sends a coordinate at
    // most once, so its lanes never meet at one sum; a coordinate with one sender gets 0 + g as
    // everywhere else; x itself is read again from global memory, which still holds the round's
    // model; a sum of zero leaves x as it is, as x - 0 / R would.  No bitmaps of senders: with all
    // workers at the same coordinates their words would be fought over.
    if (crowded) {
        // x again at the end: asked for now, so that it waits in the L1 by then
        for (uint32_t line = lane; line * 32u < nel; line += 32) asm volatile("prefetch.global.L1 [%0];" ::"l"(P.x + e0 + line * 32u));
        for (uint32_t j = lane; j < (uint32_t)STILE; j += 32) xs[j] = 0.0f;
        __syncwarp();
        // The runs come through a ring of RING_N pieces of RING_E entries in the slot's candidate
        // buffer (free: a crowded tile is never staged), filled by asynchronous 16-byte copies that
        // run RING_N - 1 pieces ahead of the walk and across the change from one worker to the next:
        // a load from the L2 or from HBM takes microseconds while the broadcast's stores fill the
        // memory system, and one load per 32 entries would wait that long every time.
        constexpr uint32_t RING_E = 64, RING_N = 6;
        static_assert(RING_E * RING_N <= (uint32_t)CB, "the ring lives in the candidate buffer");
        const bool ring = cb != nullptr && !staged && (P.cap & 1ull) == 0ull && (reinterpret_cast<uintptr_t>(P.stage) & 15u) == 0u;
        uint32_t iw = 0, ic = 0, islot = 0;            // filling: worker slot, piece of its run, ring place
        auto fill = [&]() {
            uint32_t cnt_i = 0;
            while (iw < (uint32_t)L.nact && ic * RING_E >= (cnt_i = __shfl_sync(0xffffffffu, cnt, iw))) { ++iw; ic = 0; }
            if (iw < (uint32_t)L.nact) {
                const uint32_t r_i = __shfl_sync(0xffffffffu, my_r, iw);
                const uint32_t at = ic * RING_E + 2u * (uint32_t)lane;        // this lane's pair of entries (rows are even: a pair never crosses a row's end)
                const uint2* src = P.stage + (size_t)r_i * P.cap + (size_t)tile * STILE + at;
                if (at < cnt_i)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(cb + (islot % RING_N) * RING_E + 2u * (uint32_t)lane)), "l"(src) : "memory");
                ++ic;
            }
            asm volatile("cp.async.commit_group;" ::: "memory");     // (an empty group keeps the count in step)
            ++islot;
        };
        if (ring)
            for (uint32_t q = 0; q + 1 < RING_N; ++q) fill();
        uint32_t cslot = 0;
        for (int w = 0; w < L.nact; ++w) {
            const uint32_t cnt_w = __shfl_sync(0xffffffffu, cnt, w);
            const uint32_t r_w = __shfl_sync(0xffffffffu, my_r, w);
            // the unit of the tile's first segment, from the lane that holds this worker's
            UnitLite uw;
            uw.tau = __shfl_sync(0xffffffffu, un.tau, w); uw.tie_max = __shfl_sync(0xffffffffu, un.tie_max, w);
            uw.k = __shfl_sync(0xffffffffu, un.k, w); uw.end = __shfl_sync(0xffffffffu, un.end, w);
            uw.norm = __shfl_sync(0xffffffffu, un.norm, w); uw.c = __shfl_sync(0xffffffffu, un.c, w);
            uw.lo = __shfl_sync(0xffffffffu, un.lo, w);
            UnitLite lw = {0u, 0u, 0u, 0u, 0.0f, 0.0f, 0.0f};
            if (ring) {
                for (uint32_t c0 = 0; c0 < cnt_w; c0 += RING_E) {
                    fill();
                    asm volatile("cp.async.wait_group %0;" ::"n"(RING_N - 1) : "memory");
                    __syncwarp();                     // every lane's part of the piece has landed
                    const uint2* piece = cb + (cslot % RING_N) * RING_E;
#pragma unroll
                    for (uint32_t h = 0; h < RING_E; h += 32) {
                        const uint32_t i = c0 + h + (uint32_t)lane;
                        uint32_t pos = 0;
                        float g = 0.0f;
                        if (i < cnt_w && first_look<RANDK>(P, r_w, uw, lw, gseg, e0, nel, piece[h + lane], mem_update, &pos, &g))
                            xs[pos] = xs[pos] + g;
                    }
                    __syncwarp();                     // the piece may be filled again
                    ++cslot;
                }
            } else {
                const uint2* run_w = staged ? cb + __shfl_sync(0xffffffffu, pbefore, w) : P.stage + (size_t)r_w * P.cap + (size_t)tile * STILE;
                uint2 nxt = make_uint2(0u, 0u);
                if ((uint32_t)lane < cnt_w) nxt = run_w[lane];
                for (uint32_t i = lane; i < cnt_w; i += 32) {
                    const uint2 ent = nxt;
                    if (i + 32u < cnt_w) nxt = run_w[i + 32u];
                    if (!staged && (lane & 15) == 0 && i + AHEAD * 16u < cnt_w) asm volatile("prefetch.global.L1 [%0];" ::"l"(run_w + i + AHEAD * 16u));
                    uint32_t pos = 0;
                    float g = 0.0f;
                    if (first_look<RANDK>(P, r_w, uw, lw, gseg, e0, nel, ent, mem_update, &pos, &g)) xs[pos] = xs[pos] + g;
                }
            }
            __syncwarp();
        }
        if (ring) asm volatile("cp.async.wait_group 0;" ::: "memory");
        for (uint32_t m0 = 0; m0 < (uint32_t)(STILE / 32); m0 += 4) {
            float xv[4];
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) {
                const uint32_t j = (m0 + q) * 32u + (uint32_t)lane;
                xv[q] = j < nel ? P.x[e0 + j] : 0.0f;
            }
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) {
                const uint32_t j = (m0 + q) * 32u + (uint32_t)lane;
                bool ch = false;
                if (j < nel) {
                    const float sum = xs[j];
                    ch = sum != 0.0f;
                    xs[j] = ch ? xv[q] - sum / rdiv : xv[q];
                }
                const uint32_t bits = __ballot_sync(0xffffffffu, ch);
                if (lane == 0) W.bm1[m0 + q] = bits;
            }
        }
        __syncwarp();
    } else {
    // senders per coordinate
    for (uint32_t i = my_j; i < cnt; i += J) {
        uint32_t pos = 0;
        float g = 0.0f;
        if (cand(i, true, &pos, &g)) {
            const uint32_t bit = 1u << (pos & 31u);
            if (atomicOr(&W.bm1[pos >> 5], bit) & bit) atomicOr(&W.bm2[pos >> 5], bit);
        }
    }
    __syncwarp();
    const uint32_t m_lo = W.bm2[lane], m_hi = W.bm2[lane + 32];
    const bool any_multi = __any_sync(0xffffffffu, (m_lo | m_hi) != 0u);
    // rank of a coordinate among those with several senders: popcounts before its word
    uint32_t npos = 0;
    if (any_multi) {
        const uint32_t c_lo = __popc(m_lo), c_hi = __popc(m_hi);
        const uint32_t i_lo = warp_incl_scan(c_lo, lane), i_hi = warp_incl_scan(c_hi, lane);
        const uint32_t n_lo = __shfl_sync(0xffffffffu, i_lo, 31);
        npos = n_lo + __shfl_sync(0xffffffffu, i_hi, 31);
        W.pref[lane] = i_lo - c_lo;
        W.pref[lane + 32] = n_lo + i_hi - c_hi;
        __syncwarp();
    }
    if (npos > wp) {
        // Many coordinates with several senders (small tensors that every worker sends whole):
        // the sums are formed in the tile's own buffer, worker after worker in their order, all
        // lanes on one worker's entries at a time; x itself is read again from global memory, which
        // still holds the round's model.  A worker sends a coordinate at most once, so its lanes
        // never meet at one sum, and a coordinate with one sender gets 0 + g as everywhere else.
        // Time is in proportion to the candidates.
        for (uint32_t j = lane; j < nel; j += 32)
            if ((W.bm1[j >> 5] >> (j & 31u)) & 1u) xs[j] = 0.0f;
        __syncwarp();
        for (int w = 0; w < L.nact; ++w) {
            const uint32_t cnt_w = __shfl_sync(0xffffffffu, cnt, w);
            const uint32_t pb_w = __shfl_sync(0xffffffffu, pbefore, w);
            const uint32_t r_w = __shfl_sync(0xffffffffu, my_r, w);
            const uint2* run_w = staged ? cb + pb_w : P.stage + (size_t)r_w * P.cap + (size_t)tile * STILE;
            for (uint32_t i0 = 0; i0 < cnt_w; i0 += 128u) {
                uint2 e[4];
                if (!staged && i0 + 256u + (uint32_t)lane * 16u < cnt_w)            // the batch after the next, by lines
                    asm volatile("prefetch.global.L1 [%0];" ::"l"(run_w + i0 + 256u + (uint32_t)lane * 16u));
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t i = i0 + (uint32_t)q * 32u + (uint32_t)lane;
                    e[q] = i < cnt_w ? run_w[i] : make_uint2(0u, 0u);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (e[q].x >> 31) {
                        const uint32_t pos = e[q].x & (uint32_t)(STILE - 1);
                        xs[pos] = xs[pos] + __uint_as_float(e[q].y);
                    }
            }
            __syncwarp();
        }
        for (uint32_t j = lane; j < nel; j += 32)
            if ((W.bm1[j >> 5] >> (j & 31u)) & 1u) xs[j] = P.x[e0 + j] - xs[j] / rdiv;
        __syncwarp();
    } else {
    // coordinates with one sender
    for (uint32_t i = my_j; i < cnt; i += J) {
        uint32_t pos = 0;
        float g = 0.0f;
        if (cand(i, false, &pos, &g) && !((W.bm2[pos >> 5] >> (pos & 31u)) & 1u)) {
            float acc = 0.0f;
            acc = acc + g;
            xs[pos] = xs[pos] - acc / rdiv;
        }
    }
    if (any_multi) {
        for (uint32_t w0 = 0; w0 < npos; w0 += wp) {
            for (uint32_t i = my_j; i < cnt; i += J) {
                uint32_t pos = 0;
                float g = 0.0f;
                if (!cand(i, false, &pos, &g)) continue;
                const uint32_t wbits = W.bm2[pos >> 5];
                if (!((wbits >> (pos & 31u)) & 1u)) continue;
                const uint32_t rank = W.pref[pos >> 5] + __popc(wbits & ((1u << (pos & 31u)) - 1u));
                if (rank < w0 || rank >= w0 + wp) continue;
                const uint32_t at = atomicAdd(&W.nm, 1u);
                if (at < (uint32_t)ML_CAP) { W.mpos[at] = pos | ((uint32_t)L.my_w << 16); W.mg[at] = g; }
            }
            __syncwarp();
            const uint32_t n = W.nm < (uint32_t)ML_CAP ? W.nm : (uint32_t)ML_CAP;
            if (W.nm > (uint32_t)ML_CAP) set_status(P, QS_STATE);          // (at most wp x nact entries are listed)
            for (uint32_t j = lane; j < n; j += 32) {
                const uint32_t me = W.mpos[j], pos = me & 0xffffu, slot = me >> 16;
                bool owner = true;
                for (uint32_t i = 0; i < n; ++i) {
                    const uint32_t o = W.mpos[i];
                    if ((o & 0xffffu) == pos && (o >> 16) < slot) owner = false;
                }
                if (!owner) continue;
                float acc = 0.0f;
                int last = -1;
                for (;;) {                            // the senders in increasing worker order
                    int best = 1 << 30;
                    float gb = 0.0f;
                    for (uint32_t i = 0; i < n; ++i) {
                        const uint32_t o = W.mpos[i];
                        const int so = (int)(o >> 16);
                        if ((o & 0xffffu) == pos && so > last && so < best) { best = so; gb = W.mg[i]; }
                    }
                    if (best == (1 << 30)) break;
                    acc = acc + gb;
                    last = best;
                }
                xs[pos] = xs[pos] - acc / rdiv;
            }
            __syncwarp();
            if (lane == 0) W.nm = 0u;
            __syncwarp();
        }
    }
    }
    }
    __syncwarp();                                     // every lane is done with the tile and the bitmaps
    // x in global memory: every changed coordinate's 32-byte sector, whole and once (a sector
    // written in full needs no read of what it held), or the whole tile by the caller
    const uint32_t b_lo = W.bm1[lane], b_hi = W.bm1[lane + 32];
    const uint32_t changed = warp_sum(__popc(b_lo) + __popc(b_hi));
    const bool whole = can_whole && changed >= WHOLE_TILE_MIN;
    if (!whole && changed) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t bits = h ? b_hi : b_lo;
            const uint32_t p0 = ((uint32_t)lane + 32u * h) * 32u;      // first position of the word
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (!((bits >> (8 * q)) & 0xffu)) continue;
                const uint32_t p = p0 + 8u * q;
                if (((reinterpret_cast<uintptr_t>(P.x + e0 + p)) & 31u) == 0 && p + 8u <= nel) {
                    const float4 a = *reinterpret_cast<const float4*>(xs + p), b = *reinterpret_cast<const float4*>(xs + p + 4);
                    *reinterpret_cast<float4*>(P.x + e0 + p) = a;
                    *reinterpret_cast<float4*>(P.x + e0 + p + 4) = b;
                } else {                              // rows off the 32-byte grid, or the ragged end: the changed coordinates alone
                    for (uint32_t i = 0; i < 8u; ++i)
                        if ((bits >> (8 * q + i)) & 1u) P.x[e0 + p + i] = xs[p + i];
                }
            }
        }
    }
    W.bm1[lane] = 0u; W.bm1[lane + 32] = 0u; W.bm2[lane] = 0u; W.bm2[lane + 32] = 0u;
    return whole;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// bounded wait that also gives up when another warp of the block has
__device__ __forceinline__ bool mbar_wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
    }
}

__device__ __forceinline__ uint32_t tile_count(const Plan& P, const LaneMap& L, uint32_t tile) {
    uint32_t c = (L.live && tile < P.ntile) ? P.tile_cnt[(size_t)L.my_r * P.nblk * BLK_TILES + tile] : 0u;
    return c < (uint32_t)STILE ? c : (uint32_t)STILE;
}

// 16-byte-aligned rows: warp 0 copies, warps 1 .. NWORK work on the tiles
// pack_chunks > 0: the block's other warps write the records meanwhile (pack_by_warps)
template <bool RANDK>
__device__ void stage_update_broadcast(const Plan& P, const Active& act, BcBlock& B, bool mem_update, uint32_t pack_chunks,
                                       uint32_t* wire, long long stride, long long* bits_out) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int i = 0; i < NSLOT; ++i) { mbar_init(&B.full[i], 1); mbar_init(&B.done[i], 1); }
        B.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (wid >= 1 && wid <= NWORK) {
        BcScratch& W = B.scr[wid - 1];
        W.bm1[lane] = 0u; W.bm1[lane + 32] = 0u; W.bm2[lane] = 0u; W.bm2[lane + 32] = 0u;
        if (lane == 0) W.nm = 0u;
    }
    fence_async_smem();                               // the buffers were ordinary shared memory until now
    __syncthreads();
    if (wid > NWORK) {
        if (pack_chunks) pack_by_warps<RANDK>(P, pack_chunks, wire, stride, bits_out, lane);
        return;
    }
    const LaneMap L = lane_map(act, lane);
    const bool one_seg = P.nseg == 1;
    const uint32_t ntile = P.ntile;
    volatile int* abort_flag = &B.abort;
    if (wid == 0) {
        // ---- the copying warp
        asm volatile("fence.proxy.async.global;" ::: "memory");   // x and the runs may have been written with ordinary stores
        // tickets are drawn two tiles ahead of the copies and counts read one tile ahead, so that
        // neither round trip is on the path
        uint32_t tA = 0, tB = 0;
        auto draw = [&]() -> uint32_t {                // the next tile in the order they are handed out
            const uint32_t t = atomicAdd(P.bar + 2, 1u);
            return (P.tile_order && t < ntile) ? P.tile_order[t] : t;
        };
        if (lane == 0) { tA = draw(); tB = draw(); }
        tA = __shfl_sync(0xffffffffu, tA, 0);
        tB = __shfl_sync(0xffffffffu, tB, 0);
        auto gseg_of = [&](uint32_t tile) -> uint32_t {
            return (!one_seg && lane < STILE / GROUP && tile < ntile) ? P.grp_seg[(size_t)tile * (STILE / GROUP) + lane] : 0u;
        };
        uint32_t cntA = tile_count(P, L, tA), gsA = gseg_of(tA);
        // starts the copies of the next tile into slot s (or leaves the end mark there)
        auto arm = [&](uint32_t s) {
            BcSlot& S = B.slot[s];
            const uint32_t tile = tA;
            uint32_t tC = 0;
            if (lane == 0) tC = draw();
            const uint32_t cntB = tile_count(P, L, tB), gsB = gseg_of(tB);
            if (tile >= ntile) {
                if (lane == 0) { S.tile = NO_TILE; mbar_expect(&B.full[s], 0u); }
            } else {
                const uint32_t e0 = tile * (uint32_t)STILE;
                const uint32_t nel = P.d - e0 < (uint32_t)STILE ? P.d - e0 : (uint32_t)STILE;
                const uint32_t padded = L.my_j == 0u ? (cntA + 1u) & ~1u : 0u;
                const uint32_t pincl = warp_incl_scan(padded, lane);
                const uint32_t ptotal = __shfl_sync(0xffffffffu, pincl, 31);
                const bool staged = ptotal <= (uint32_t)CB;
                if (L.my_j == 0u) { S.cnt[L.my_w] = cntA; S.pbefore[L.my_w] = pincl - padded; }
                if (lane < STILE / GROUP) S.gseg[lane] = gsA;
                if (lane == 0) {
                    S.tile = tile;
                    S.staged = staged ? 1u : 0u;
                    S.crowded = ptotal >= CROWDED_MIN ? 1u : 0u;
                    mbar_expect(&B.full[s], nel * 4u + (staged ? ptotal * 8u : 0u));
                    bulk_load(S.xs, P.x + e0, nel * 4u, &B.full[s]);
                }
                __syncwarp();                         // the bytes are announced before any run's copy starts
                if (staged && cntA && L.my_j == 0u)
                    bulk_load(&S.cb[pincl - padded], P.stage + (size_t)L.my_r * P.cap + (size_t)tile * STILE, padded * 8u, &B.full[s]);
            }
            tA = tB; cntA = cntB; gsA = gsB;
            tB = __shfl_sync(0xffffffffu, tC, 0);
            __syncwarp();                             // the slot's header is visible to the whole warp
        };
        uint32_t armed = 0;                           // tiles (or end marks) whose slot has been armed
        for (; armed < (uint32_t)(NSLOT - 1); ++armed) arm(armed);
        uint32_t si = 0;
        for (;; ++si) {
            const uint32_t s = si % NSLOT;
            BcSlot& S = B.slot[s];
            const uint32_t tile = S.tile;             // written by this warp
            if (tile == NO_TILE) break;
            const bool ok = mbar_wait_or_abort(&B.done[s], (si / NSLOT) & 1u, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            if (lane == 0) {
                const uint32_t e0 = tile * (uint32_t)STILE;
                const uint32_t nel = P.d - e0 < (uint32_t)STILE ? P.d - e0 : (uint32_t)STILE;
                if (S.whole) bulk_store(P.x + e0, S.xs, nel * 4u);
                for (int w = 0; w < act.n; ++w) {
                    bulk_store(P.xw + (size_t)act.r[w] * P.d + e0, S.xs, nel * 4u);
                    if (P.anchors) bulk_store(P.anchors + (size_t)act.r[w] * P.d + e0, S.xs, nel * 4u);
                }
                bulk_commit();
                bulk_wait_read<1>();                  // the stores of the tile before have read their slot: it is armed next
            }
            __syncwarp();
            arm(armed % NSLOT);
            ++armed;
        }
        if (!*abort_flag) {
            // the slot that has not seen an end mark yet (only its header is written: the stores that
            // may still be reading its tile are not disturbed)
            arm(armed % NSLOT);
            ++armed;
        }
        if (*abort_flag) {
            // copies already started get a bounded chance to land before the block leaves
            for (uint32_t i = si; i < armed; ++i) mbar_wait(&B.full[i % NSLOT], (i / NSLOT) & 1u);
            if (lane == 0) set_status(P, QS_TIMEOUT);
        }
        if (lane == 0) bulk_wait_all();               // nothing of this block may still be reading shared memory
    } else {
        // ---- a working warp: the tiles that come through slot wid - 1
        BcScratch& W = B.scr[wid - 1];
        UnitLite un = unit_lite(P, L, 0u);
        const uint32_t s = (uint32_t)(wid - 1);
        BcSlot& S = B.slot[s];
        for (uint32_t use = 0;; ++use) {
            const bool ok = mbar_wait_or_abort(&B.full[s], use & 1u, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            const uint32_t tile = S.tile;
            if (tile == NO_TILE) break;
            if (!one_seg) un = unit_lite(P, L, S.gseg[0]);
            const uint32_t cnt = L.live ? S.cnt[L.my_w] : 0u;
            const bool whole = apply_tile<RANDK>(P, L, lane, tile, cnt, S.staged != 0u, S.cb, L.live ? S.pbefore[L.my_w] : 0u, S.gseg, S.xs,
                                                 W, un, mem_update, true, S.crowded != 0u);
            if (lane == 0) S.whole = whole ? 1u : 0u;
            fence_async_smem();                       // the tile as updated must be what the bulk stores read
            __syncwarp();
            if (lane == 0) mbar_arrive(&B.done[s]);
        }
    }
}

// rows that are not 16-byte aligned: warps 0 .. NWORK - 1 take a tile each by ticket, ordinary loads and stores
template <bool RANDK>
__device__ void stage_update_broadcast_plain(const Plan& P, const Active& act, BcBlock& B, bool mem_update, uint32_t pack_chunks,
                                             uint32_t* wire, long long stride, long long* bits_out) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (wid >= NWORK) {
        if (pack_chunks) pack_by_warps<RANDK>(P, pack_chunks, wire, stride, bits_out, lane);
        return;
    }
    BcScratch& W = B.scr[wid];
    float* xs = B.slot[wid].xs;
    uint32_t* gseg = B.slot[wid].gseg;
    W.bm1[lane] = 0u; W.bm1[lane + 32] = 0u; W.bm2[lane] = 0u; W.bm2[lane + 32] = 0u;
    if (lane == 0) W.nm = 0u;
    __syncwarp();
    const LaneMap L = lane_map(act, lane);
    const bool one_seg = P.nseg == 1;
    UnitLite un = unit_lite(P, L, 0u);
    for (;;) {
        uint32_t tile = 0;
        if (lane == 0) tile = atomicAdd(P.bar + 2, 1u);
        tile = __shfl_sync(0xffffffffu, tile, 0);
        if (tile >= P.ntile) break;
        const uint32_t e0 = tile * (uint32_t)STILE;
        const uint32_t nel = P.d - e0 < (uint32_t)STILE ? P.d - e0 : (uint32_t)STILE;
        for (uint32_t i = lane; i < nel; i += 32) xs[i] = P.x[e0 + i];
        if (lane < STILE / GROUP) gseg[lane] = one_seg ? 0u : P.grp_seg[(size_t)tile * (STILE / GROUP) + lane];
        __syncwarp();
        if (!one_seg) un = unit_lite(P, L, gseg[0]);
        apply_tile<RANDK>(P, L, lane, tile, tile_count(P, L, tile), false, nullptr, 0u, gseg, xs, W, un, mem_update, false, false);
        __syncwarp();
        for (int w = 0; w < act.n; ++w)
            for (uint32_t i = lane; i < nel; i += 32) {
                const float v = xs[i];
                P.xw[(size_t)act.r[w] * P.d + e0 + i] = v;
                if (P.anchors) P.anchors[(size_t)act.r[w] * P.d + e0 + i] = v;
            }
        __syncwarp();
    }
}

// ------------------------------------------------------------------ the persistent kernel
// In a whole round with a level-1 quantizer (sign, none) nothing of the records depends on the
// closing stage and nothing of the closing stage on the records: both start from the thresholds
// and norms.  When the chunks are few enough (a couple per packing warp) the records are written
// by the warps that have no part in the closing stage, in its shadow; otherwise, and for QSGD
// (whose levels need a stage of their own first), every block packs its share before it.
constexpr uint32_t PACK_WARPS = BT / 32 - 1 - NWORK;      // warps of a block free to pack during the closing stage
constexpr uint32_t PACK_CHUNKS_PER_WARP = 2;

template <bool RANDK>
__global__ void __launch_bounds__(BT, 4) mid_kernel(const MidArgs a) {
    __shared__ uint32_t sh_scan[33];
    __shared__ uint32_t sh_small[8];              // unit id, prefix, select scratch
    __shared__ uint32_t sh_w[BT / 32];
    __shared__ uint32_t sh_cnt[2 * 8 * GPW];
    __shared__ uint32_t sh_flag[4];
    __shared__ int sh_abort;
    // One pool of dynamic shared memory (MID_POOL_BYTES).  Its first part is the unit table (four
    // arrays) / the candidate-count sums of the order stage, then 8 KB of stage scratch (fallback
    // bins / radix bins / exponent sums / UnitSh); the closing stage takes all of it for its warps'
    // buffers.
    extern __shared__ __align__(128) unsigned char sh_pool[];
    uint32_t* sh_tab = reinterpret_cast<uint32_t*>(sh_pool);
    unsigned char* sh_big = sh_pool + (ORDER_ITEMS_MAX + 8) * sizeof(uint32_t);
    static_assert(MID_SCRATCH_BYTES <= MID_POOL_BYTES, "the stages' scratch must fit the pool");
    static_assert(4 * UT_MAX + 5 <= ORDER_ITEMS_MAX + 8, "the unit table (four arrays of up to UT_MAX + 1 entries) must fit");
    static_assert(sizeof(UnitSh) <= FB_BINS * 4, "the unit stage's scratch must fit");
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
    // a barrier that gives up ends the stages; the block still takes part in the closing count below
#define QS_BARRIER() if (!grid_barrier(P, target, &sh_abort)) break

    do {
    if (a.do_pack) {
        // the records are built with OR: start from zero words (a later barrier precedes their use)
        for (int w = 0; w < act.n; ++w) {
            uint32_t* row = a.wire + (size_t)act.r[w] * a.stride;
            for (long long i = (long long)blockIdx.x * BT + threadIdx.x; i < a.wire_words; i += (long long)gridDim.x * BT) row[i] = 0u;
        }
    }
    Tab tab;
    const bool fused = a.do_compress && a.do_pack && a.do_decode;   // whole round: the master update is part of the closing stage
    const bool merge = fused && qz_early(P.qz);                     // level-1 quantizers: no quantize stage of its own
    bool warp_pack = false;                                          // the records are written in the closing stage's shadow
    if (a.do_compress) {
        const bool even = P.nsup * (uint32_t)act.n <= P.order_sups_max;
        if (even) stage_order_even<RANDK>(P, act, 0u, bins, sh_tab, sh_scan);
        else stage_order<RANDK>(P, act, 0u, bins);
        QS_BARRIER();
        uint32_t missed = 0;
        if (!table_step(P, act, sh_tab, sh_scan, sh_flag, &tab, &missed, target, &sh_abort)) break;
        if (missed) {                              // the same value in every block
            stage_fb_hist<RANDK>(P, act, missed, bins);
            QS_BARRIER();
            stage_fb_guess(P, act, missed, sh_scan, &sh_small[0]);
            QS_BARRIER();
            stage_reflag<RANDK>(P, act, missed, sh_cnt);
            QS_BARRIER();
            if (even) stage_order_even<RANDK>(P, act, missed, bins, sh_tab, sh_scan);
            else stage_order<RANDK>(P, act, missed, bins);
            QS_BARRIER();
            uint32_t again = 0;
            if (!table_step(P, act, sh_tab, sh_scan, sh_flag, &tab, &again, target, &sh_abort)) break;
            if (again) set_status(P, QS_STATE);    // the exact pass cannot miss
            if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd((unsigned long long*)&P.stats[0], (unsigned long long)__popc(missed));
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            unsigned long long cands = 0;
            for (int w = 0; w < act.n; ++w) cands += P.seg_start[(size_t)act.r[w] * (P.nseg + 1) + P.nseg];
            atomicAdd((unsigned long long*)&P.stats[1], cands);
        }
        warp_pack = merge && tab.fast && !P.block_pack && tab.total_chunks <= PACK_CHUNKS_PER_WARP * PACK_WARPS * gridDim.x;
        if (warp_pack) publish_table(P, tab);
        // the candidate counts have been consumed: clear them for the next dense pass
        for (uint32_t i = blockIdx.x * BT + threadIdx.x; i < (uint32_t)P.R * P.nblk; i += gridDim.x * BT) P.blk_count[i] = 0;
        for (uint32_t i = blockIdx.x * BT + threadIdx.x; i < (uint32_t)P.R * P.nsup; i += gridDim.x * BT) P.sup_count[i] = 0;
        // select: the first radix level of the long units, and the short units whole, block by block
        if (tab.total_long) stage_hist<RANDK>(P, tab, 1, bins, &sh_small[0], &sh_small[1], &sh_small[2], sh_w);
        __syncthreads();                           // the scratch changes hands
        if (tab.any_short) stage_unit<RANDK>(P, tab, act, merge, *reinterpret_cast<UnitSh*>(sh_big), sh_w);
        QS_BARRIER();
        if (tab.total_long) {
            bool gave_up = false;
            for (int level = 2; level < 4; ++level) {          // (the last level ends with each unit's threshold and tie cut)
                stage_hist<RANDK>(P, tab, level, bins, &sh_small[0], &sh_small[1], &sh_small[2], sh_w);
                if (!grid_barrier(P, target, &sh_abort)) { gave_up = true; break; }
            }
            if (gave_up) break;
            if (P.fail[0]) {                       // some long list has more equal keys than slots (same in every block)
                stage_tie_count<RANDK>(P, tab, &sh_small[0], sh_w);
                QS_BARRIER();
                stage_tie_find<RANDK>(P, tab, sh_scan, &sh_small[2], sh_w);
                QS_BARRIER();
            }
            stage_norm_accum<RANDK>(P, tab, merge, reinterpret_cast<uint32_t(*)[4]>(sh_big), &sh_small[0], sh_w, sh_cnt);
            QS_BARRIER();
        }
    } else if (a.do_pack) {
        uint32_t unused = 0;
        if (!table_step(P, act, sh_tab, sh_scan, sh_flag, &tab, &unused, target, &sh_abort)) break;
        QS_BARRIER();                              // the zeroed records
    }
    // Thresholds, tie cuts and norms are known.
    if (a.do_compress) {
        if (!merge) {
            stage_quant<RANDK>(P, tab, &sh_small[0], sh_w);
            QS_BARRIER();
        }
        if (!tab.fast) {
            stage_chunk_scan(P, tab, act, sh_scan);
            QS_BARRIER();
        }
    }
    if (a.do_pack && !warp_pack) {
        if (!tab.fast) stage_pack_dir(P, act, a.wire, a.stride, a.bits_out);
        stage_pack<RANDK>(P, tab, merge, a.wire, a.stride, a.bits_out, &sh_small[0], sh_scan);
    }
    if (fused) {
        const uint32_t pack_chunks = warp_pack ? tab.total_chunks : 0u;
        __syncthreads();                           // the unit table and the scratch change hands: the closing stage's buffers now
        if (a.aligned) stage_update_broadcast<RANDK>(P, act, *reinterpret_cast<BcBlock*>(sh_pool), merge, pack_chunks, a.wire, a.stride, a.bits_out);
        else stage_update_broadcast_plain<RANDK>(P, act, *reinterpret_cast<BcBlock*>(sh_pool), merge, pack_chunks, a.wire, a.stride, a.bits_out);
    } else if (a.do_decode) {
        if (a.do_pack) QS_BARRIER();
        if (P.nseg > 1) {
            stage_dec_prep(P, act, a.wire, a.stride, sh_scan);
            QS_BARRIER();
        }
        stage_dec_mark(P, act, a.wire, a.stride);
        QS_BARRIER();
        stage_dec_apply(P, act, a.wire, a.stride);
    }
    } while (0);
#undef QS_BARRIER
    // the last block to leave resets the barrier for the next launch
    __syncthreads();
    if (P.trace && threadIdx.x == 0) {             // when block 0 was done, and when the last block was
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (blockIdx.x == 0) P.trace[TRACE_SLOTS - 2] = t;
        atomicMax(P.trace + TRACE_SLOTS - 1, t);
    }
    if (threadIdx.x == 0) {
        if (atomicAdd(P.bar + 1, 1u) == gridDim.x - 1) {
            P.bar[0] = 0;
            P.bar[1] = 0;
            P.bar[2] = 0;                            // tile tickets of the closing stage
            P.bar[3] = 0;                            // tile tickets of the next dense pass
            P.bar[4] = 0;                            // unit tickets
            P.bar[6] = 0;                            // chunk tickets of the packing warps
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
        if (norm) norm[u] = P.qz == QS_MINMAX ? order_float(P.units[u].emax) : P.units[u].norm;
        if (n) n[u] = P.units[u].n;
    }
}

// ------------------------------------------------------------------ launchers
int mid_blocks_per_sm(bool randk) {
    int per_sm = 0;
    cudaError_t e = randk ? cudaFuncSetAttribute(mid_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MID_POOL_BYTES)
                          : cudaFuncSetAttribute(mid_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MID_POOL_BYTES);
    if (e != cudaSuccess) return 0;
    e = randk ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mid_kernel<true>, BT, MID_POOL_BYTES)
              : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mid_kernel<false>, BT, MID_POOL_BYTES);
    return e == cudaSuccess ? per_sm : 0;
}

cudaError_t launch_mid(const Plan& P, const Active& act, int do_compress, int do_pack, int do_decode,
                       int do_broadcast, int aligned, uint32_t* wire, long long stride, long long wire_words,
                       long long* bits_out, int grid, cudaStream_t st) {
    MidArgs a;
    a.P = P; a.act = act;
    a.do_compress = do_compress; a.do_pack = do_pack; a.do_decode = do_decode;
    a.do_broadcast = do_broadcast; a.aligned = aligned;
    a.wire = wire; a.stride = stride; a.wire_words = wire_words; a.bits_out = bits_out;
    void* params[] = {&a};
    const void* fn = P.sp == QS_RANDK ? (const void*)mid_kernel<true> : (const void*)mid_kernel<false>;
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(BT), params, MID_POOL_BYTES, st);
}

void launch_export(const Plan& P, long long* sel_idx, int* level, uint8_t* sign, float* norm, long long* n,
                   int sms, cudaStream_t st) {
    export_kernel<<<sms * 4, 256, 0, st>>>(P, sel_idx, level, sign, norm, n);
}

}  // namespace qs
