// Dense pass with the bulk-copy engine (TMA) feeding shared memory: the 16-byte-aligned fast path.
//
// A block walks tiles of 2048 coordinates (two 128-coordinate groups per warp) and, for every
// tile, the active workers in turn.  One thread keeps a ring of (xw, mem) tile pairs filling
// with cp.async.bulk loads several items ahead; each arrival is announced on an mbarrier.  The
// eight warps read their quads from shared memory, form u = mem + (x - xw), overwrite the mem
// tile in place, vote the candidate flags, and the finished tile goes back to global memory as
// one bulk store while the tile's few candidates (index, value) are written out in order.  Loads
// and stores never pass through registers of the computing warps, so the depth of the ring, not
// the occupancy, sets the bytes in flight.
//
// Variants (template flags): ANCH, Algorithm 2: the worker's anchor tile rides in the ring in
// place of the shared x tile.  STEP, the local step that precedes the synchronisation taken here:
// the gradient tile (STEP >= 1) and the velocity tile (STEP == 2, updated and stored back) ride
// in the ring too, and u is formed from xw - eta * (grad or velocity) without writing it.
//
// Every wait is bounded: a barrier that does not complete records QS_TIMEOUT, the block waits
// for its own copies in flight and leaves.
#include <cstdlib>

#include "qs_bulk.cuh"
#include "qs_kernels.h"

namespace qs {

#ifndef QS_TMA_STAGES
#define QS_TMA_STAGES 3
#endif
#ifndef QS_TMA_PER_SM
#define QS_TMA_PER_SM 3
#endif
constexpr int GP = GPW;                    // groups of 128 coordinates per warp and tile
constexpr int TILE = STILE;                // coordinates per tile: 8 warps x GP groups
constexpr int STAGES = QS_TMA_STAGES;      // items in the ring (2 when an item has five tiles)
#ifndef QS_TMA_XSLOTS
#define QS_TMA_XSLOTS 2
#endif
constexpr int XSLOTS = QS_TMA_XSLOTS;      // x tiles in their ring

constexpr int MAX_STAGES = STAGES > 4 ? STAGES : 4;

struct TmaCtl {
    alignas(16) uint32_t gseg[4][STILE / GROUP];   // segment of each group's first coordinate, for the last tile iterations
    uint64_t full[MAX_STAGES];
    uint64_t xfull[XSLOTS];
    uint32_t cnt[2][8 * GPW];              // candidates per group of the current tile (double-buffered)
    uint32_t tiles[4];                     // tile of each of the last tile iterations (>= ntiles: no tile is left)
    int abort_flag;
};

__host__ __device__ constexpr int tiles_per_item(bool anch, int step) { return 2 + (anch ? 1 : 0) + step; }

// shared memory: ring [nst][NT][TILE] floats, x ring [XSLOTS][TILE] (no anchors), TmaCtl, thresholds + offsets
__host__ __device__ inline size_t tma_ring_bytes(bool anch, int step, int nst) {
    return ((size_t)nst * tiles_per_item(anch, step) + (anch ? 0 : XSLOTS)) * TILE * sizeof(float);
}

// Rows 16-byte aligned.  Tiles of an item inside its ring slot: 0 xw, 1 mem (overwritten with u),
// then the anchor (ANCH), the gradient (STEP >= 1), the velocity (STEP == 2, overwritten).
template <bool RANDK, bool ANCH, int STEP>
__global__ void __launch_bounds__(256) pass_a_tma_kernel(const Plan P, const Active act, const StepArgs sa,
                                                         const int nst, const int prefetch) {
    constexpr int NT = tiles_per_item(ANCH, STEP);
    constexpr int T_ANCH = 2, T_GRAD = 2 + (ANCH ? 1 : 0), T_VEL = T_GRAD + 1;
    extern __shared__ __align__(128) unsigned char sh_raw[];
    float* ring = reinterpret_cast<float*>(sh_raw);
    float* xs = ring + (size_t)nst * NT * TILE;
    TmaCtl& S = *reinterpret_cast<TmaCtl*>(sh_raw + tma_ring_bytes(ANCH, STEP, nst));
    uint32_t* tab = reinterpret_cast<uint32_t*>(sh_raw + tma_ring_bytes(ANCH, STEP, nst) + sizeof(TmaCtl));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ntiles = (P.d + TILE - 1) / TILE;
    const int nact = act.n;
    // thresholds of all workers, then segment offsets
    const uint32_t ng = (uint32_t)P.R * P.nseg;
    for (uint32_t i = threadIdx.x; i < ng; i += 256) tab[i] = P.guess[i];
    for (uint32_t i = threadIdx.x; i <= (uint32_t)P.nseg; i += 256) tab[ng + i] = P.seg_off[i];
    const uint32_t* seg_off = tab + ng;
    if (threadIdx.x == 0) {
        for (int s = 0; s < nst; ++s) mbar_init(&S.full[s], 1);
        for (int s = 0; s < XSLOTS; ++s) mbar_init(&S.xfull[s], 1);
        S.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Items of this block: tile iteration `it` x active worker.  Tiles are handed out by a ticket
    // counter (the next ticket is drawn one tile ahead, off the path), so that every block works
    // until the pass is over whatever its share of the memory system was; a ticket beyond the
    // last tile is passed on to the consumers as the end mark.
    auto slot = [&](int s, int t) { return ring + ((size_t)s * NT + t) * TILE; };

    // running position of the producer (the item whose loads start next) and of the consumers: tile
    // iteration, worker, ring slot, and for the consumers the slot's phase; no divisions in the loop
    uint32_t p_it = 0, p_j = 0, p_tile = 0, ticket = 0;
    int p_w = 0, p_s = 0;
    bool more = true;
    if (threadIdx.x == 0) ticket = atomicAdd(P.bar + 3, 1u);
    auto issue = [&]() {                     // thread 0: start the loads of the producer's item
        const uint32_t it = p_it;
        const int w = p_w;
        if (w == 0) {                        // a new tile
            p_tile = ticket;
            S.tiles[it & 3u] = p_tile;
            if (p_tile >= ntiles) {          // the end mark travels on the item's barrier, with no bytes
                more = false;
                mbar_expect(&S.full[p_s], 0u);
                ++p_j;
                return;
            }
            ticket = atomicAdd(P.bar + 3, 1u);
        }
        const uint32_t tile = p_tile;
        const uint32_t e0 = tile * TILE;
        const uint32_t bytes = (P.d - e0 < TILE ? P.d - e0 : TILE) * 4u;
        const int s = p_s;
        const size_t row = (size_t)act.r[w] * P.d + e0;
        if (!ANCH && w == 0) {
            const int xsl = (int)(it % XSLOTS);
            mbar_expect(&S.xfull[xsl], bytes);
            bulk_load(xs + (size_t)xsl * TILE, P.x + e0, bytes, &S.xfull[xsl]);
        }
        // several segments: the tile's sixteen group-to-segment entries come with its first item
        const bool segs = w == 0 && P.nseg > 1;
        mbar_expect(&S.full[s], (uint32_t)NT * bytes + (segs ? (uint32_t)sizeof(S.gseg[0]) : 0u));
        if (segs) bulk_load(S.gseg[it & 3u], P.grp_seg + (size_t)tile * (STILE / GROUP), (uint32_t)sizeof(S.gseg[0]), &S.full[s]);
        bulk_load(slot(s, 0), P.xw + row, bytes, &S.full[s]);
        bulk_load(slot(s, 1), P.mem + row, bytes, &S.full[s]);
        if (ANCH) bulk_load(slot(s, T_ANCH), P.anchors + row, bytes, &S.full[s]);
        if (STEP >= 1) bulk_load(slot(s, T_GRAD), sa.grad + row, bytes, &S.full[s]);
        if (STEP == 2) bulk_load(slot(s, T_VEL), sa.vel + row, bytes, &S.full[s]);
        ++p_j;
        if (++p_w == nact) { p_w = 0; ++p_it; }
        if (++p_s == nst) p_s = 0;
    };

    if (threadIdx.x == 0)
        while (p_j < (uint32_t)prefetch && more) issue();
    // stores (one group per item) that may still be reading their slot when the slot `prefetch`
    // items ahead is refilled: that slot was last used nst - prefetch items before the current one
    const int pending_ok = nst - prefetch - 1;

    bool bad = false;
    int sq0[GP] = {};                        // segment of each group's first coordinate, refreshed once per tile
    bool uni[GP];                            // the whole group lies in that segment (the rule, segments being long)
#pragma unroll
    for (int k = 0; k < GP; ++k) uni[k] = true;
    uint32_t j = 0, it = 0, ph = 0, tile = 0;
    int w = 0, s = 0;
    for (;; ++j) {
        const int r = act.r[w];
        const int xsl = (int)(it % XSLOTS);
        if (threadIdx.x == 0 && more) {
            if (pending_ok >= 2) bulk_wait_read<2>();
            else if (pending_ok == 1) bulk_wait_read<1>();
            else bulk_wait_read<0>();
            issue();
        }
        // Rand_k: the keys do not depend on the data, only on (worker, coordinate): their ten Philox
        // rounds are worked out before the wait for the item's copies, in its shadow.  (The item's
        // tile was noted by the producer at least one iteration, and block barrier, ago.)
        uint4 hq[GP];
        uint32_t tile_pre = tile;
        if (RANDK) {
            if (w == 0) tile_pre = *reinterpret_cast<volatile uint32_t*>(&S.tiles[it & 3u]);
#pragma unroll
            for (int k = 0; k < GP; ++k)
                hq[k] = philox_quad(P, (uint32_t)r, (tile_pre * TILE + (warp * GP + k) * GROUP + lane * 4) >> 2, 1u);
        }
        bool ok = mbar_wait(&S.full[s], ph);
        if (w == 0 && ok) tile = S.tiles[it & 3u];       // written by the producer before it armed the barrier
        if (!ANCH && w == 0 && tile < ntiles) ok = ok && mbar_wait(&S.xfull[xsl], (uint32_t)((it / XSLOTS) & 1));   // no x tile comes with the end mark
        if (!ok) S.abort_flag = 1;           // seen by everyone at the barrier below

        const uint32_t* gs = tab + (size_t)r * P.nseg;
        const float* ref = ANCH ? slot(s, T_ANCH) : xs + (size_t)xsl * TILE;
        uint32_t bal[GPW][4];
        float uu[GPW][4];
        // all shared-memory reads of the item first: the stores below must not order them
        float4 xq_[GP], wq_[GP], mq_[GP], dq_[GP], vq_[GP];
#pragma unroll
        for (int k = 0; k < GP; ++k) {
            const uint32_t q = (warp * GP + k) * GROUP + lane * 4;   // offset inside the tile
            xq_[k] = *reinterpret_cast<const float4*>(ref + q);
            wq_[k] = *reinterpret_cast<const float4*>(slot(s, 0) + q);
            mq_[k] = *reinterpret_cast<const float4*>(slot(s, 1) + q);
            if (STEP >= 1) dq_[k] = *reinterpret_cast<const float4*>(slot(s, T_GRAD) + q);
            if (STEP == 2) vq_[k] = *reinterpret_cast<const float4*>(slot(s, STEP == 2 ? T_VEL : 0) + q);
        }
#pragma unroll
        for (int k = 0; k < GP; ++k) {
            const uint32_t g = tile * (TILE / GROUP) + warp * GP + k;
            const uint32_t q = (warp * GP + k) * GROUP + lane * 4;
            const uint32_t e0 = tile * TILE + q;
            if (w == 0 && P.nseg > 1 && tile < ntiles) {     // (the end mark brings no entries: nothing to look up)
                // segment of the group's first coordinate: the table's entries for this tile came in
                // with the tile's first item (a load from global memory here would stall the tile
                // behind the copies in flight)
                const uint32_t ent = S.gseg[it & 3u][warp * GP + k];
                const int lo = (int)(ent < (uint32_t)P.nseg ? ent : (uint32_t)P.nseg - 1u);
                const uint32_t first = g * (uint32_t)GROUP;
                sq0[k] = lo;
                uni[k] = lo + 1 >= P.nseg || seg_off[lo + 1] >= first + (uint32_t)GROUP;
            }
            const float4 xq = xq_[k], mq = mq_[k];
            float4 wq = wq_[k];
            if (STEP >= 1) {                 // the local step: every product and sum rounded on its own
                float4 dq = dq_[k];
                if (STEP == 2) {
                    const float4 vq = vq_[k];
                    dq.x = sa.mu * vq.x + dq.x; dq.y = sa.mu * vq.y + dq.y;
                    dq.z = sa.mu * vq.z + dq.z; dq.w = sa.mu * vq.w + dq.w;
                    *reinterpret_cast<float4*>(slot(s, STEP == 2 ? T_VEL : 0) + q) = dq;
                }
                wq.x = wq.x - sa.eta * dq.x; wq.y = wq.y - sa.eta * dq.y;
                wq.z = wq.z - sa.eta * dq.z; wq.w = wq.w - sa.eta * dq.w;
            }
            uu[k][0] = mq.x + (xq.x - wq.x);
            uu[k][1] = mq.y + (xq.y - wq.y);
            uu[k][2] = mq.z + (xq.z - wq.z);
            uu[k][3] = mq.w + (xq.w - wq.w);
            *reinterpret_cast<float4*>(slot(s, 1) + q) = make_float4(uu[k][0], uu[k][1], uu[k][2], uu[k][3]);
            const bool in = e0 < P.d;                            // d is a multiple of 4: whole quads
            uint32_t sk[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                sk[jj] = topk_key(uu[k][jj]);
                if (in) bad |= sk[jj] >= 0xFF000000u;
            }
            if (RANDK) {
                const uint4 h = tile == tile_pre ? hq[k] : philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
                sk[0] = ~h.x; sk[1] = ~h.y; sk[2] = ~h.z; sk[3] = ~h.w;
            }
            if (uni[k]) {                    // one threshold for the whole group (the same branch in every lane)
                const uint32_t thr = gs[sq0[k]];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) bal[k][jj] = __ballot_sync(0xffffffffu, in && sk[jj] >= thr);
            } else {                         // a segment border inside the group: per coordinate
                int sq = sq0[k];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    while (sq + 1 < P.nseg && e0 + jj >= seg_off[sq + 1]) ++sq;
                    bal[k][jj] = __ballot_sync(0xffffffffu, in && sk[jj] >= gs[sq]);
                }
            }
        }
        tile_counts(S.cnt[j & 1], warp, lane, bal);
        fence_async_smem();                  // the tiles written above must be visible to the bulk stores
        __syncthreads();
        if (S.abort_flag) break;
        if (tile >= ntiles) break;           // the end mark: nothing was loaded for this item (every thread read the same mark)
        if (threadIdx.x == 0) {
            const uint32_t t0 = tile * TILE;
            const uint32_t bytes = (P.d - t0 < TILE ? P.d - t0 : TILE) * 4u;
            bulk_store(P.mem + (size_t)r * P.d + t0, slot(s, 1), bytes);
            if (STEP == 2) bulk_store(sa.vel + (size_t)r * P.d + t0, slot(s, STEP == 2 ? T_VEL : 0), bytes);
            bulk_commit();
        }
        tile_write(P, r, tile, S.cnt[j & 1], warp, lane, bal, uu);
        if (++w == nact) { w = 0; ++it; }
        if (++s == nst) { s = 0; ph ^= 1u; }
    }
    if (threadIdx.x == 0) {
        if (S.abort_flag) {
            // give the loads already issued a bounded chance to land before the block leaves
            for (uint32_t jj = j; jj < p_j; ++jj) {
                mbar_wait(&S.full[s], ph);
                if (++s == nst) { s = 0; ph ^= 1u; }
            }
            set_status(P, QS_TIMEOUT);
        }
        bulk_wait_all();                     // nothing of this block may still be reading shared memory
    }
    if (bad) set_status(P, QS_NONFINITE);
}

// items in the ring: QSPARSE_TMA_DEPTH (2..MAX_STAGES) overrides the default for tuning
static int ring_depth(bool anch, int step) {
    static const int forced = [] {
        const char* e = getenv("QSPARSE_TMA_DEPTH");
        const int v = e ? atoi(e) : 0;
        return v >= 2 && v <= MAX_STAGES ? v : 0;
    }();
    if (forced) return forced;
    // resident blocks beat ring depth: the shallow ring wherever it lets one more block share the SM
    auto blocks = [&](int nst) {
        const size_t per_block = tma_ring_bytes(anch, step, nst) + 2048;
        const size_t fit = (size_t)227 * 1024 / per_block;
        return fit < (size_t)QS_TMA_PER_SM ? (int)fit : QS_TMA_PER_SM;
    };
    return blocks(STAGES) >= blocks(2) ? STAGES : 2;
}

size_t pass_a_tma_smem(const Plan& P, int step) {
    const bool anch = P.anchors != nullptr;
    return tma_ring_bytes(anch, step, ring_depth(anch, step)) + sizeof(TmaCtl) + ((size_t)P.R * P.nseg + P.nseg + 1) * 4;
}

bool pass_a_tma_usable(const Plan& P, bool aligned, int step) {
    return aligned && pass_a_tma_smem(P, step) <= 200 * 1024;
}

template <bool RANDK, bool ANCH, int STEP>
static cudaError_t tma_launch(const Plan& P, const Active& act, const StepArgs& sa, int sms, cudaStream_t st) {
    const size_t smem = pass_a_tma_smem(P, STEP);
    const int nst = ring_depth(ANCH, STEP);
    int prefetch = nst >= 3 ? nst - 2 : 1;
    if (!ANCH && prefetch > (XSLOTS - 1) * act.n) prefetch = (XSLOTS - 1) * act.n;   // an x slot is refilled only after its tile is done
    cudaError_t e = cudaFuncSetAttribute(pass_a_tma_kernel<RANDK, ANCH, STEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // tiles are dealt to blocks by stride, so the grid holds only blocks that are resident together
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pass_a_tma_kernel<RANDK, ANCH, STEP>, 256, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    if (per_sm > QS_TMA_PER_SM) per_sm = QS_TMA_PER_SM;
    const uint32_t ntiles = (P.d + TILE - 1) / TILE;
    const uint32_t cap = (uint32_t)sms * (uint32_t)per_sm;
    const int grid = (int)(ntiles < cap ? ntiles : cap);
    pass_a_tma_kernel<RANDK, ANCH, STEP><<<grid, 256, smem, st>>>(P, act, sa, nst, prefetch);
    return cudaGetLastError();
}

template <bool RANDK, bool ANCH>
static cudaError_t tma_launch_step(const Plan& P, const Active& act, const StepArgs& sa, int step, int sms, cudaStream_t st) {
    if (step == 2) return tma_launch<RANDK, ANCH, 2>(P, act, sa, sms, st);
    if (step == 1) return tma_launch<RANDK, ANCH, 1>(P, act, sa, sms, st);
    return tma_launch<RANDK, ANCH, 0>(P, act, sa, sms, st);
}

// step: 0 none, 1 plain local step (sa.grad, sa.eta), 2 with momentum (sa.vel, sa.mu too)
cudaError_t launch_pass_a_tma(const Plan& P, const Active& act, const StepArgs& sa, int step, int sms, cudaStream_t st) {
    const bool rk = P.sp == QS_RANDK;
    if (P.anchors) return rk ? tma_launch_step<true, true>(P, act, sa, step, sms, st) : tma_launch_step<false, true>(P, act, sa, step, sms, st);
    return rk ? tma_launch_step<true, false>(P, act, sa, step, sms, st) : tma_launch_step<false, false>(P, act, sa, step, sms, st);
}

}  // namespace qs
