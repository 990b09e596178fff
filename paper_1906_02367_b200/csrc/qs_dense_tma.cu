// Dense pass with the bulk-copy engine (TMA) feeding shared memory: the 16-byte-aligned fast path.
//
// A block walks tiles of 2048 coordinates (two 128-coordinate groups per warp) and, for every
// tile, the active workers in turn.  One thread keeps a ring of (xw, mem) tile pairs filling
// with cp.async.bulk loads several items ahead; each arrival is announced on an mbarrier.  The
// eight warps read their quads from shared memory, form u = mem + (x - xw), overwrite the mem
// tile in place, vote the candidate flags, and the finished tile goes back to global memory as
// one bulk store while the tile's few candidates (index, value) are written out in order.  Loads and stores never pass through registers of the
// computing warps, so the depth of the ring, not the occupancy, sets the bytes in flight.
//
// Every wait is bounded: a barrier that does not complete records QS_TIMEOUT, the block waits
// for its own copies in flight and leaves.
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
constexpr int STAGES = QS_TMA_STAGES;      // (xw, mem) tile pairs in the ring
#ifndef QS_TMA_XSLOTS
#define QS_TMA_XSLOTS 2
#endif
constexpr int XSLOTS = QS_TMA_XSLOTS;      // x tiles in their ring

template <bool ANCH>
struct TmaSmem {
    float stage[STAGES][ANCH ? 3 : 2][TILE];   // [0] xw tile, [1] mem tile (overwritten with u), [2] anchor tile
    float xs[ANCH ? 1 : XSLOTS][ANCH ? 4 : TILE];   // x tiles (not read when every worker has its own anchor)
    uint64_t full[STAGES];
    uint64_t xfull[XSLOTS];
    uint32_t cnt[2][8 * GPW];              // candidates per group of the current tile (double-buffered)
    int abort_flag;
};

// Rows 16-byte aligned.  ANCH: Algorithm 2, worker r's reference point is anchors_r (a third tile per
// item) instead of x.
template <bool RANDK, bool ANCH>
__global__ void __launch_bounds__(256) pass_a_tma_kernel(const Plan P, const Active act, const int prefetch) {
    extern __shared__ __align__(128) unsigned char sh_raw[];
    TmaSmem<ANCH>& S = *reinterpret_cast<TmaSmem<ANCH>*>(sh_raw);
    uint32_t* tab = reinterpret_cast<uint32_t*>(sh_raw + sizeof(TmaSmem<ANCH>));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ntiles = (P.d + TILE - 1) / TILE;
    const int nact = act.n;
    // thresholds of all workers, then segment offsets
    const uint32_t ng = (uint32_t)P.R * P.nseg;
    for (uint32_t i = threadIdx.x; i < ng; i += 256) tab[i] = P.guess[i];
    for (uint32_t i = threadIdx.x; i <= (uint32_t)P.nseg; i += 256) tab[ng + i] = P.seg_off[i];
    const uint32_t* seg_off = tab + ng;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&S.full[s], 1);
        for (int s = 0; s < XSLOTS; ++s) mbar_init(&S.xfull[s], 1);
        S.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // items of this block: tile iteration `it` (tile = blockIdx.x + it * gridDim.x) x active worker
    const uint32_t my_tiles = blockIdx.x < ntiles ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const uint64_t nitems = (uint64_t)my_tiles * nact;

    auto issue = [&](uint64_t j) {           // thread 0: start the loads of item j
        const uint32_t it = (uint32_t)(j / nact);
        const int w = (int)(j % nact);
        const uint32_t tile = blockIdx.x + it * gridDim.x;
        const uint32_t e0 = tile * TILE;
        const uint32_t bytes = (P.d - e0 < TILE ? P.d - e0 : TILE) * 4u;
        const int s = (int)(j % STAGES);
        const size_t row = (size_t)act.r[w] * P.d + e0;
        if (!ANCH && w == 0) {
            const int xsl = (int)(it % XSLOTS);
            mbar_expect(&S.xfull[xsl], bytes);
            bulk_load(S.xs[xsl], P.x + e0, bytes, &S.xfull[xsl]);
        }
        mbar_expect(&S.full[s], (ANCH ? 3u : 2u) * bytes);
        bulk_load(S.stage[s][0], P.xw + row, bytes, &S.full[s]);
        bulk_load(S.stage[s][1], P.mem + row, bytes, &S.full[s]);
        if (ANCH) bulk_load(S.stage[s][ANCH ? 2 : 0], P.anchors + row, bytes, &S.full[s]);
    };

    if (threadIdx.x == 0)
        for (uint64_t j = 0; j < (uint64_t)prefetch && j < nitems; ++j) issue(j);

    bool bad = false;
    int sg[GP][4] = {};                      // segments of this lane's quads, refreshed once per tile
    uint64_t j = 0;
    for (; j < nitems; ++j) {
        const uint32_t it = (uint32_t)(j / nact);
        const int w = (int)(j % nact);
        const int r = act.r[w];
        const uint32_t tile = blockIdx.x + it * gridDim.x;
        const int s = (int)(j % STAGES), xsl = (int)(it % XSLOTS);
        if (threadIdx.x == 0 && j + prefetch < nitems) {
            bulk_wait_read<1>();             // the ring slot about to be refilled has been read by its store
            issue(j + prefetch);
        }
        bool ok = mbar_wait(&S.full[s], (uint32_t)((j / STAGES) & 1));
        if (!ANCH && w == 0) ok = ok && mbar_wait(&S.xfull[xsl], (uint32_t)((it / XSLOTS) & 1));
        if (!ok) S.abort_flag = 1;           // seen by everyone at the barrier below

        const uint32_t* gs = tab + (size_t)r * P.nseg;
        uint32_t bal[GPW][4];
        float uu[GPW][4];
#pragma unroll
        for (int k = 0; k < GP; ++k) {
            const uint32_t g = tile * (TILE / GROUP) + warp * GP + k;
            const uint32_t q = (warp * GP + k) * GROUP + lane * 4;   // offset inside the tile
            const uint32_t e0 = tile * TILE + q;
            if (w == 0 && P.nseg > 1) {
                int sq = g < P.ngroups ? (int)P.grp_seg[g] : 0;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    while (sq + 1 < P.nseg && e0 + jj >= seg_off[sq + 1]) ++sq;
                    sg[k][jj] = sq;
                }
            }
            const float4 xq = ANCH ? *reinterpret_cast<const float4*>(&S.stage[s][ANCH ? 2 : 0][q])
                                   : *reinterpret_cast<const float4*>(&S.xs[ANCH ? 0 : xsl][ANCH ? 0 : q]);
            const float4 wq = *reinterpret_cast<const float4*>(&S.stage[s][0][q]);
            const float4 mq = *reinterpret_cast<const float4*>(&S.stage[s][1][q]);
            uu[k][0] = mq.x + (xq.x - wq.x);
            uu[k][1] = mq.y + (xq.y - wq.y);
            uu[k][2] = mq.z + (xq.z - wq.z);
            uu[k][3] = mq.w + (xq.w - wq.w);
            *reinterpret_cast<float4*>(&S.stage[s][1][q]) = make_float4(uu[k][0], uu[k][1], uu[k][2], uu[k][3]);
            const bool in = e0 < P.d;                            // d is a multiple of 4: whole quads
            uint32_t sk[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                sk[jj] = topk_key(uu[k][jj]);
                if (in) bad |= sk[jj] >= 0xFF000000u;
            }
            if (RANDK) {
                const uint4 h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
                sk[0] = ~h.x; sk[1] = ~h.y; sk[2] = ~h.z; sk[3] = ~h.w;
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
                bal[k][jj] = __ballot_sync(0xffffffffu, in && sk[jj] >= gs[sg[k][jj]]);
        }
        tile_counts(S.cnt[j & 1], warp, lane, bal);
        fence_async_smem();                  // the tile written above must be visible to the bulk store
        __syncthreads();
        if (S.abort_flag) break;
        if (threadIdx.x == 0) {
            const uint32_t t0 = tile * TILE;
            const uint32_t bytes = (P.d - t0 < TILE ? P.d - t0 : TILE) * 4u;
            bulk_store(P.mem + (size_t)r * P.d + t0, S.stage[s][1], bytes);
            bulk_commit();
        }
        tile_write(P, r, tile, S.cnt[j & 1], warp, lane, bal, uu);
    }
    if (threadIdx.x == 0) {
        if (S.abort_flag) {
            // give the loads already issued a bounded chance to land before the block leaves
            for (uint64_t jj = j; jj < nitems && jj < j + (uint64_t)prefetch; ++jj)
                mbar_wait(&S.full[jj % STAGES], (uint32_t)((jj / STAGES) & 1));
            set_status(P, QS_TIMEOUT);
        }
        bulk_wait_all();                     // nothing of this block may still be reading shared memory
    }
    if (bad) set_status(P, QS_NONFINITE);
}

size_t pass_a_tma_smem(const Plan& P) {
    return (P.anchors ? sizeof(TmaSmem<true>) : sizeof(TmaSmem<false>)) + ((size_t)P.R * P.nseg + P.nseg + 1) * 4;
}

bool pass_a_tma_usable(const Plan& P, bool aligned) { return aligned && pass_a_tma_smem(P) <= 100 * 1024; }

template <bool RANDK, bool ANCH>
static cudaError_t tma_launch(const Plan& P, const Active& act, int sms, size_t smem, int prefetch, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(pass_a_tma_kernel<RANDK, ANCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // tiles are dealt to blocks by stride, so the grid holds only blocks that are resident together
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pass_a_tma_kernel<RANDK, ANCH>, 256, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    if (per_sm > QS_TMA_PER_SM) per_sm = QS_TMA_PER_SM;
    const uint32_t ntiles = (P.d + TILE - 1) / TILE;
    const uint32_t cap = (uint32_t)sms * (uint32_t)per_sm;
    const int grid = (int)(ntiles < cap ? ntiles : cap);
    pass_a_tma_kernel<RANDK, ANCH><<<grid, 256, smem, st>>>(P, act, prefetch);
    return cudaGetLastError();
}

cudaError_t launch_pass_a_tma(const Plan& P, const Active& act, int sms, cudaStream_t st) {
    const size_t smem = pass_a_tma_smem(P);
    int prefetch = STAGES - 2;
    if (!P.anchors && prefetch > (XSLOTS - 1) * act.n) prefetch = (XSLOTS - 1) * act.n;   // an x slot is refilled only after its tile is done
    const bool rk = P.sp == QS_RANDK;
    if (P.anchors) return rk ? tma_launch<true, true>(P, act, sms, smem, prefetch, st) : tma_launch<false, true>(P, act, sms, smem, prefetch, st);
    return rk ? tma_launch<true, false>(P, act, sms, smem, prefetch, st) : tma_launch<false, false>(P, act, sms, smem, prefetch, st);
}

}  // namespace qs
