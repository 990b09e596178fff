// Dense passes of the sync round: everything that touches all R x d coordinates.
//
//   pass_a      u = mem + (anchor - xw) written over mem, and the candidates (coordinates whose
//               key passes the predicted threshold) written out per tile, in order
//   broadcast   xw_r <- x,   local_step  xw_r <- xw_r - eta grad_r
//
// One warp owns groups of 128 consecutive coordinates (4 per lane, one 128-bit access per
// array) and loops over the workers with the model quads held in registers, so x is read once
// for all R workers.  This file holds the general path; the aligned synchronous case runs the
// bulk-copy version of the pass.
#include "qs_kernels.h"

namespace qs {

template <bool ALIGNED>
__device__ __forceinline__ void load_quad(const float* __restrict__ row, uint32_t e0, uint32_t d,
                                          float v[4]) {
    if (ALIGNED) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e0 < d) t = __ldcs(reinterpret_cast<const float4*>(row + e0));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (e0 + j < d) ? __ldcs(row + e0 + j) : 0.0f;
    }
}

template <bool ALIGNED>
__device__ __forceinline__ void store_quad(float* __restrict__ row, uint32_t e0, uint32_t d,
                                           const float v[4]) {
    if (ALIGNED) {
        if (e0 < d) __stcs(reinterpret_cast<float4*>(row + e0), make_float4(v[0], v[1], v[2], v[3]));
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (e0 + j < d) __stcs(row + e0 + j, v[j]);
    }
}

constexpr int TAB_MAX = 11 * 1024;   // words of shared memory for the threshold and offset tables

// General dense pass: any alignment, either algorithm (anchors bound or not).  A block handles a
// tile of 2048 coordinates (warp w owns groups 2w and 2w+1) for the active workers in turn:
// plain loads, u = mem + (anchor - xw) written over mem, candidate flags voted per group and the
// tile's candidates written out in order.  mode 1 also writes x into xw_r (and anchors_r).
// Shared memory holds the thresholds of all workers and the segment offsets when they fit.
template <bool ALIGNED, bool RANDK, bool ANCH>
__global__ void __launch_bounds__(256) pass_a_kernel(const Plan P, const Active act, const int mode, const int tab) {
    extern __shared__ uint32_t sh_tab[];
    __shared__ uint32_t sh_cnt[2][8 * GPW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t* guess = P.guess;
    const uint32_t* seg_off = P.seg_off;
    if (tab) {
        const uint32_t ng = (uint32_t)P.R * P.nseg;
        for (uint32_t i = threadIdx.x; i < ng; i += 256) sh_tab[i] = P.guess[i];
        for (uint32_t i = threadIdx.x; i <= (uint32_t)P.nseg; i += 256) sh_tab[ng + i] = P.seg_off[i];
        __syncthreads();
        guess = sh_tab;
        seg_off = sh_tab + ng;
    }
    bool bad = false;
    uint32_t item = 0;
    for (uint32_t tile = blockIdx.x; tile < P.ntile; tile += gridDim.x) {
        int sg[GPW][4] = {};
        float xq[GPW][4];
#pragma unroll
        for (int k = 0; k < GPW; ++k) {
            const uint32_t g = tile * (uint32_t)(STILE / GROUP) + warp * GPW + k;
            const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
            if (P.nseg > 1) {
                int sq = g < P.ngroups ? (int)P.grp_seg[g] : 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    while (sq + 1 < P.nseg && e0 + j >= seg_off[sq + 1]) ++sq;
                    sg[k][j] = sq;
                }
            }
            load_quad<ALIGNED>(P.x, e0, P.d, xq[k]);
        }
        for (int w = 0; w < act.n; ++w, ++item) {
            const int r = act.r[w];
            const size_t row = (size_t)r * P.d;
            const uint32_t* gs = guess + (size_t)r * P.nseg;
            float xw[GPW][4], mm[GPW][4], an[ANCH ? GPW : 1][4];
#pragma unroll
            for (int k = 0; k < GPW; ++k) {
                const uint32_t e0 = (tile * (uint32_t)(STILE / GROUP) + warp * GPW + k) * (uint32_t)GROUP + (uint32_t)lane * 4u;
                load_quad<ALIGNED>(P.xw + row, e0, P.d, xw[k]);
                load_quad<ALIGNED>(P.mem + row, e0, P.d, mm[k]);
                if (ANCH) load_quad<ALIGNED>(P.anchors + row, e0, P.d, an[ANCH ? k : 0]);
            }
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
                    const float anchor = ANCH ? an[ANCH ? k : 0][j] : xq[k][j];
                    const float diff = anchor - xw[k][j];
                    u[k][j] = mm[k][j] + diff;
                    const uint32_t key = topk_key(u[k][j]);
                    const bool in = e0 + j < P.d;
                    if (in) bad |= key >= 0xFF000000u;
                    const uint32_t sk = RANDK ? ~hh[j] : key;
                    bal[k][j] = __ballot_sync(0xffffffffu, in && sk >= gs[sg[k][j]]);
                }
                store_quad<ALIGNED>(P.mem + row, e0, P.d, u[k]);
                if (mode == 1) {
                    store_quad<ALIGNED>(P.xw + row, e0, P.d, xq[k]);
                    if (ANCH) store_quad<ALIGNED>(P.anchors + row, e0, P.d, xq[k]);
                }
            }
            tile_counts(sh_cnt[item & 1], warp, lane, bal);
            __syncthreads();
            tile_write(P, r, tile, sh_cnt[item & 1], warp, lane, bal, u);
        }
    }
    if (bad) set_status(P, QS_NONFINITE);
}

template <bool ALIGNED>
__global__ void __launch_bounds__(256) broadcast_kernel(const Plan P, const Active act) {
    const int lane = threadIdx.x & 31;
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * 8u) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        if (e0 >= P.d) continue;
        float xq[4];
        load_quad<ALIGNED>(P.x, e0, P.d, xq);
        for (int w = 0; w < act.n; ++w) {
            const size_t row = (size_t)act.r[w] * P.d;
            store_quad<ALIGNED>(P.xw + row, e0, P.d, xq);
            if (P.anchors) store_quad<ALIGNED>(P.anchors + row, e0, P.d, xq);
        }
    }
}

template <bool ALIGNED, bool MOMENTUM>
__global__ void __launch_bounds__(256) local_step_kernel(const Plan P, const Active act, const StepArgs sa) {
    const int lane = threadIdx.x & 31;
    const int r = act.r[blockIdx.y];
    const size_t row = (size_t)r * P.d;
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * 8u) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        if (e0 >= P.d) continue;
        float w[4], gr[4], v[4];
        load_quad<ALIGNED>(P.xw + row, e0, P.d, w);
        load_quad<ALIGNED>(sa.grad + row, e0, P.d, gr);
        if (MOMENTUM) {
            load_quad<ALIGNED>(sa.vel + row, e0, P.d, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float carried = sa.mu * v[j];
                gr[j] = carried + gr[j];
            }
            store_quad<ALIGNED>(sa.vel + row, e0, P.d, gr);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float step = sa.eta * gr[j];
            w[j] = w[j] - step;
        }
        store_quad<ALIGNED>(P.xw + row, e0, P.d, w);
    }
}

// ------------------------------------------------------------------ launchers
static inline int dense_grid(const Plan& P, int sms, int per_sm) {
    const uint32_t need = (P.ngroups + 7u) / 8u;
    const uint32_t cap = (uint32_t)(sms * per_sm);
    return (int)(need < cap ? (need ? need : 1u) : cap);
}

template <bool ALIGNED, bool RANDK>
static void pass_a_dispatch(const Plan& P, const Active& act, int mode, int grid, int tab, size_t smem, cudaStream_t st) {
    if (P.anchors) pass_a_kernel<ALIGNED, RANDK, true><<<grid, 256, smem, st>>>(P, act, mode, tab);
    else pass_a_kernel<ALIGNED, RANDK, false><<<grid, 256, smem, st>>>(P, act, mode, tab);
}

void launch_pass_a(const Plan& P, const Active& act, int mode, bool aligned, int sms, cudaStream_t st) {
    const uint32_t cap = (uint32_t)sms * 4u;
    const int grid = (int)(P.ntile < cap ? P.ntile : cap);
    const size_t words = (size_t)P.R * P.nseg + P.nseg + 1;
    const int tab = words <= (size_t)TAB_MAX;
    const size_t smem = tab ? words * 4 : 0;
    const bool rk = P.sp == QS_RANDK;
    if (aligned) {
        if (rk) pass_a_dispatch<true, true>(P, act, mode, grid, tab, smem, st);
        else pass_a_dispatch<true, false>(P, act, mode, grid, tab, smem, st);
    } else {
        if (rk) pass_a_dispatch<false, true>(P, act, mode, grid, tab, smem, st);
        else pass_a_dispatch<false, false>(P, act, mode, grid, tab, smem, st);
    }
}

void launch_broadcast(const Plan& P, const Active& act, bool aligned, int sms, cudaStream_t st) {
    const int grid = dense_grid(P, sms, 4);
    if (aligned) broadcast_kernel<true><<<grid, 256, 0, st>>>(P, act);
    else broadcast_kernel<false><<<grid, 256, 0, st>>>(P, act);
}

void launch_local_step(const Plan& P, const Active& act, const StepArgs& sa, bool aligned, int sms, cudaStream_t st) {
    const dim3 grid(dense_grid(P, sms, 2), act.n);
    if (sa.vel) {
        if (aligned) local_step_kernel<true, true><<<grid, 256, 0, st>>>(P, act, sa);
        else local_step_kernel<false, true><<<grid, 256, 0, st>>>(P, act, sa);
    } else {
        if (aligned) local_step_kernel<true, false><<<grid, 256, 0, st>>>(P, act, sa);
        else local_step_kernel<false, false><<<grid, 256, 0, st>>>(P, act, sa);
    }
}

}  // namespace qs
