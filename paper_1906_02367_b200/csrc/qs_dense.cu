// Dense passes of the sync round: everything that touches all R x d coordinates.
//
//   pass_a      u = mem + (anchor - xw) written over mem, candidate bitmap against the
//               predicted threshold with per-block candidate counts, and (fused round) the
//               broadcast of the old model
//   broadcast   xw_r <- x,   local_step  xw_r <- xw_r - eta grad_r
//
// One warp owns a group of 128 consecutive coordinates (4 per lane, one 128-bit access
// per array) and loops over the workers with the model quad held in registers, so x is
// read once for all R workers.
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

// Store that asks the L2 to keep the line: used for the few quads that hold a candidate, which
// the selection stages read back right after this pass.
template <bool ALIGNED>
__device__ __forceinline__ void store_quad_keep(float* __restrict__ row, uint32_t e0, uint32_t d, const float v[4],
                                                uint64_t policy) {
    if (ALIGNED) {
        if (e0 < d)
            asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(row + e0), "f"(v[0]),
                         "f"(v[1]), "f"(v[2]), "f"(v[3]), "l"(policy)
                         : "memory");
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (e0 + j < d)
                asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(row + e0 + j), "f"(v[j]), "l"(policy)
                             : "memory");
    }
}

constexpr int WB = 4;            // workers whose loads are issued together
constexpr int TAB_MAX = 11 * 1024;   // words of shared memory for the threshold and offset tables

// mode 0: compress only; mode 1: fused round (xw_r, and anchors_r if bound, receive x).
// Shared memory holds the candidate thresholds of all workers and the segment offsets when
// they fit (tab != 0), so that the inner loop never waits on global memory for them.
template <bool ALIGNED, bool RANDK, bool ANCH>
__global__ void __launch_bounds__(256) pass_a_kernel(const Plan P, const Active act, const int mode, const int tab) {
    extern __shared__ uint32_t sh_tab[];
    const int lane = threadIdx.x & 31;
    const uint32_t nwarps = gridDim.x * 8u;
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
    uint64_t keep;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += nwarps) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        int sg[4] = {0, 0, 0, 0};
        if (P.nseg > 1) {
            int sq = (int)P.grp_seg[g];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                while (sq + 1 < P.nseg && e0 + j >= seg_off[sq + 1]) ++sq;
                sg[j] = sq;
            }
        }
        float xq[4];
        load_quad<ALIGNED>(P.x, e0, P.d, xq);
        for (int w0 = 0; w0 < act.n; w0 += WB) {
            float xw[WB][4], mm[WB][4], an[ANCH ? WB : 1][4];
#pragma unroll
            for (int b = 0; b < WB; ++b) {
                if (w0 + b < act.n) {
                    const size_t row = (size_t)act.r[w0 + b] * P.d;
                    load_quad<ALIGNED>(P.xw + row, e0, P.d, xw[b]);
                    load_quad<ALIGNED>(P.mem + row, e0, P.d, mm[b]);
                    if (ANCH) load_quad<ALIGNED>(P.anchors + row, e0, P.d, an[ANCH ? b : 0]);
                }
            }
#pragma unroll
            for (int b = 0; b < WB; ++b) {
                if (w0 + b >= act.n) break;
                const int r = act.r[w0 + b];
                const size_t row = (size_t)r * P.d;
                const uint32_t* gs = guess + (size_t)r * P.nseg;
                uint4 h = make_uint4(0, 0, 0, 0);
                if (RANDK) h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
                const uint32_t hh[4] = {h.x, h.y, h.z, h.w};
                float u[4];
                uint32_t fl[4];
                const uint32_t g0 = gs[sg[0]];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float anchor = ANCH ? an[ANCH ? b : 0][j] : xq[j];
                    const float diff = anchor - xw[b][j];
                    u[j] = mm[b][j] + diff;
                    const uint32_t key = topk_key(u[j]);
                    bad |= key >= 0xFF000000u;
                    const uint32_t gj = (sg[j] == sg[0]) ? g0 : gs[sg[j]];
                    const uint32_t sk = RANDK ? ~hh[j] : key;
                    fl[j] = (e0 + j < P.d) && (sk >= gj);
                }
                if (fl[0] | fl[1] | fl[2] | fl[3]) store_quad_keep<ALIGNED>(P.mem + row, e0, P.d, u, keep);
                else store_quad<ALIGNED>(P.mem + row, e0, P.d, u);
                if (mode == 1) {
                    store_quad<ALIGNED>(P.xw + row, e0, P.d, xq);
                    if (ANCH) store_quad<ALIGNED>(P.anchors + row, e0, P.d, xq);
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

template <bool ALIGNED>
__global__ void __launch_bounds__(256) local_step_kernel(const Plan P, const Active act,
                                                         const float* __restrict__ grad, const float eta) {
    const int lane = threadIdx.x & 31;
    const int r = act.r[blockIdx.y];
    const size_t row = (size_t)r * P.d;
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * 8u) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        if (e0 >= P.d) continue;
        float w[4], gr[4];
        load_quad<ALIGNED>(P.xw + row, e0, P.d, w);
        load_quad<ALIGNED>(grad + row, e0, P.d, gr);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float step = eta * gr[j];
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
    const int grid = dense_grid(P, sms, 2);
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

void launch_local_step(const Plan& P, const Active& act, const float* grad, float eta, bool aligned,
                       int sms, cudaStream_t st) {
    const dim3 grid(dense_grid(P, sms, 2), act.n);
    if (aligned) local_step_kernel<true><<<grid, 256, 0, st>>>(P, act, grad, eta);
    else local_step_kernel<false><<<grid, 256, 0, st>>>(P, act, grad, eta);
}

}  // namespace qs
