// Dense passes of the sync round: everything that touches all R x d coordinates.
//
//   pass_a      u = mem + (anchor - xw) written over mem, candidate bitmap against the
//               predicted threshold, and (fused round) the broadcast of the old model
//   fb_*        exact fallback when a prediction missed: histogram of the top key bits,
//               new threshold, bitmap rebuilt from the stored u
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

// segment of each coordinate of a quad
__device__ __forceinline__ void quad_segments(const Plan& P, uint32_t g, uint32_t e0, int sg[4]) {
    if (P.nseg == 1) {
        sg[0] = sg[1] = sg[2] = sg[3] = 0;
        return;
    }
    int sq = (int)P.grp_seg[g];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        while (sq + 1 < P.nseg && e0 + j >= P.seg_off[sq + 1]) ++sq;
        sg[j] = sq;
    }
}

constexpr int WB = 4;  // workers whose loads are issued together

// mode 0: compress only; mode 1: fused round (xw_r, and anchors_r if bound, receive x).
template <bool ALIGNED, bool RANDK>
__global__ void __launch_bounds__(256) pass_a_kernel(const Plan P, const Active act, const int mode) {
    const int lane = threadIdx.x & 31;
    const uint32_t nwarps = gridDim.x * 8u;
    bool bad = false;
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += nwarps) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        int sg[4];
        quad_segments(P, g, e0, sg);
        float xq[4];
        load_quad<ALIGNED>(P.x, e0, P.d, xq);
        for (int w0 = 0; w0 < act.n; w0 += WB) {
            float xw[WB][4], mm[WB][4], an[WB][4];
#pragma unroll
            for (int b = 0; b < WB; ++b) {
                if (w0 + b < act.n) {
                    const size_t row = (size_t)act.r[w0 + b] * P.d;
                    load_quad<ALIGNED>(P.xw + row, e0, P.d, xw[b]);
                    load_quad<ALIGNED>(P.mem + row, e0, P.d, mm[b]);
                    if (P.anchors) load_quad<ALIGNED>(P.anchors + row, e0, P.d, an[b]);
                }
            }
#pragma unroll
            for (int b = 0; b < WB; ++b) {
                if (w0 + b >= act.n) break;
                const int r = act.r[w0 + b];
                const size_t row = (size_t)r * P.d;
                const uint32_t* gs = P.guess + (size_t)r * P.nseg;
                uint4 h;
                if (RANDK) h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
                const uint32_t hh[4] = {RANDK ? h.x : 0u, RANDK ? h.y : 0u, RANDK ? h.z : 0u,
                                        RANDK ? h.w : 0u};
                float u[4];
                uint32_t fl[4];
                const uint32_t g0 = gs[sg[0]];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float anchor = P.anchors ? an[b][j] : xq[j];
                    const float diff = anchor - xw[b][j];
                    u[j] = mm[b][j] + diff;
                    const uint32_t key = topk_key(u[j]);
                    bad |= key >= 0xFF000000u;
                    const uint32_t gj = (sg[j] == sg[0]) ? g0 : gs[sg[j]];
                    const uint32_t sk = RANDK ? ~hh[j] : key;
                    fl[j] = (e0 + j < P.d) && (sk >= gj);
                }
                store_quad<ALIGNED>(P.mem + row, e0, P.d, u);
                if (mode == 1) {
                    store_quad<ALIGNED>(P.xw + row, e0, P.d, xq);
                    if (P.anchors) store_quad<ALIGNED>(P.anchors + row, e0, P.d, xq);
                }
                const uint32_t b0 = __ballot_sync(0xffffffffu, fl[0]);
                const uint32_t b1 = __ballot_sync(0xffffffffu, fl[1]);
                const uint32_t b2 = __ballot_sync(0xffffffffu, fl[2]);
                const uint32_t b3 = __ballot_sync(0xffffffffu, fl[3]);
                if (lane == 0)
                    reinterpret_cast<uint4*>(P.bitmap)[(size_t)r * P.ngroups + g] =
                        make_uint4(b0, b1, b2, b3);
            }
        }
    }
    if (bad) set_status(P, QS_NONFINITE);
}

// Rebuilds the bitmap of the workers whose prediction missed from the stored u.
template <bool RANDK>
__global__ void __launch_bounds__(256) reflag_kernel(const Plan P, const Active act) {
    const int lane = threadIdx.x & 31;
    const int r = act.r[blockIdx.y];
    if (!P.fail[r]) return;
    const size_t row = (size_t)r * P.d;
    const uint32_t* gs = P.guess + (size_t)r * P.nseg;
    for (uint32_t g = blockIdx.x * 8u + (threadIdx.x >> 5); g < P.ngroups; g += gridDim.x * 8u) {
        const uint32_t e0 = g * (uint32_t)GROUP + (uint32_t)lane * 4u;
        int sg[4];
        quad_segments(P, g, e0 < P.d ? e0 : P.d - 1, sg);
        uint4 h;
        if (RANDK) h = philox_quad(P, (uint32_t)r, e0 >> 2, 1u);
        const uint32_t hh[4] = {RANDK ? h.x : 0u, RANDK ? h.y : 0u, RANDK ? h.z : 0u, RANDK ? h.w : 0u};
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
        if (lane == 0)
            reinterpret_cast<uint4*>(P.bitmap)[(size_t)r * P.ngroups + g] = make_uint4(b0, b1, b2, b3);
    }
}

// Histogram of the top 11 key bits of one stretch of one segment, for missed workers.
template <bool RANDK>
__global__ void __launch_bounds__(256) fb_hist_kernel(const Plan P, const Active act) {
    __shared__ uint32_t sh[FB_BINS];
    const int r = act.r[blockIdx.y];
    if (!P.fail[r]) return;
    const FbBlock blk = P.fb_tab[blockIdx.x];
    for (int i = threadIdx.x; i < FB_BINS; i += 256) sh[i] = 0;
    __syncthreads();
    const size_t row = (size_t)r * P.d;
    for (uint32_t base = 0; base < blk.len; base += 256) {
        const uint32_t i = base + threadIdx.x;
        const bool valid = i < blk.len;
        const uint32_t live = __ballot_sync(0xffffffffu, valid);
        if (valid) {
            const uint32_t e = blk.start + i;
            const uint32_t sk = RANDK ? ~philox_word(P, (uint32_t)r, e, 1u) : topk_key(P.mem[row + e]);
            const uint32_t bin = sk >> FB_SHIFT;
            const uint32_t peers = __match_any_sync(live, bin);
            if ((threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&sh[bin], __popc(peers));
        }
    }
    __syncthreads();
    uint32_t* out = P.fb_hist + ((size_t)r * P.nseg + blk.seg) * FB_BINS;
    for (int i = threadIdx.x; i < FB_BINS; i += 256)
        if (sh[i]) atomicAdd(&out[i], sh[i]);
}

// New threshold of each segment of a missed worker: the lowest bin edge that still leaves
// at least `target` coordinates above it.  Clears the histogram.
__global__ void __launch_bounds__(256) fb_guess_kernel(const Plan P, const Active act) {
    __shared__ uint32_t scan[33];
    __shared__ uint32_t best;
    const int r = act.r[blockIdx.y];
    if (!P.fail[r]) return;
    const uint32_t seg = blockIdx.x;
    uint32_t* hist = P.fb_hist + ((size_t)r * P.nseg + seg) * FB_BINS;
    // thread t owns bins descending from the top: 2047 - 8t .. 2040 - 8t
    uint32_t v[8], s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int bin = FB_BINS - 1 - 8 * (int)threadIdx.x - i;
        v[i] = hist[bin];
        hist[bin] = 0;
        s += v[i];
    }
    if (threadIdx.x == 0) best = 0;
    uint32_t total;
    const uint32_t excl = block_excl_scan(s, scan, &total);
    const uint32_t target = P.target[seg];
    // the owner of the crossing: excl < target <= excl + s
    if (excl < target && excl + s >= target) {
        uint32_t run = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            run += v[i];
            if (run >= target) { best = (uint32_t)(FB_BINS - 1 - 8 * (int)threadIdx.x - i); break; }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) P.guess[(size_t)r * P.nseg + seg] = best << FB_SHIFT;
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

void launch_pass_a(const Plan& P, const Active& act, int mode, bool aligned, int sms, cudaStream_t st) {
    const int grid = dense_grid(P, sms, 4);
    const bool rk = P.sp == QS_RANDK;
    if (aligned) {
        if (rk) pass_a_kernel<true, true><<<grid, 256, 0, st>>>(P, act, mode);
        else pass_a_kernel<true, false><<<grid, 256, 0, st>>>(P, act, mode);
    } else {
        if (rk) pass_a_kernel<false, true><<<grid, 256, 0, st>>>(P, act, mode);
        else pass_a_kernel<false, false><<<grid, 256, 0, st>>>(P, act, mode);
    }
}

void launch_fallback(const Plan& P, const Active& act, int sms, cudaStream_t st) {
    const bool rk = P.sp == QS_RANDK;
    const dim3 gh(P.nfb, act.n), gg(P.nseg, act.n), gr(dense_grid(P, sms, 2), act.n);
    if (rk) fb_hist_kernel<true><<<gh, 256, 0, st>>>(P, act);
    else fb_hist_kernel<false><<<gh, 256, 0, st>>>(P, act);
    fb_guess_kernel<<<gg, 256, 0, st>>>(P, act);
    if (rk) reflag_kernel<true><<<gr, 256, 0, st>>>(P, act);
    else reflag_kernel<false><<<gr, 256, 0, st>>>(P, act);
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
