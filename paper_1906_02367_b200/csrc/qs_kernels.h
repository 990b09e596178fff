// Host-side launchers of the kernel families (one translation unit each).
#pragma once
#include "qs_common.cuh"

namespace qs {

inline int chunk_grid(const Plan& P, int sms) {
    const uint32_t cap = (uint32_t)sms * 8u;
    return (int)(P.maxchunks < cap ? (P.maxchunks ? P.maxchunks : 1u) : cap);
}

// qs_dense.cu
void launch_pass_a(const Plan& P, const Active& act, int mode, bool aligned, int sms, cudaStream_t st);
void launch_fallback(const Plan& P, const Active& act, int sms, cudaStream_t st);
void launch_broadcast(const Plan& P, const Active& act, bool aligned, int sms, cudaStream_t st);
void launch_local_step(const Plan& P, const Active& act, const float* grad, float eta, bool aligned,
                       int sms, cudaStream_t st);
// qs_select.cu
void launch_candidates(const Plan& P, const Active& act, int only_failed, cudaStream_t st);
void launch_select(const Plan& P, const Active& act, int sms, cudaStream_t st);
// qs_codec.cu
void launch_quantize(const Plan& P, const Active& act, int sms, cudaStream_t st);
void launch_pack(const Plan& P, const Active& act, uint32_t* wire, long long stride, long long* bits_out,
                 int sms, cudaStream_t st);
void launch_decode(const Plan& P, const Active& act, const uint32_t* wire, long long stride, int patch,
                   int sms, cudaStream_t st);
void launch_export(const Plan& P, long long* sel_idx, int* level, uint8_t* sign, float* norm, long long* n,
                   int sms, cudaStream_t st);

// kernels each launcher enqueues (for the launch counter)
constexpr int N_PASS_A = 1, N_FALLBACK = 3, N_CANDIDATES = 3, N_SELECT = 7, N_QUANTIZE = 4, N_PACK = 2,
              N_DECODE = 3, N_BROADCAST = 1, N_LOCAL_STEP = 1, N_EXPORT = 1;

}  // namespace qs
