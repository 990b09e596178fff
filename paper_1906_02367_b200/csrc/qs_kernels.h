// Host-side launchers of the kernel families (one translation unit each).
#pragma once
#include "qs_common.cuh"

namespace qs {

// qs_dense.cu
void launch_pass_a(const Plan& P, const Active& act, int mode, bool aligned, int sms, cudaStream_t st);
void launch_broadcast(const Plan& P, const Active& act, bool aligned, int sms, cudaStream_t st);
// the local step: sa.vel == nullptr plain, otherwise with momentum
void launch_local_step(const Plan& P, const Active& act, const StepArgs& sa, bool aligned, int sms, cudaStream_t st);
// qs_dense_tma.cu: the dense pass fed by bulk copies (aligned rows); step 0 none, 1 the plain local
// step taken on the way (sa.grad, sa.eta), 2 the step with momentum (sa.vel, sa.mu too)
bool pass_a_tma_usable(const Plan& P, bool aligned, int step);
cudaError_t launch_pass_a_tma(const Plan& P, const Active& act, const StepArgs& sa, int step, int sms, cudaStream_t st);
// qs_mid.cu: the persistent kernel that runs every stage after the dense pass
int mid_blocks_per_sm(bool randk);
cudaError_t launch_mid(const Plan& P, const Active& act, int do_compress, int do_pack, int do_decode,
                       int do_broadcast, int aligned, uint32_t* wire, long long stride, long long wire_words,
                       long long* bits_out, int grid, cudaStream_t st);
void launch_export(const Plan& P, long long* sel_idx, int* level, uint8_t* sign, float* norm, long long* n,
                   int sms, cudaStream_t st);

// qs_gaps.cu: plain records <-> gap-coded records
uint32_t gap_chunk(void);
uint32_t gap_unit_words(void);           // words of the per-unit table, per (worker, segment)
cudaError_t launch_recode_gaps(const Plan& P, const Active& act, const uint32_t* wire, long long stride, uint32_t* out,
                               long long out_stride, long long* bits_out, uint32_t longest_k, uint32_t most_words,
                               uint32_t row_chunks, cudaStream_t st);
cudaError_t launch_decode_gaps(const Plan& P, const Active& act, const uint32_t* packed, long long packed_stride,
                               uint32_t* wire, long long stride, uint32_t longest_k, uint32_t most_words,
                               uint32_t row_chunks, cudaStream_t st);

}  // namespace qs
