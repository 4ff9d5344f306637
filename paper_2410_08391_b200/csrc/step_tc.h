// Host interface of the tensor-core projections of the base model's single-token step for
// batches too large for the CUDA-core kernels to stay bandwidth-bound (bf16 weights).
#pragma once
#include "common.cuh"

enum StepPrepMode : int { PREP_PLAIN = 0, PREP_NORM = 1, PREP_SWIGLU = 2 };

// Rows of the operand buffer: batch rounded up to a multiple of 8 (hi rows, then as many lo rows).
inline int step_tc_rows(int batch) { return (batch + 7) / 8 * 8; }
bool step_tc_supported(int batch, int K, int ldw, const void* W, const void* XB);

// XB[b, :] = bf16(v_b), XB[Bp + b, :] = bf16(v_b - bf16(v_b)) for b < batch (zero rows up to Bp), where
//   PREP_PLAIN:  v_b = x[b, 0:K]
//   PREP_NORM:   v_b = gain * x[b] / sqrt(mean(x[b]^2) + eps)
//   PREP_SWIGLU: v_b[c] = silu(x[b, gate row c]) * x[b, up row c], c < K = ffn, rows placed as in the packed w_gate/w_up
// Also clears zero_ptr[b, 0:zero_n] (row stride zero_ld) for b < batch when zero_ptr is given.
void launch_step_prep(const LaunchCtx&, int mode, const float* x, int ldx, int K, int batch, const float* gain, float eps,
                      int G, bf16* XB, float* zero_ptr, int zero_ld, int zero_n);

// Y[b, n] += sum_k W[n, k] (XB[b, k] + XB[Bp + b, k]) for b < batch, n < N; fp32 atomic adds.
// next_w / next_bytes: the weight matrix the next projection will read (or null): its first megabytes are asked into L2.
cudaError_t launch_step_gemm_tc(const bf16* W, int ldw, int N, int K, const bf16* XB, int batch, float* Y, int ldy,
                                int n_sm, int* status, cudaStream_t st, int64_t* n_launch, const void* next_w = nullptr,
                                size_t next_bytes = 0);
