// Host interface of the tcgen05 GEMM (bf16 operands, fp32 accumulation in tensor memory).
#pragma once
#include "common.cuh"

enum TcEpi : int {
  TC_STORE = 0,   // C[m, n] = bf16(acc)
  TC_RESID = 1,   // X[m, n] += acc (fp32 residual stream)
  TC_SWIGLU = 2,  // W rows interleaved (64 gate rows, 64 up rows); C[m, c] = bf16(silu(gate_c) * up_c) (+ remainder to C_lo)
  TC_QKV = 3,     // RoPE on columns < rot_cols, bf16 hi to C, bf16 lo of columns >= lo_col_begin to C_lo
  TC_PAGED = 4    // predictor: columns scattered into cache pages
};

struct TcGemm {
  const bf16* A; int lda;          // [M, K]
  const bf16* A2; int lda2;        // lo part of A or null
  int split_begin;                 // tiles reaching columns >= split_begin add A2 W^T
  const bf16* W; int ldw;          // [N, K]
  int M, N, K;
  int epi;
  bf16* C; int ldc;
  float* X; int ldx;
  bf16* C_lo; int ld_lo; int lo_col_begin;
  int rot_cols; int hd;
  const float2* rope_tab;          // [hd/4][position] entries of (cos, sin) of two neighbouring frequencies
  int tab_stride;                  // positions in the table
  const int* tok_pos;              // [M] position of each row in its sequence
  int ffn;
  // TC_QKV with query / key norm: columns < q_cols are query heads (gain q_gain), the other rotated columns key
  // heads (gain k_gain); null gains = no norm
  const float* q_gain; const float* k_gain; int q_cols; float eps;
  PagedOut paged;
  // RMSNorm folded into the neighbouring GEMMs (all null / 0 = off).
  // TC_RESID with H: besides X += A W^T the epilogue writes H[m, n] = bf16(X[m, n] * gain_next[n]) (row stride ldh;
  // H_lo = the bf16 remainder, or null) and adds the row's share of sum_n X[m, n]^2 to ss_out[m] (cleared by the
  // caller).  Only where tc_gemm_resid_can_fuse() holds (every output tile computed by one CTA).
  // TC_QKV / TC_SWIGLU with ss_in: the accumulator rows are scaled by rsqrt(ss_in[m] / K + rms_eps).
  bf16* H; bf16* H_lo; int ldh; const float* gain_next; float* ss_out;
  const float* ss_in; float rms_eps;
  int lo_is_half;                             // TC_QKV: C_lo receives the whole value as an IEEE half (not the bf16 remainder)
  int h_is_half;                              // TC_RESID with H: H is written as IEEE halves (then without H_lo)
  int c_is_half;                   // TC_QKV: C is written as IEEE halves (for an attention that takes half operands)
  int f16_operands;                // A and W hold IEEE halves instead of bf16 (same 2 bytes; both operands alike)
  int n_sm;
  int bn;                          // tile width: 128, 256, or 0 = chosen by the launcher
};

bool tc_gemm_supported(const TcGemm& g);
bool tc_gemm_resid_can_fuse(int M, int N, int n_sm);
cudaError_t launch_gemm_tc(const TcGemm& g, int* status, cudaStream_t st, int64_t* n_launch);
void launch_rope_table(const LaunchCtx& ctx, float2* tab, int n_pos, int hd, float theta);
