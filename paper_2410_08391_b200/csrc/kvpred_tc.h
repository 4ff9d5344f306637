// Host interface of the fused K/V projection + KV predictor kernel (tcgen05, sm_100a).
#pragma once
#include "common.cuh"

struct KvPred {
  const bf16* A; int lda;            // [M, K] projection input (bf16); with ss_in: x * gain, not yet scaled by 1 / rms
  const bf16* A_lo; int lda_lo;      // its bf16 remainder, or null
  const bf16* Wkv; int ldw;          // [2 * dkv, K]: rows of Wk, then rows of Wv
  int M, K;
  int dkv, hd;                       // auxiliary layer's kv width (multiple of 64, <= 384) and head_dim (64 | 128)
  int kv_begin, kv_end;              // which of (0 = K, 1 = V) this launch computes
  const float* ss_in; float rms_eps; // folded RMSNorm: rows scaled by rsqrt(ss_in[m] / K + rms_eps); null = off
  const float2* rope_tab; int tab_stride; const int* tok_pos;
  const float* k_gain; float eps;    // key norm gain [hd] or null
  bf16* C; int ldc; int k_col;       // q|k|v buffer of the layer: keys at column k_col, values at k_col + dkv
  const void* FK; const void* FV;    // stacked predictor matrices [n_tot, dkv], IEEE halves
  int n_tot;                         // sum of the fed base layers' kv widths (multiple of 64)
  PagedOut paged[2];                 // where the predicted K (0) and V (1) columns go
  int n_sm;
};

bool kvpred_tc_supported(const KvPred& g);
cudaError_t launch_kvpred_tc(const KvPred& g, int* status, cudaStream_t st, int64_t* n_launch);
