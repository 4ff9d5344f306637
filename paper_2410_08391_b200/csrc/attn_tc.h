// Host interface of the tcgen05 causal GQA attention (bf16, head_dim 64 or 128).
#pragma once
#include "common.cuh"

bool attn_tc_supported(int hd, int ld, const void* qkv, int ldo, const void* out);
// qkv: [total, (nq + 2 nkv) * hd] bf16 with row stride ld (q heads, then k heads, then v heads; q and k
// after RoPE); cu_dev: [batch + 1] sequence starts; out: [total, nq * hd] bf16 with row stride ldo.
cudaError_t launch_attn_tc(const bf16* qkv, int ld, int total, int nq, int nkv, int hd, const int* cu_dev, int batch,
                           bf16* out, int ldo, int* status, cudaStream_t st, int64_t* n_launch);
