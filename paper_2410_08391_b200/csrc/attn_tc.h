// Host interface of the tcgen05 causal GQA attention (bf16, head_dim 64 or 128).
#pragma once
#include "common.cuh"

bool attn_tc_supported(int hd, int ld, const void* qkv, int ldo, const void* out);
// Number of work items (`tiles` = 2 or 1 query tiles of 128 rows each) of a ragged batch; cu_host: [batch + 1] sequence starts.
int attn_tc_items(const int* cu_host, int batch, int tiles);
// Fills sched[0 .. items) from the device copy of the sequence starts (once per call of the path).
void launch_attn_schedule(const int* cu_dev, int batch, int tiles, int2* sched, cudaStream_t st, int64_t* n_launch);
// qkv: [total, (nq + 2 nkv) * hd] bf16 with row stride ld (q heads, then k heads, then v heads; q and k
// after RoPE); out: [total, nq * hd] bf16 with row stride ldo.  half_operands: qkv holds IEEE halves instead of bf16.
// out_lo (or null): receives the bf16 remainder of the output, same layout as out.
cudaError_t launch_attn_tc(const bf16* qkv, int ld, int total, int nq, int nkv, int hd, const int* cu_dev, const int2* sched,
                           int n_items, int tiles, bf16* out, int ldo, int* status, cudaStream_t st, int64_t* n_launch,
                           bool half_operands = false, bf16* out_lo = nullptr);
