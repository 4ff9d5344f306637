// Kernels of the training-time forward (Sec. 4.1 "Training", Sec. 4.3): the base model over the whole
// prompt with the predicted cache as keys and values, and the consistency terms L1(KV_hat, KV_B).
// Both work on the projection buffer of one layer, [T, (nq + 2 nkv) * hd] with the layer's own keys (after
// RoPE) and values in its last 2 * nkv * hd columns, and on the paged predicted cache of that layer.
#include "common.cuh"

namespace {

// element (t, c) of a layer's cache: c = head * hd + dim, slot = page * PAGE_TOKENS + row of token t
__device__ __forceinline__ size_t cache_off(int slot, int c, int nkv, int hd) {
  const int page = slot / PAGE_TOKENS, row = slot - page * PAGE_TOKENS;
  const int head = c / hd, dim = c - head * hd;
  return (((size_t)page * nkv + head) * PAGE_TOKENS + row) * hd + dim;
}

// sums[0] += inv_n * sum |K_hat - K_B|, sums[1] += inv_n * sum |V_hat - V_B| over all tokens and columns.
// The layer's own keys and values are read as hi (+ lo, bf16 mode) parts.
template <class T, class QT>
__global__ void __launch_bounds__(256) kv_l1_kernel(const QT* __restrict__ qkv, int ld, int k_col, const bf16* __restrict__ kv_lo,
                                                    int ld_lo, int T_tokens, int nkv, int hd, const int* __restrict__ tok_slot,
                                                    const typename KvOf<T>::type* __restrict__ kpool,
                                                    const typename KvOf<T>::type* __restrict__ vpool, float inv_n,
                                                    float* __restrict__ sum_k, float* __restrict__ sum_v) {
  const int dkv = nkv * hd;
  const size_t n = (size_t)T_tokens * dkv;
  float sk = 0.f, sv = 0.f;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(e / dkv), c = (int)(e - (size_t)t * dkv);
    const int slot = tok_slot[t];
    if (slot < 0) continue;
    float k = to_f(qkv[(size_t)t * ld + k_col + c]), v = to_f(qkv[(size_t)t * ld + k_col + dkv + c]);
    if (kv_lo) { k += to_f(kv_lo[(size_t)t * ld_lo + c]); v += to_f(kv_lo[(size_t)t * ld_lo + dkv + c]); }
    const size_t off = cache_off(slot, c, nkv, hd);
    sk += fabsf(to_f(kpool[off]) - k);
    sv += fabsf(to_f(vpool[off]) - v);
  }
  __shared__ float red[2][8];
  sk = warp_sum(sk); sv = warp_sum(sv);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sk; red[1][threadIdx.x >> 5] = sv; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int w = 0; w < 8; ++w) { a += red[0][w]; b += red[1][w]; }
    atomicAdd(sum_k, a * inv_n);
    atomicAdd(sum_v, b * inv_n);
  }
}

// The layer's key and value columns of the projection buffer take the predicted cache's entries.
template <class T, class QT>
__global__ void __launch_bounds__(256) kv_take_kernel(QT* __restrict__ qkv, int ld, int k_col, int T_tokens, int nkv, int hd,
                                                      const int* __restrict__ tok_slot,
                                                      const typename KvOf<T>::type* __restrict__ kpool,
                                                      const typename KvOf<T>::type* __restrict__ vpool) {
  const int dkv = nkv * hd;
  const size_t n = (size_t)T_tokens * dkv;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(e / dkv), c = (int)(e - (size_t)t * dkv);
    const int slot = tok_slot[t];
    if (slot < 0) continue;
    const size_t off = cache_off(slot, c, nkv, hd);
    qkv[(size_t)t * ld + k_col + c] = from_f<QT>(to_f(kpool[off]));          // exact when QT is the cache's own type
    qkv[(size_t)t * ld + k_col + dkv + c] = from_f<QT>(to_f(vpool[off]));
  }
}

int grid_of(size_t n) { size_t g = (n + 255) / 256; return (int)(g < 1 ? 1 : (g > 4096 ? 4096 : g)); }

}  // namespace

void launch_kv_l1(const LaunchCtx& ctx, const void* qkv, int ld, int k_col, const void* kv_lo, int ld_lo, int T_tokens, int nkv,
                  int hd, const int* tok_slot, const void* kpool, const void* vpool, float* sum_k, float* sum_v, bool qkv_is_half) {
  const size_t n = (size_t)T_tokens * nkv * hd;
  if (n == 0) return;
  const float inv_n = 1.f / (float)n;
  ++*ctx.n_launch;
  if (ctx.dtype == 0)
    kv_l1_kernel<float, float><<<grid_of(n), 256, 0, ctx.st>>>((const float*)qkv, ld, k_col, nullptr, 0, T_tokens, nkv, hd, tok_slot,
                                                       (const float*)kpool, (const float*)vpool, inv_n, sum_k, sum_v);
  else if (qkv_is_half)
    kv_l1_kernel<bf16, kv16><<<grid_of(n), 256, 0, ctx.st>>>((const kv16*)qkv, ld, k_col, nullptr, 0, T_tokens, nkv, hd,
                                                            tok_slot, (const kv16*)kpool, (const kv16*)vpool, inv_n, sum_k, sum_v);
  else
    kv_l1_kernel<bf16, bf16><<<grid_of(n), 256, 0, ctx.st>>>((const bf16*)qkv, ld, k_col, (const bf16*)kv_lo, ld_lo, T_tokens, nkv, hd,
                                                            tok_slot, (const kv16*)kpool, (const kv16*)vpool, inv_n, sum_k, sum_v);
}

void launch_kv_take(const LaunchCtx& ctx, void* qkv, int ld, int k_col, int T_tokens, int nkv, int hd, const int* tok_slot,
                    const void* kpool, const void* vpool, bool qkv_is_half) {
  const size_t n = (size_t)T_tokens * nkv * hd;
  if (n == 0) return;
  ++*ctx.n_launch;
  if (ctx.dtype == 0)
    kv_take_kernel<float, float><<<grid_of(n), 256, 0, ctx.st>>>((float*)qkv, ld, k_col, T_tokens, nkv, hd, tok_slot, (const float*)kpool,
                                                         (const float*)vpool);
  else if (qkv_is_half)
    kv_take_kernel<bf16, kv16><<<grid_of(n), 256, 0, ctx.st>>>((kv16*)qkv, ld, k_col, T_tokens, nkv, hd, tok_slot, (const kv16*)kpool,
                                                              (const kv16*)vpool);
  else
    kv_take_kernel<bf16, bf16><<<grid_of(n), 256, 0, ctx.st>>>((bf16*)qkv, ld, k_col, T_tokens, nkv, hd, tok_slot, (const kv16*)kpool,
                                                              (const kv16*)vpool);
}
