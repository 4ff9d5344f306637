// Kernels of the base model's single-token step: everything here is bound by HBM
// bandwidth (each weight and each cached K/V element is read once), activations are fp32.
#include <math.h>

#include "common.cuh"

// ---------------------------------------------------------------------------------------
// Skinny GEMM  y[b, n] = sum_k W[n, k] x[b, k]  for a handful of rows b.
// One warp per output column n, 16-byte weight loads, fp32 accumulation, warp-shuffle
// reduction.  MODE: store / add into y / SwiGLU of a (gate, up) row pair.
// ---------------------------------------------------------------------------------------
namespace {
template <class T> struct Vec8;
template <> struct Vec8<bf16> {
  static __device__ __forceinline__ void load(const bf16* p, float* f) {
    uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
  }
};
template <> struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, float* f) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
  }
};

template <class T, int BB>
__device__ __forceinline__ void row_dot(const T* __restrict__ w, const float* __restrict__ x, int ldx, int K, int nb,
                                        bool vec_ok, int lane, float* acc) {
  if (vec_ok) {
    for (int k = lane * 8; k < K; k += 256) {
      float wf[8];
      Vec8<T>::load(w + k, wf);
#pragma unroll
      for (int b = 0; b < BB; ++b) {
        if (b < nb) {
          float4 x0 = *reinterpret_cast<const float4*>(x + (size_t)b * ldx + k);
          float4 x1 = *reinterpret_cast<const float4*>(x + (size_t)b * ldx + k + 4);
          acc[b] += wf[0] * x0.x + wf[1] * x0.y + wf[2] * x0.z + wf[3] * x0.w + wf[4] * x1.x + wf[5] * x1.y +
                    wf[6] * x1.z + wf[7] * x1.w;
        }
      }
    }
  } else {
    for (int k = lane; k < K; k += 32) {
      float wv = to_f(w[k]);
#pragma unroll
      for (int b = 0; b < BB; ++b)
        if (b < nb) acc[b] = fmaf(wv, x[(size_t)b * ldx + k], acc[b]);
    }
  }
}

template <class T, int BB, int MODE>
__global__ void __launch_bounds__(256) step_gemv_kernel(const T* __restrict__ W, int ldw, int N, int K,
                                                        const float* __restrict__ x, int ldx, int batch,
                                                        float* __restrict__ y, int ldy, RowMap mg, RowMap mu) {
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n = blockIdx.x * 8 + warp;
  if (n >= N) return;
  int b0 = blockIdx.y * BB;
  int nb = min(BB, batch - b0);
  const float* xb = x + (size_t)b0 * ldx;
  bool vec_ok = (K % 8 == 0) && (ldw % 8 == 0) && (ldx % 4 == 0);
  float acc[BB];
#pragma unroll
  for (int b = 0; b < BB; ++b) acc[b] = 0.f;
  if (MODE == GEMV_SWIGLU) {
    float accu[BB];
#pragma unroll
    for (int b = 0; b < BB; ++b) accu[b] = 0.f;
    row_dot<T, BB>(W + (size_t)map_row(mg, n) * ldw, xb, ldx, K, nb, vec_ok, lane, acc);
    row_dot<T, BB>(W + (size_t)map_row(mu, n) * ldw, xb, ldx, K, nb, vec_ok, lane, accu);
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float g = warp_sum(acc[b]), u = warp_sum(accu[b]);
      if (lane == 0 && b < nb) y[(size_t)(b0 + b) * ldy + n] = g / (1.f + __expf(-g)) * u;
    }
  } else {
    row_dot<T, BB>(W + (size_t)n * ldw, xb, ldx, K, nb, vec_ok, lane, acc);
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float v = warp_sum(acc[b]);
      if (lane == 0 && b < nb) {
        float* dst = y + (size_t)(b0 + b) * ldy + n;
        *dst = (MODE == GEMV_RESID) ? *dst + v : v;
      }
    }
  }
}

template <class T, int BB>
void gemv_go(const LaunchCtx& ctx, const void* W, int ldw, int N, int K, const float* x, int ldx, int batch, float* y,
             int ldy, int mode, int G, int ffn) {
  dim3 grid((N + 7) / 8, (batch + BB - 1) / BB);
  RowMap mg{0, G, 0, ffn}, mu{G == 0 ? ffn : 0, G, 1, ffn};
  if (mode == GEMV_STORE) step_gemv_kernel<T, BB, GEMV_STORE><<<grid, 256, 0, ctx.st>>>((const T*)W, ldw, N, K, x, ldx, batch, y, ldy, mg, mu);
  else if (mode == GEMV_RESID) step_gemv_kernel<T, BB, GEMV_RESID><<<grid, 256, 0, ctx.st>>>((const T*)W, ldw, N, K, x, ldx, batch, y, ldy, mg, mu);
  else step_gemv_kernel<T, BB, GEMV_SWIGLU><<<grid, 256, 0, ctx.st>>>((const T*)W, ldw, N, K, x, ldx, batch, y, ldy, mg, mu);
}
}  // namespace

void launch_step_gemv(const LaunchCtx& ctx, const void* W, int ldw, int N, int K, const float* x, int ldx, int batch,
                      float* y, int ldy, int mode, int G, int ffn) {
  if (batch == 0 || N == 0) return;
  ++*ctx.n_launch;
  if (ctx.dtype == 0) {
    if (batch == 1) gemv_go<float, 1>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
    else if (batch <= 4) gemv_go<float, 4>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
    else gemv_go<float, 8>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
  } else {
    if (batch == 1) gemv_go<bf16, 1>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
    else if (batch <= 4) gemv_go<bf16, 4>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
    else gemv_go<bf16, 8>(ctx, W, ldw, N, K, x, ldx, batch, y, ldy, mode, G, ffn);
  }
}

// ---------------------------------------------------------------------------------------
// Single-query GQA attention over the paged cache, split over the key range.
// grid (n_split, n_kv_heads, batch), 4 warps; a CTA serves the `group` query heads that
// share one kv head, applies RoPE to q at position n_keys - 1, and walks its key range
// 32 keys per warp step (lane = key for the scores, lane = dim for the value sum).
// With more than one split, partial (m, l, o) per (sequence, q head, split) go to the
// scratch buffer `part` and a second kernel merges them.
// ---------------------------------------------------------------------------------------
namespace {
constexpr int MAXG = 8;     // q heads per kv head

template <class T>
__global__ void __launch_bounds__(128) step_attn_kernel(const float* __restrict__ q, int ldq, int nq, int nkv, int hd,
                                                        const __grid_constant__ InvFreq inv,
                                                        const T* __restrict__ kpool, const T* __restrict__ vpool,
                                                        const int* __restrict__ block_table, int mpps, int n_pages,
                                                        const int* __restrict__ seq_lens, int extra, int n_split,
                                                        float* __restrict__ part, float* __restrict__ out, int* status) {
  extern __shared__ float sm[];
  int group = nq / nkv;
  float* qs = sm;                              // [MAXG][hd]
  float* red = qs + MAXG * hd;                 // [4 warps][MAXG][hd + 2]
  int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n_keys = seq_lens[b] + extra;
  int pos = n_keys - 1;
  float scale = rsqrtf((float)hd);
  int half = hd >> 1;
  for (int i = threadIdx.x; i < group * half; i += blockDim.x) {
    int h = i / half, c = i - h * half;
    const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * hd;
    float sn, cs;
    rope_sincos(pos, inv.f[c], &sn, &cs);
    float x1 = qh[c], x2 = qh[c + half];
    qs[h * hd + c] = (x1 * cs - x2 * sn) * scale;
    qs[h * hd + c + half] = (x2 * cs + x1 * sn) * scale;
  }
  __syncthreads();
  int chunk = ((n_keys + n_split - 1) / n_split + 31) & ~31;
  int s0 = sp * chunk, s1 = min(n_keys, s0 + chunk);
  float m[MAXG], l[MAXG], o[MAXG][4];
#pragma unroll
  for (int h = 0; h < MAXG; ++h) { m[h] = -INFINITY; l[h] = 0.f; o[h][0] = o[h][1] = o[h][2] = o[h][3] = 0.f; }
  bool vec_ok = (hd % 8 == 0);
  for (int t0 = s0 + warp * 32; t0 < s1; t0 += 128) {
    int s = t0 + lane;
    int slot = -1;
    if (s < s1) {
      int pg = s / PAGE_TOKENS;
      int page = pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
      if (page >= 0 && page < n_pages) slot = page * PAGE_TOKENS + (s % PAGE_TOKENS);
      else dev_flag(status, DEV_BAD_PAGE);
    }
    float sc[MAXG];
#pragma unroll
    for (int h = 0; h < MAXG; ++h) sc[h] = 0.f;
    if (slot >= 0) {
      int page = slot / PAGE_TOKENS, row = slot - page * PAGE_TOKENS;
      const T* kr = kpool + (((size_t)page * nkv + kvh) * PAGE_TOKENS + row) * hd;
      if (vec_ok) {
        for (int c = 0; c < hd; c += 8) {
          float kf[8];
          Vec8<T>::load(kr + c, kf);
#pragma unroll
          for (int h = 0; h < MAXG; ++h)
            if (h < group) {
#pragma unroll
              for (int e = 0; e < 8; ++e) sc[h] = fmaf(kf[e], qs[h * hd + c + e], sc[h]);
            }
        }
      } else {
        for (int c = 0; c < hd; ++c) {
          float kf = to_f(kr[c]);
#pragma unroll
          for (int h = 0; h < MAXG; ++h)
            if (h < group) sc[h] = fmaf(kf, qs[h * hd + c], sc[h]);
        }
      }
    }
    float p[MAXG];
#pragma unroll
    for (int h = 0; h < MAXG; ++h) {
      p[h] = 0.f;
      if (h < group) {
        float v = slot >= 0 ? sc[h] : -INFINITY;
        float mt = warp_max(v);
        float mn = fmaxf(m[h], mt);
        float alpha = (mn == -INFINITY) ? 1.f : __expf(m[h] - mn);
        p[h] = (slot >= 0) ? __expf(v - mn) : 0.f;
        l[h] = l[h] * alpha + warp_sum(p[h]);
        m[h] = mn;
#pragma unroll
        for (int i = 0; i < 4; ++i) o[h][i] *= alpha;
      }
    }
    int nk = min(32, s1 - t0);
    for (int j = 0; j < nk; ++j) {
      int sj = __shfl_sync(0xffffffffu, slot, j);
      if (sj < 0) continue;
      int page = sj / PAGE_TOKENS, row = sj - page * PAGE_TOKENS;
      const T* vr = vpool + (((size_t)page * nkv + kvh) * PAGE_TOKENS + row) * hd;
      float vv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { int c = lane + 32 * i; vv[i] = c < hd ? to_f(vr[c]) : 0.f; }
#pragma unroll
      for (int h = 0; h < MAXG; ++h)
        if (h < group) {
          float pj = __shfl_sync(0xffffffffu, p[h], j);
#pragma unroll
          for (int i = 0; i < 4; ++i) o[h][i] = fmaf(pj, vv[i], o[h][i]);
        }
    }
  }
  // merge the 4 warps
  int ldr = hd + 2;
#pragma unroll
  for (int h = 0; h < MAXG; ++h)
    if (h < group) {
      float* r = red + ((size_t)warp * MAXG + h) * ldr;
#pragma unroll
      for (int i = 0; i < 4; ++i) { int c = lane + 32 * i; if (c < hd) r[c] = o[h][i]; }
      if (lane == 0) { r[hd] = m[h]; r[hd + 1] = l[h]; }
    }
  __syncthreads();
  for (int i = threadIdx.x; i < group * hd; i += blockDim.x) {
    int h = i / hd, c = i - h * hd;
    float mm = -INFINITY;
    for (int w = 0; w < 4; ++w) mm = fmaxf(mm, red[((size_t)w * MAXG + h) * ldr + hd]);
    float ll = 0.f, oo = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float* r = red + ((size_t)w * MAXG + h) * ldr;
      float f = (r[hd] == -INFINITY) ? 0.f : __expf(r[hd] - mm);
      ll += r[hd + 1] * f;
      oo += r[c] * f;
    }
    int qh = kvh * group + h;
    if (n_split == 1) {
      out[(size_t)b * nq * hd + (size_t)qh * hd + c] = oo / ll;
    } else {
      float* pr = part + (((size_t)b * nq + qh) * n_split + sp) * ldr;
      pr[c] = oo;
      if (c == 0) { pr[hd] = mm; pr[hd + 1] = ll; }
    }
  }
}

__global__ void step_attn_merge_kernel(const float* __restrict__ part, int nq, int hd, int n_split, float* __restrict__ out) {
  int qh = blockIdx.x, b = blockIdx.y;
  int ldr = hd + 2;
  const float* pr = part + (((size_t)b * nq + qh) * n_split) * ldr;
  float mm = -INFINITY;
  for (int s = 0; s < n_split; ++s) mm = fmaxf(mm, pr[(size_t)s * ldr + hd]);
  for (int c = threadIdx.x; c < hd; c += blockDim.x) {
    float ll = 0.f, oo = 0.f;
    for (int s = 0; s < n_split; ++s) {
      const float* r = pr + (size_t)s * ldr;
      float f = (r[hd] == -INFINITY) ? 0.f : __expf(r[hd] - mm);
      ll += r[hd + 1] * f;
      oo += r[c] * f;
    }
    out[(size_t)b * nq * hd + (size_t)qh * hd + c] = oo / ll;
  }
}
}  // namespace

int step_attn_splits(int batch, int nkv, int max_keys) {
  int want = (2 * 148 + batch * nkv - 1) / (batch * nkv);
  int cap = (max_keys + 127) / 128;
  int n = want < cap ? want : cap;
  if (n < 1) n = 1;
  if (n > 64) n = 64;
  return n;
}

void launch_step_attn(const LaunchCtx& ctx, const float* q, int ldq, int nq, int nkv, int hd, float theta,
                      const void* kpool, const void* vpool, const int* block_table, int mpps, int n_pages,
                      const int* seq_lens, int extra, int batch, int max_keys, float* part, float* out) {
  // every sequence attends to seq_lens[b] + extra keys; max_keys bounds that count (host copy).
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  int n_split = step_attn_splits(batch, nkv, max_keys);
  dim3 grid(n_split, nkv, batch);
  size_t smem = (size_t)(MAXG * hd + 4 * MAXG * (hd + 2)) * sizeof(float);
  ++*ctx.n_launch;
  if (ctx.dtype == 0)
    step_attn_kernel<float><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const float*)kpool, (const float*)vpool,
                                                         block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status);
  else
    step_attn_kernel<bf16><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const bf16*)kpool, (const bf16*)vpool,
                                                        block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status);
  if (n_split > 1) {
    ++*ctx.n_launch;
    step_attn_merge_kernel<<<dim3(nq, batch), 64, 0, ctx.st>>>(part, nq, hd, n_split, out);
  }
}

// ---------------------------------------------------------------------------------------
// Generation step: RoPE the new key at position seq_lens[b] and append k, v to the cache.
// ---------------------------------------------------------------------------------------
namespace {
template <class T>
__global__ void step_append_kernel(const float* __restrict__ qkv, int nq, int nkv, int hd, const __grid_constant__ InvFreq inv,
                                   T* __restrict__ kpool, T* __restrict__ vpool, const int* __restrict__ block_table,
                                   int mpps, int n_pages, const int* __restrict__ seq_lens, int* status) {
  int b = blockIdx.x;
  int pos = seq_lens[b];
  int pg = pos / PAGE_TOKENS;
  int page = pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
  if (page < 0 || page >= n_pages) { if (threadIdx.x == 0) dev_flag(status, DEV_BAD_PAGE); return; }
  int row = pos % PAGE_TOKENS, half = hd >> 1;
  const float* kin = qkv + (size_t)b * (nq + 2 * nkv) * hd + (size_t)nq * hd;
  const float* vin = kin + (size_t)nkv * hd;
  for (int i = threadIdx.x; i < nkv * half; i += blockDim.x) {
    int h = i / half, c = i - h * half;
    float sn, cs;
    rope_sincos(pos, inv.f[c], &sn, &cs);
    float x1 = kin[h * hd + c], x2 = kin[h * hd + c + half];
    size_t off = (((size_t)page * nkv + h) * PAGE_TOKENS + row) * hd;
    kpool[off + c] = from_f<T>(x1 * cs - x2 * sn);
    kpool[off + c + half] = from_f<T>(x2 * cs + x1 * sn);
    vpool[off + c] = from_f<T>(vin[h * hd + c]);
    vpool[off + c + half] = from_f<T>(vin[h * hd + c + half]);
  }
}
}  // namespace

void launch_step_append(const LaunchCtx& ctx, const float* qkv, int nq, int nkv, int hd, float theta, void* kpool,
                        void* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int batch) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  ++*ctx.n_launch;
  if (ctx.dtype == 0)
    step_append_kernel<float><<<batch, 128, 0, ctx.st>>>(qkv, nq, nkv, hd, inv, (float*)kpool, (float*)vpool, block_table, mpps, n_pages, seq_lens, ctx.status);
  else
    step_append_kernel<bf16><<<batch, 128, 0, ctx.st>>>(qkv, nq, nkv, hd, inv, (bf16*)kpool, (bf16*)vpool, block_table, mpps, n_pages, seq_lens, ctx.status);
}
