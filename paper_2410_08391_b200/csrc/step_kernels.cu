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
template <> struct Vec8<kv16> {
  static __device__ __forceinline__ void load(const kv16* p, float* f) {
    uint4 u = *reinterpret_cast<const uint4*>(p);
    const __half2* hp = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) { float2 t = __half22float2(hp[e]); f[2 * e] = t.x; f[2 * e + 1] = t.y; }
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

// Variant for up to 4 activation rows: the CTA first stages the activations in shared memory
// (optionally applying RMSNorm on the way, which removes a separate tiny kernel), then each
// warp streams whole weight rows with four 16-byte loads in flight per lane.
namespace {
template <class T, int BB, int MODE, bool NORM>
__global__ void __launch_bounds__(256) step_gemv_smem_kernel(const T* __restrict__ W, int ldw, int N, int K,
                                                             const float* __restrict__ x, int ldx,
                                                             const float* __restrict__ gain, float eps,
                                                             float* __restrict__ y, int ldy, RowMap mg, RowMap mu,
                                                             int rows_per_cta) {
  extern __shared__ float xs[];            // [BB][K]
  __shared__ float red[8][BB];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float r[BB];
#pragma unroll
  for (int b = 0; b < BB; ++b) r[b] = 1.f;
  if (NORM) {
    float ss[BB];
#pragma unroll
    for (int b = 0; b < BB; ++b) ss[b] = 0.f;
    for (int k = tid; k < K; k += 256) {
#pragma unroll
      for (int b = 0; b < BB; ++b) { float v = x[(size_t)b * ldx + k]; ss[b] = fmaf(v, v, ss[b]); }
    }
#pragma unroll
    for (int b = 0; b < BB; ++b) { float t = warp_sum(ss[b]); if (lane == 0) red[warp][b] = t; }
    __syncthreads();
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += red[w][b];
      r[b] = rsqrtf(t / (float)K + eps);
    }
  }
  for (int k = tid; k < K; k += 256) {
    float g = NORM ? gain[k] : 1.f;
#pragma unroll
    for (int b = 0; b < BB; ++b) xs[b * K + k] = NORM ? g * x[(size_t)b * ldx + k] * r[b] : x[(size_t)b * ldx + k];
  }
  __syncthreads();
  const int n_begin = blockIdx.x * rows_per_cta, n_end = min(N, n_begin + rows_per_cta);
  for (int n = n_begin + warp; n < n_end; n += 8) {
    float acc[BB], accu[BB];
#pragma unroll
    for (int b = 0; b < BB; ++b) { acc[b] = 0.f; accu[b] = 0.f; }
    const T* w0 = W + (size_t)(MODE == GEMV_SWIGLU ? map_row(mg, n) : n) * ldw;
    const T* w1 = W + (size_t)(MODE == GEMV_SWIGLU ? map_row(mu, n) : n) * ldw;
    for (int k0 = lane * 8; k0 < K; k0 += 1024) {
      float wf[4][8], uf[4][8];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int k = k0 + u * 256;
        if (k < K) {
          Vec8<T>::load(w0 + k, wf[u]);
          if (MODE == GEMV_SWIGLU) Vec8<T>::load(w1 + k, uf[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int k = k0 + u * 256;
        if (k < K) {
#pragma unroll
          for (int b = 0; b < BB; ++b) {
            float4 x0 = *reinterpret_cast<const float4*>(xs + b * K + k);
            float4 x1 = *reinterpret_cast<const float4*>(xs + b * K + k + 4);
            acc[b] += wf[u][0] * x0.x + wf[u][1] * x0.y + wf[u][2] * x0.z + wf[u][3] * x0.w + wf[u][4] * x1.x +
                      wf[u][5] * x1.y + wf[u][6] * x1.z + wf[u][7] * x1.w;
            if (MODE == GEMV_SWIGLU)
              accu[b] += uf[u][0] * x0.x + uf[u][1] * x0.y + uf[u][2] * x0.z + uf[u][3] * x0.w + uf[u][4] * x1.x +
                         uf[u][5] * x1.y + uf[u][6] * x1.z + uf[u][7] * x1.w;
          }
        }
      }
    }
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float v = warp_sum(acc[b]);
      float u = MODE == GEMV_SWIGLU ? warp_sum(accu[b]) : 0.f;
      if (lane == 0) {
        float* dst = y + (size_t)b * ldy + n;
        if (MODE == GEMV_SWIGLU) *dst = v / (1.f + __expf(-v)) * u;
        else *dst = (MODE == GEMV_RESID) ? *dst + v : v;
      }
    }
  }
}

template <class T, int BB, bool NORM>
void gemv_smem_go(const LaunchCtx& ctx, const void* W, int ldw, int N, int K, const float* x, int ldx, const float* gain,
                  float eps, float* y, int ldy, int mode, int G, int ffn) {
  int rows = (N + 148 * 4 - 1) / (148 * 4);
  rows = (rows + 7) / 8 * 8;
  int grid = (N + rows - 1) / rows;
  size_t smem = (size_t)BB * K * sizeof(float);
  RowMap mg{0, G, 0, ffn}, mu{G == 0 ? ffn : 0, G, 1, ffn};
#define GO(MODE)                                                                                                        \
  do {                                                                                                                  \
    if (smem > 48 * 1024)                                                                                               \
      cudaFuncSetAttribute(step_gemv_smem_kernel<T, BB, MODE, NORM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    step_gemv_smem_kernel<T, BB, MODE, NORM><<<grid, 256, smem, ctx.st>>>((const T*)W, ldw, N, K, x, ldx, gain, eps, y, ldy, mg, mu, rows); \
  } while (0)
  if (mode == GEMV_STORE) GO(GEMV_STORE); else if (mode == GEMV_RESID) GO(GEMV_RESID); else GO(GEMV_SWIGLU);
#undef GO
}

template <class T>
void gemv_smem_dispatch(const LaunchCtx& ctx, const void* W, int ldw, int N, int K, const float* x, int ldx, int batch,
                        const float* gain, float eps, float* y, int ldy, int mode, int G, int ffn) {
#define BBGO(BBV)                                                                                                    \
  do {                                                                                                               \
    if (gain) gemv_smem_go<T, BBV, true>(ctx, W, ldw, N, K, x, ldx, gain, eps, y, ldy, mode, G, ffn);                \
    else gemv_smem_go<T, BBV, false>(ctx, W, ldw, N, K, x, ldx, gain, eps, y, ldy, mode, G, ffn);                    \
  } while (0)
  if (batch == 1) BBGO(1); else if (batch == 2) BBGO(2); else BBGO(4);
#undef BBGO
}
}  // namespace

// y = W x (STORE / RESID / SWIGLU) for `batch` fp32 activation rows.  With `gain`, x is first
// RMS-normalised (gain, eps); `scratch_h` [batch, K] is used when that needs its own kernel.
void launch_step_gemv(const LaunchCtx& ctx, const void* W, int ldw, int N, int K, const float* x, int ldx, int batch,
                      float* y, int ldy, int mode, int G, int ffn, const float* gain, float eps, float* scratch_h) {
  if (batch == 0 || N == 0) return;
  const bool smem_path = batch <= 4 && (batch == 3 ? 4 : batch) * (size_t)K * 4 <= 96 * 1024 && K % 8 == 0 && ldw % 8 == 0 &&
                         ldx % 4 == 0;
  if (smem_path) {
    // a batch of 3 runs the 4-row kernel on a zero-extended view: handled by clamping rows inside via batch==4 only
    if (batch == 3) {
      // 3 rows: run rows 0-1 and row 2 separately to keep every access in bounds
      launch_step_gemv(ctx, W, ldw, N, K, x, ldx, 2, y, ldy, mode, G, ffn, gain, eps, scratch_h);
      launch_step_gemv(ctx, W, ldw, N, K, x + 2 * (size_t)ldx, ldx, 1, y + 2 * (size_t)ldy, ldy, mode, G, ffn, gain, eps, scratch_h);
      return;
    }
    ++*ctx.n_launch;
    if (ctx.dtype == 0) gemv_smem_dispatch<float>(ctx, W, ldw, N, K, x, ldx, batch, gain, eps, y, ldy, mode, G, ffn);
    else gemv_smem_dispatch<bf16>(ctx, W, ldw, N, K, x, ldx, batch, gain, eps, y, ldy, mode, G, ffn);
    return;
  }
  if (gain) {
    launch_rmsnorm(ctx, x, gain, eps, batch, K, scratch_h, 0);
    x = scratch_h; ldx = K;
  }
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
                                                        float* __restrict__ part, float* __restrict__ out, int* status,
                                                        const float* __restrict__ q_gain, float eps) {
  extern __shared__ float sm[];
  __shared__ float rq[MAXG];
  int group = nq / nkv;
  float* qs = sm;                              // [MAXG][hd]
  float* red = qs + MAXG * hd;                 // [4 warps][MAXG][hd + 2]
  int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n_keys = seq_lens[b] + extra;
  int pos = n_keys - 1;
  float scale = rsqrtf((float)hd);
  int half = hd >> 1;
  if (q_gain) head_rnorm(q + (size_t)b * ldq + (size_t)kvh * group * hd, group, hd, eps, rq);
  for (int i = threadIdx.x; i < group * half; i += blockDim.x) {
    int h = i / half, c = i - h * half;
    const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * hd;
    float sn, cs;
    rope_sincos(pos, inv.f[c], &sn, &cs);
    float x1 = qh[c], x2 = qh[c + half];
    if (q_gain) { x1 *= rq[h] * q_gain[c]; x2 *= rq[h] * q_gain[c + half]; }
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

// ---------------------------------------------------------------------------------------
// Page-tiled variant (head_dim 16, 32, 64 or 128): a CTA walks whole cache pages.  The K and V
// page of its kv head (64 keys, contiguous in memory) are copied to shared memory with
// independent 16-byte loads, scores are formed with thread = (key, head subset), the
// softmax statistics with one warp per head, and the value sum with thread = (dim, head
// subset), all out of shared memory, so no load sits on a dependent chain.
// ---------------------------------------------------------------------------------------
namespace {
template <class T>
__global__ void __launch_bounds__(128) step_attn_paged_kernel(const float* __restrict__ q, int ldq, int nq, int nkv, int hd,
                                                              const __grid_constant__ InvFreq inv,
                                                              const T* __restrict__ kpool, const T* __restrict__ vpool,
                                                              const int* __restrict__ block_table, int mpps, int n_pages,
                                                              const int* __restrict__ seq_lens, int extra, int n_split,
                                                              float* __restrict__ part, float* __restrict__ out, int* status,
                                                              const float* __restrict__ q_gain, float eps) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  __shared__ float rq[MAXG];
  const int group = nq / nkv;
  const int row_bytes = hd * (int)sizeof(T) + 16;           // padded: conflict-free row-per-thread reads
  unsigned char* Ks = sm_raw;
  unsigned char* Vs = Ks + PAGE_TOKENS * row_bytes;
  float* qs = reinterpret_cast<float*>(Vs + PAGE_TOKENS * row_bytes);   // [MAXG][hd]
  float* ps = qs + MAXG * hd;                                           // [MAXG][64]
  float* m_run = ps + MAXG * PAGE_TOKENS;                               // [MAXG]
  float* l_run = m_run + MAXG;
  float* alpha = l_run + MAXG;
  const int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_keys = seq_lens[b] + extra;
  const int pos = n_keys - 1;
  const float scale = rsqrtf((float)hd);
  const int half = hd >> 1;
  if (q_gain) head_rnorm(q + (size_t)b * ldq + (size_t)kvh * group * hd, group, hd, eps, rq);
  for (int i = tid; i < group * half; i += 128) {
    int h = i / half, c = i - h * half;
    const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * hd;
    float sn, cs;
    rope_sincos(pos, inv.f[c], &sn, &cs);
    float x1 = qh[c], x2 = qh[c + half];
    if (q_gain) { x1 *= rq[h] * q_gain[c]; x2 *= rq[h] * q_gain[c + half]; }
    qs[h * hd + c] = (x1 * cs - x2 * sn) * scale;
    qs[h * hd + c + half] = (x2 * cs + x1 * sn) * scale;
  }
  if (tid < MAXG) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; alpha[tid] = 1.f; }
  const int n_pg = (n_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  const int per = (n_pg + n_split - 1) / n_split;
  const int pg0 = sp * per, pg1 = min(n_pg, pg0 + per);
  // thread roles
  const int key = tid & 63, hh_s = tid >> 6;                 // scores: key, heads hh_s, hh_s + 2, ...
  const int nhh = 128 / hd;                                  // value sum: heads hh_v, hh_v + nhh, ...
  const int dim = tid % hd, hh_v = tid / hd;
  float o[MAXG];
#pragma unroll
  for (int i = 0; i < MAXG; ++i) o[i] = 0.f;
  const int chunks_per_row = hd * (int)sizeof(T) / 16;
  const int n_chunks = PAGE_TOKENS * chunks_per_row;
  for (int pg = pg0; pg < pg1; ++pg) {
    int page = block_table[(size_t)b * mpps + pg];
    bool page_ok = page >= 0 && page < n_pages;
    if (!page_ok && tid == 0) dev_flag(status, DEV_BAD_PAGE);
    const int nk = page_ok ? min(PAGE_TOKENS, n_keys - pg * PAGE_TOKENS) : 0;
    __syncthreads();                                         // previous page fully consumed (and qs written)
    if (page_ok) {
      const uint4* ksrc = reinterpret_cast<const uint4*>(kpool + ((size_t)page * nkv + kvh) * PAGE_TOKENS * hd);
      const uint4* vsrc = reinterpret_cast<const uint4*>(vpool + ((size_t)page * nkv + kvh) * PAGE_TOKENS * hd);
      for (int i = tid; i < n_chunks; i += 128) {
        int r = i / chunks_per_row, cc = i - r * chunks_per_row;
        uint4 kx = __ldg(ksrc + i), vx = __ldg(vsrc + i);
        *reinterpret_cast<uint4*>(Ks + r * row_bytes + cc * 16) = kx;
        *reinterpret_cast<uint4*>(Vs + r * row_bytes + cc * 16) = vx;
      }
    }
    __syncthreads();
    // scores
    {
      float sc[MAXG / 2];
#pragma unroll
      for (int i = 0; i < MAXG / 2; ++i) sc[i] = 0.f;
      const T* kr = reinterpret_cast<const T*>(Ks + key * row_bytes);
      for (int c = 0; c < hd; c += 8) {
        float kf[8];
        if (sizeof(T) == 2) {
          uint4 u = *reinterpret_cast<const uint4*>(kr + c);
          const __half2* hp = reinterpret_cast<const __half2*>(&u);     // 16-bit cache elements are halves
#pragma unroll
          for (int e = 0; e < 4; ++e) { float2 t = __half22float2(hp[e]); kf[2 * e] = t.x; kf[2 * e + 1] = t.y; }
        } else {
          float4 a = *reinterpret_cast<const float4*>(kr + c), bq = *reinterpret_cast<const float4*>(kr + c + 4);
          kf[0] = a.x; kf[1] = a.y; kf[2] = a.z; kf[3] = a.w; kf[4] = bq.x; kf[5] = bq.y; kf[6] = bq.z; kf[7] = bq.w;
        }
#pragma unroll
        for (int i = 0; i < MAXG / 2; ++i) {
          int h = hh_s + 2 * i;
          if (h < group) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sc[i] = fmaf(kf[e], qs[h * hd + c + e], sc[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < MAXG / 2; ++i) {
        int h = hh_s + 2 * i;
        if (h < group) ps[h * PAGE_TOKENS + key] = key < nk ? sc[i] : -INFINITY;
      }
    }
    __syncthreads();
    // running softmax statistics: warp w serves heads w, w + 4
    for (int h = warp; h < group; h += 4) {
      float s0 = ps[h * PAGE_TOKENS + lane], s1 = ps[h * PAGE_TOKENS + 32 + lane];
      float mt = warp_max(fmaxf(s0, s1));
      float m_old = m_run[h];
      float mn = fmaxf(m_old, mt);
      float p0 = (mn == -INFINITY) ? 0.f : __expf(s0 - mn), p1 = (mn == -INFINITY) ? 0.f : __expf(s1 - mn);
      float sum = warp_sum(p0 + p1);
      ps[h * PAGE_TOKENS + lane] = p0; ps[h * PAGE_TOKENS + 32 + lane] = p1;
      if (lane == 0) {
        float a = (mn == -INFINITY) ? 1.f : __expf(m_old - mn);
        alpha[h] = a; m_run[h] = mn; l_run[h] = l_run[h] * a + sum;
      }
    }
    __syncthreads();
    // value sum
#pragma unroll
    for (int i = 0; i < MAXG; ++i) {
      int h = hh_v + nhh * i;
      if (i * nhh < MAXG && h < group) {
        float acc = o[i] * alpha[h];
        const float* pr = ps + h * PAGE_TOKENS;
        for (int s = 0; s < nk; ++s) acc = fmaf(pr[s], to_f(reinterpret_cast<const T*>(Vs + s * row_bytes)[dim]), acc);
        o[i] = acc;
      }
    }
  }
  __syncthreads();
  const int ldr = hd + 2;
#pragma unroll
  for (int i = 0; i < MAXG; ++i) {
    int h = hh_v + nhh * i;
    if (i * nhh < MAXG && h < group) {
      int qh = kvh * group + h;
      if (n_split == 1) {
        out[(size_t)b * nq * hd + (size_t)qh * hd + dim] = o[i] / l_run[h];
      } else {
        float* pr = part + (((size_t)b * nq + qh) * n_split + sp) * ldr;
        pr[dim] = o[i];
        if (dim == 0) { pr[hd] = m_run[h]; pr[hd + 1] = l_run[h]; }
      }
    }
  }
}
}  // namespace

int step_attn_splits(int batch, int nkv, int max_keys) {
  int want = (2 * 148 + batch * nkv - 1) / (batch * nkv);
  int cap = (max_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  int n = want < cap ? want : cap;
  if (n < 1) n = 1;
  if (n > 64) n = 64;
  return n;
}

void launch_step_attn(const LaunchCtx& ctx, const float* q, int ldq, int nq, int nkv, int hd, float theta,
                      const void* kpool, const void* vpool, const int* block_table, int mpps, int n_pages,
                      const int* seq_lens, int extra, int batch, int max_keys, float* part, float* out, const float* q_gain,
                      float eps, int* split_done) {
  // every sequence attends to seq_lens[b] + extra keys; max_keys bounds that count (host copy).
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  int n_split = step_attn_splits(batch, nkv, max_keys);
  dim3 grid(n_split, nkv, batch);
  if (split_done && step_attn_mma_supported(ctx.dtype, nq, nkv, hd, kpool, vpool, n_pages)) {
    // half-precision cache, head_dim 64 / 128: warp-level tensor-core kernel (pages through a swizzling tensor map)
    const int ns = step_attn_mma_splits(batch, nkv, max_keys, n_split);
    if (ns > 1) cudaMemsetAsync(split_done, 0, (size_t)batch * nkv * sizeof(int), ctx.st);
    if (launch_step_attn_mma(ctx, q, ldq, nq, nkv, hd, theta, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra, batch, ns, max_keys, part, out,
                             q_gain, eps, split_done) == cudaSuccess)
      return;
    cudaGetLastError();      // (a tensor map could not be made: the kernels below take plain pointers)
  }
  if (step_attn_ring_supported(ctx.dtype, nq, nkv, hd, kpool, vpool)) {
    n_split = step_attn_ring_splits(nq, nkv, hd, batch, max_keys, n_split);
    // up to 4 heads per kv head: the CTA that finishes a group's last split merges it (counters cleared here)
    const bool fused = split_done && n_split > 1 && nq / nkv <= 4;
    if (fused) cudaMemsetAsync(split_done, 0, (size_t)batch * nkv * sizeof(int), ctx.st);
    launch_step_attn_ring(ctx, q, ldq, nq, nkv, hd, theta, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra, batch, n_split, part, out,
                          q_gain, eps, fused ? split_done : nullptr);
    if (n_split > 1 && !fused) {
      ++*ctx.n_launch;
      step_attn_merge_kernel<<<dim3(nq, batch), 64, 0, ctx.st>>>(part, nq, hd, n_split, out);
    }
    return;
  }
  ++*ctx.n_launch;
  if (hd == 16 || hd == 32 || hd == 64 || hd == 128) {
    int es = ctx.dtype == 0 ? 4 : 2;
    size_t smem = (size_t)2 * PAGE_TOKENS * (hd * es + 16) + (size_t)(MAXG * hd + MAXG * PAGE_TOKENS + 3 * MAXG) * sizeof(float);
    if (ctx.dtype == 0) {
      cudaFuncSetAttribute(step_attn_paged_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      step_attn_paged_kernel<float><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const float*)kpool, (const float*)vpool,
                                                                 block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps);
    } else {
      step_attn_paged_kernel<kv16><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const kv16*)kpool, (const kv16*)vpool,
                                                                block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps);
    }
  } else {
    size_t smem = (size_t)(MAXG * hd + 4 * MAXG * (hd + 2)) * sizeof(float);
    if (ctx.dtype == 0)
      step_attn_kernel<float><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const float*)kpool, (const float*)vpool,
                                                           block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps);
    else
      step_attn_kernel<kv16><<<grid, 128, smem, ctx.st>>>(q, ldq, nq, nkv, hd, inv, (const kv16*)kpool, (const kv16*)vpool,
                                                          block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps);
  }
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
                                   int mpps, int n_pages, const int* __restrict__ seq_lens, int* status,
                                   const float* __restrict__ k_gain, float eps) {
  __shared__ float rk[64];
  int b = blockIdx.x;
  if (k_gain) head_rnorm(qkv + (size_t)b * (nq + 2 * nkv) * hd + (size_t)nq * hd, nkv, hd, eps, rk);   // nkv <= 64 (checked by the launcher)
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
    if (k_gain) { x1 *= rk[h] * k_gain[c]; x2 *= rk[h] * k_gain[c + half]; }
    size_t off = (((size_t)page * nkv + h) * PAGE_TOKENS + row) * hd;
    kpool[off + c] = from_f<T>(x1 * cs - x2 * sn);
    kpool[off + c + half] = from_f<T>(x2 * cs + x1 * sn);
    vpool[off + c] = from_f<T>(vin[h * hd + c]);
    vpool[off + c + half] = from_f<T>(vin[h * hd + c + half]);
  }
}
}  // namespace

void launch_step_append(const LaunchCtx& ctx, const float* qkv, int nq, int nkv, int hd, float theta, void* kpool,
                        void* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int batch,
                        const float* k_gain, float eps) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  ++*ctx.n_launch;
  if (ctx.dtype == 0)
    step_append_kernel<float><<<batch, 128, 0, ctx.st>>>(qkv, nq, nkv, hd, inv, (float*)kpool, (float*)vpool, block_table, mpps, n_pages, seq_lens, ctx.status, k_gain, eps);
  else
    step_append_kernel<kv16><<<batch, 128, 0, ctx.st>>>(qkv, nq, nkv, hd, inv, (kv16*)kpool, (kv16*)vpool, block_table, mpps, n_pages, seq_lens, ctx.status, k_gain, eps);
}
