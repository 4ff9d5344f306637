// Small memory-bound kernels: weight packing, token index, embedding gather, RMSNorm,
// RoPE, SwiGLU, argmax.  All arithmetic in fp32 (RoPE angles in fp64).
#include <math.h>

#include "common.cuh"

#define LAUNCH_COUNT(ctx) (++*(ctx).n_launch)

static inline int grid_for(size_t n, int threads) {
  size_t g = (n + threads - 1) / threads;
  size_t cap = 148 * 16;
  return (int)(g < cap ? g : cap);
}

void fill_inv_freq(InvFreq* f, int hd, float theta) {
  for (int c = 0; c < hd / 2 && c < 64; ++c) f->f[c] = pow((double)theta, -2.0 * c / hd);
}

// ---------------------------------------------------------------------------------------
// weight packing: dst[map(r), c] = convert(src[r, c])
// ---------------------------------------------------------------------------------------
template <class S, class D>
__global__ void pack_rows_kernel(const S* __restrict__ src, D* __restrict__ dst, int rows, int cols,
                                 RowMap map) {
  size_t n = (size_t)rows * cols;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    int r = (int)(i / cols), c = (int)(i - (size_t)r * cols);
    dst[(size_t)map_row(map, r) * cols + c] = from_f<D>(to_f(src[i]));
  }
}

void launch_pack_rows(const LaunchCtx& ctx, const void* src, int sdt, void* dst, int ddt, int rows, int cols,
                      RowMap map) {
  size_t n = (size_t)rows * cols;
  if (n == 0) return;
  int grid = grid_for(n, 256);
  LAUNCH_COUNT(ctx);
  if (sdt == 0 && ddt == 0) pack_rows_kernel<float, float><<<grid, 256, 0, ctx.st>>>((const float*)src, (float*)dst, rows, cols, map);
  else if (sdt == 0 && ddt == 1) pack_rows_kernel<float, bf16><<<grid, 256, 0, ctx.st>>>((const float*)src, (bf16*)dst, rows, cols, map);
  else if (sdt == 1 && ddt == 0) pack_rows_kernel<bf16, float><<<grid, 256, 0, ctx.st>>>((const bf16*)src, (float*)dst, rows, cols, map);
  else if (sdt == 0 && ddt == 2) pack_rows_kernel<float, kv16><<<grid, 256, 0, ctx.st>>>((const float*)src, (kv16*)dst, rows, cols, map);
  else if (sdt == 1 && ddt == 2) pack_rows_kernel<bf16, kv16><<<grid, 256, 0, ctx.st>>>((const bf16*)src, (kv16*)dst, rows, cols, map);
  else pack_rows_kernel<bf16, bf16><<<grid, 256, 0, ctx.st>>>((const bf16*)src, (bf16*)dst, rows, cols, map);
}

// ---------------------------------------------------------------------------------------
// token index: for every packed token t its position in its sequence and its cache slot
// ---------------------------------------------------------------------------------------
struct CuSeq { int cu[257]; };

__global__ void build_index_kernel(const __grid_constant__ CuSeq cs, int batch, int total, int* cu_dev,
                                   int* tok_pos, int* tok_slot, int* last_tok_idx,
                                   const int* __restrict__ block_table, int mpps, int n_pages,
                                   int* seq_lens, int* status) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t <= batch) cu_dev[t] = cs.cu[t];
  if (t < batch) {
    last_tok_idx[t] = cs.cu[t + 1] - 1;
    seq_lens[t] = cs.cu[t + 1] - cs.cu[t];
  }
  if (t >= total) return;
  int lo = 0, hi = batch;   // largest b with cu[b] <= t
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cs.cu[mid] <= t) lo = mid; else hi = mid;
  }
  int pos = t - cs.cu[lo];
  tok_pos[t] = pos;
  int pg = pos / PAGE_TOKENS;
  int slot = -1;
  if (pg < mpps) {
    int page = block_table[(size_t)lo * mpps + pg];
    if (page >= 0 && page < n_pages) slot = page * PAGE_TOKENS + (pos % PAGE_TOKENS);
  }
  if (slot < 0) dev_flag(status, DEV_BAD_PAGE);
  tok_slot[t] = slot;
}

void launch_build_index(const LaunchCtx& ctx, const int* cu_host, int batch, int total, int* cu_dev,
                        int* tok_pos, int* tok_slot, int* last_tok_idx, const int* block_table,
                        int mpps, int n_pages, int* seq_lens) {
  CuSeq cs;
  for (int i = 0; i <= batch; ++i) cs.cu[i] = cu_host[i];
  for (int i = batch + 1; i < 257; ++i) cs.cu[i] = cu_host[batch];
  int n = total > batch + 1 ? total : batch + 1;
  LAUNCH_COUNT(ctx);
  build_index_kernel<<<(n + 255) / 256, 256, 0, ctx.st>>>(cs, batch, total, cu_dev, tok_pos, tok_slot,
                                                          last_tok_idx, block_table, mpps, n_pages,
                                                          seq_lens, ctx.status);
}

// ---------------------------------------------------------------------------------------
// embedding gather: x[r, :] = table[tokens[idx(r)], :] as fp32
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void embed_kernel(const int* __restrict__ tokens, const int* __restrict__ gather_idx,
                             const T* __restrict__ table, int vocab, int d, float* __restrict__ x, int* status) {
  int r = blockIdx.x;
  int tok = tokens[gather_idx ? gather_idx[r] : r];
  bool ok = tok >= 0 && tok < vocab;
  if (!ok && threadIdx.x == 0) dev_flag(status, DEV_BAD_TOKEN);
  const T* src = table + (size_t)(ok ? tok : 0) * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = ok ? to_f(src[c]) : 0.f;
}

void launch_embed(const LaunchCtx& ctx, const int* tokens, const int* gather_idx, int n_rows, const void* table,
                  int vocab, int d, float* x) {
  if (n_rows == 0) return;
  LAUNCH_COUNT(ctx);
  if (ctx.dtype == 0) embed_kernel<float><<<n_rows, 128, 0, ctx.st>>>(tokens, gather_idx, (const float*)table, vocab, d, x, ctx.status);
  else embed_kernel<bf16><<<n_rows, 128, 0, ctx.st>>>(tokens, gather_idx, (const bf16*)table, vocab, d, x, ctx.status);
}

// ---------------------------------------------------------------------------------------
// RMSNorm: out = gain * x / sqrt(mean(x^2) + eps), one warp per row
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ gain, float eps, int rows,
                               int d, T* __restrict__ out, T* __restrict__ out_lo) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  pdl_trigger();
  pdl_wait();
  if (row >= rows) return;
  const float* xr = x + (size_t)row * d;
  float ss = 0.f;
  for (int c = lane; c < d; c += 32) { float v = xr[c]; ss += v * v; }
  ss = warp_sum(ss);
  float r = rsqrtf(ss / (float)d + eps);
  for (int c = lane; c < d; c += 32) {
    float v = gain[c] * xr[c] * r;
    T hi = from_f<T>(v);
    out[(size_t)row * d + c] = hi;
    if (out_lo) out_lo[(size_t)row * d + c] = from_f<T>(v - to_f(hi));
  }
}

// out_half: the 16-bit output is written as IEEE halves (and no remainder)
void launch_rmsnorm(const LaunchCtx& ctx, const float* x, const float* gain, float eps, int rows, int d, void* out,
                    int out_dtype, void* out_lo, bool out_half) {
  if (rows == 0) return;
  LAUNCH_COUNT(ctx);
  int grid = (rows + 7) / 8;
  if (out_dtype != 0 && out_half) launch_overlapped(rmsnorm_kernel<kv16>, dim3(grid), dim3(256), 0, ctx.st, x, gain, eps, rows, d, (kv16*)out, (kv16*)nullptr);
  else if (out_dtype == 0) launch_overlapped(rmsnorm_kernel<float>, dim3(grid), dim3(256), 0, ctx.st, x, gain, eps, rows, d, (float*)out, (float*)nullptr);
  else launch_overlapped(rmsnorm_kernel<bf16>, dim3(grid), dim3(256), 0, ctx.st, x, gain, eps, rows, d, (bf16*)out, (bf16*)out_lo);
}

// ---------------------------------------------------------------------------------------
// RoPE (rotate-half pairing) on an fp32 projection output, then the store in the run dtype;
// K and V heads also leave their bf16 rounding remainder (lo part) for the predictor.
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void rope_split_kernel(const float* __restrict__ in, int ld_in, int rows, int n_heads, int n_heads_rot,
                                  int hd, const int* __restrict__ tok_pos, const __grid_constant__ InvFreq inv,
                                  T* __restrict__ out, int ld_out, T* __restrict__ out_lo, int ld_lo,
                                  int lo_head_begin, int n_q_heads, const float* __restrict__ q_gain,
                                  const float* __restrict__ k_gain, float eps) {
  int half = hd >> 1;
  size_t n = (size_t)rows * n_heads * half;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    int c = (int)(i % half);
    size_t rh = i / half;
    int h = (int)(rh % n_heads);
    int r = (int)(rh / n_heads);
    const float* p = in + (size_t)r * ld_in + (size_t)h * hd + c;
    float y1 = p[0], y2 = p[half];
    if (h < n_heads_rot) {
      const float* gain = h < n_q_heads ? q_gain : k_gain;
      if (gain) {   // query / key norm over the head (this generic path recomputes the head's mean square per element)
        const float* hp = in + (size_t)r * ld_in + (size_t)h * hd;
        float ss = 0.f;
        for (int e = 0; e < hd; ++e) ss = fmaf(hp[e], hp[e], ss);
        const float rn = rsqrtf(ss / (float)hd + eps);
        y1 *= rn * gain[c]; y2 *= rn * gain[c + half];
      }
      float sn, cs;
      rope_sincos(tok_pos[r], inv.f[c], &sn, &cs);
      float x1 = y1, x2 = y2;
      y1 = x1 * cs - x2 * sn;
      y2 = x2 * cs + x1 * sn;
    }
    T h1 = from_f<T>(y1), h2 = from_f<T>(y2);
    T* o = out + (size_t)r * ld_out + (size_t)h * hd + c;
    o[0] = h1; o[half] = h2;
    if (out_lo && h >= lo_head_begin) {
      T* l = out_lo + (size_t)r * ld_lo + (size_t)(h - lo_head_begin) * hd + c;
      l[0] = from_f<T>(y1 - to_f(h1));
      l[half] = from_f<T>(y2 - to_f(h2));
    }
  }
}

void launch_rope_split(const LaunchCtx& ctx, const float* in, int ld_in, int rows, int n_heads, int n_heads_rot, int hd,
                       const int* tok_pos, float theta, void* out, int ld_out, void* out_lo, int ld_lo,
                       int lo_head_begin, int n_q_heads, const float* q_gain, const float* k_gain, float eps) {
  size_t n = (size_t)rows * n_heads * (hd / 2);
  if (n == 0) return;
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  int grid = grid_for(n, 256);
  LAUNCH_COUNT(ctx);
  if (ctx.dtype == 0)
    rope_split_kernel<float><<<grid, 256, 0, ctx.st>>>(in, ld_in, rows, n_heads, n_heads_rot, hd, tok_pos, inv, (float*)out, ld_out, (float*)nullptr, 0, 0, n_q_heads, q_gain, k_gain, eps);
  else
    rope_split_kernel<bf16><<<grid, 256, 0, ctx.st>>>(in, ld_in, rows, n_heads, n_heads_rot, hd, tok_pos, inv, (bf16*)out, ld_out, (bf16*)out_lo, ld_lo, lo_head_begin, n_q_heads, q_gain, k_gain, eps);
}

// ---------------------------------------------------------------------------------------
// SwiGLU on the packed gate/up GEMM output: act[r, c] = silu(gate_c) * up_c
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void swiglu_kernel(const T* __restrict__ gu, int rows, int ffn, RowMap mg, RowMap mu, T* __restrict__ act) {
  size_t n = (size_t)rows * ffn;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    int r = (int)(i / ffn), c = (int)(i - (size_t)r * ffn);
    float g = to_f(gu[(size_t)r * 2 * ffn + map_row(mg, c)]);
    float u = to_f(gu[(size_t)r * 2 * ffn + map_row(mu, c)]);
    act[i] = from_f<T>(g / (1.f + __expf(-g)) * u);
  }
}

void launch_swiglu(const LaunchCtx& ctx, const void* gu, int rows, int ffn, int G, void* act) {
  size_t n = (size_t)rows * ffn;
  if (n == 0) return;
  RowMap mg{0, G, 0, ffn}, mu{G == 0 ? ffn : 0, G, 1, ffn};
  int grid = grid_for(n, 256);
  LAUNCH_COUNT(ctx);
  if (ctx.dtype == 0) swiglu_kernel<float><<<grid, 256, 0, ctx.st>>>((const float*)gu, rows, ffn, mg, mu, (float*)act);
  else swiglu_kernel<bf16><<<grid, 256, 0, ctx.st>>>((const bf16*)gu, rows, ffn, mg, mu, (bf16*)act);
}

// ---------------------------------------------------------------------------------------
// argmax per row, lowest index on ties
// ---------------------------------------------------------------------------------------
__global__ void argmax_kernel(const float* __restrict__ logits, int vocab, int* __restrict__ out) {
  const float* row = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
    float v = row[c];
    if (v > best || (v == best && c < bi)) { best = v; bi = c; }
  }
  __shared__ float sv[256];
  __shared__ int si[256];
  sv[threadIdx.x] = best; si[threadIdx.x] = bi;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) {
      float v = sv[threadIdx.x + s]; int i = si[threadIdx.x + s];
      if (v > sv[threadIdx.x] || (v == sv[threadIdx.x] && i < si[threadIdx.x])) { sv[threadIdx.x] = v; si[threadIdx.x] = i; }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) out[blockIdx.x] = si[0] == 0x7fffffff ? 0 : si[0];
}

void launch_argmax(const LaunchCtx& ctx, const float* logits, int batch, int vocab, int* out) {
  LAUNCH_COUNT(ctx);
  argmax_kernel<<<batch, 256, 0, ctx.st>>>(logits, vocab, out);
}

__global__ void add_int_kernel(int* v, int n, int delta) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) v[i] += delta;
}
void launch_add_int(const LaunchCtx& ctx, int* v, int n, int delta) {
  LAUNCH_COUNT(ctx);
  add_int_kernel<<<(n + 255) / 256, 256, 0, ctx.st>>>(v, n, delta);
}
