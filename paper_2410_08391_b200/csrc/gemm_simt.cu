// CUDA-core GEMM  D[M,N] = A[M,K] * W[N,K]^T  with fp32 accumulation, and CUDA-core
// causal attention.  They are the fp32-mode kernels (no tensor-core type multiplies in
// fp32) and the generic path for shapes the tensor-core kernels do not take.
#include "common.cuh"

namespace {
constexpr int BM = 64, BN = 64, BK = 16;

// 64x64 tile, K step 16, 256 threads, 4x4 outputs per thread.
template <class T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const T* __restrict__ A = (const T*)g.A;
  const T* __restrict__ W = (const T*)g.W;
  int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const T* __restrict__ A2 = (g.A2 && n0 + BN > g.split_begin) ? (const T*)g.A2 : nullptr;
  int tid = threadIdx.x;
  int tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  int lr = tid >> 2, lk = (tid & 3) * 4;   // each thread stages 4 consecutive k of one row
  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int k = k0 + lk + i;
      int am = m0 + lr, wn = n0 + lr;
      float av = (am < g.M && k < g.K) ? to_f(A[(size_t)am * g.lda + k]) : 0.f;
      if (A2 && am < g.M && k < g.K) av += to_f(A2[(size_t)am * g.lda2 + k]);
      As[lk + i][lr] = av;
      Ws[lk + i][lr] = (wn < g.N && k < g.K) ? to_f(W[(size_t)wn * g.ldw + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
    int slot = 0;
    if (EPI == EPI_PAGED) { slot = g.paged.tok_slot[m]; if (slot < 0) continue; }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float v = acc[i][j];
      if (EPI == EPI_STORE) {
        ((T*)g.C)[(size_t)m * g.ldc + n] = from_f<T>(v);
      } else if (EPI == EPI_STORE32) {
        ((float*)g.C)[(size_t)m * g.ldc + n] = v;
      } else if (EPI == EPI_RESID) {
        g.X[(size_t)m * g.ldx + n] += v;
      } else {
        const PagedOut& p = g.paged;
        int s = 0;
        while (s + 1 < p.n_seg && n >= p.col0[s + 1]) ++s;
        int c = n - p.col0[s];
        int head = c / p.head_dim, dim = c - head * p.head_dim;
        if (p.bias) v += p.bias[n];
        int page = slot / PAGE_TOKENS, row = slot - page * PAGE_TOKENS;
        size_t off = (((size_t)page * p.n_kv[s] + head) * PAGE_TOKENS + row) * p.head_dim + dim;
        typedef typename KvOf<T>::type KT;     // cache element of this run dtype
        ((KT*)p.pool[s])[off] = from_f<KT>(v);
      }
    }
  }
}
}  // namespace

void launch_gemm_simt(const LaunchCtx& ctx, const GemmArgs& g, int epi) {
  if (g.M == 0 || g.N == 0) return;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  ++*ctx.n_launch;
#define GO(T, E) gemm_simt_kernel<T, E><<<grid, 256, 0, ctx.st>>>(g)
  if (ctx.dtype == 0) {
    if (epi == EPI_STORE) GO(float, EPI_STORE); else if (epi == EPI_RESID) GO(float, EPI_RESID); else if (epi == EPI_STORE32) GO(float, EPI_STORE32); else GO(float, EPI_PAGED);
  } else {
    if (epi == EPI_STORE) GO(bf16, EPI_STORE); else if (epi == EPI_RESID) GO(bf16, EPI_RESID); else if (epi == EPI_STORE32) GO(bf16, EPI_STORE32); else GO(bf16, EPI_PAGED);
  }
#undef GO
}

// ---------------------------------------------------------------------------------------
// CUDA-core causal GQA attention over a ragged batch.  One CTA = 8 warps = 8 consecutive
// queries of one sequence and one q head; keys and values are staged through shared
// memory 64 at a time; online softmax in fp32 (lane = key for scores, lane = dim for PV).
// ---------------------------------------------------------------------------------------
namespace {
constexpr int AQ = 8, AKV = 64;

template <class T>
__global__ void __launch_bounds__(256) attn_prefill_simt_kernel(const T* __restrict__ qkv, int ld, int nq, int nkv, int hd,
                                                                const int* __restrict__ cu, int batch, T* __restrict__ out,
                                                                int ldo, float scale) {
  extern __shared__ float smem[];
  int ldk = hd + 1;
  float* Ks = smem;                       // [AKV][hd+1]
  float* Vs = Ks + AKV * ldk;             // [AKV][hd+1]
  float* Qs = Vs + AKV * ldk;             // [AQ][hd]
  __shared__ int s_b, s_q0;
  if (threadIdx.x == 0) {
    int blk = blockIdx.x, b = 0;
    for (; b < batch; ++b) {
      int nb = (cu[b + 1] - cu[b] + AQ - 1) / AQ;
      if (blk < nb) break;
      blk -= nb;
    }
    s_b = b; s_q0 = blk * AQ;
  }
  __syncthreads();
  int b = s_b;
  if (b >= batch) return;
  int head = blockIdx.y, kvh = head / (nq / nkv);
  int base = cu[b], L = cu[b + 1] - base;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int qi = s_q0 + warp;                   // query position of this warp
  bool qok = qi < L;
  if (qok)
    for (int c = lane; c < hd; c += 32) Qs[warp * hd + c] = to_f(qkv[(size_t)(base + qi) * ld + head * hd + c]) * scale;
  int koff = nq * hd + kvh * hd, voff = (nq + nkv) * hd + kvh * hd;
  float o[4] = {0.f, 0.f, 0.f, 0.f};
  float m = -INFINITY, l = 0.f;
  int kmax = min(L, s_q0 + AQ);           // keys any query of this CTA can see
  for (int k0 = 0; k0 < kmax; k0 += AKV) {
    __syncthreads();
    for (int i = threadIdx.x; i < AKV * hd; i += blockDim.x) {
      int s = i / hd, c = i - s * hd;
      int ks = k0 + s;
      float kx = 0.f, vx = 0.f;
      if (ks < kmax) {
        kx = to_f(qkv[(size_t)(base + ks) * ld + koff + c]);
        vx = to_f(qkv[(size_t)(base + ks) * ld + voff + c]);
      }
      Ks[s * ldk + c] = kx; Vs[s * ldk + c] = vx;
    }
    __syncthreads();
    if (!qok) continue;
    float sc[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      int s = lane + 32 * h, ks = k0 + s;
      float a = 0.f;
      for (int c = 0; c < hd; ++c) a = fmaf(Qs[warp * hd + c], Ks[s * ldk + c], a);
      sc[h] = (ks <= qi && ks < L) ? a : -INFINITY;
    }
    float mt = warp_max(fmaxf(sc[0], sc[1]));
    if (mt == -INFINITY) continue;
    float mn = fmaxf(m, mt);
    float alpha = __expf(m - mn);
    float p0 = __expf(sc[0] - mn), p1 = __expf(sc[1] - mn);
    l = l * alpha + warp_sum(p0 + p1);
    m = mn;
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] *= alpha;
    for (int s = 0; s < AKV; ++s) {
      float p = __shfl_sync(0xffffffffu, s < 32 ? p0 : p1, s & 31);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int c = lane + 32 * i;
        if (c < hd) o[i] = fmaf(p, Vs[s * ldk + c], o[i]);
      }
    }
  }
  if (qok) {
    float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int c = lane + 32 * i;
      if (c < hd) out[(size_t)(base + qi) * ldo + head * hd + c] = from_f<T>(o[i] * inv);
    }
  }
}
}  // namespace

void launch_attn_prefill_simt(const LaunchCtx& ctx, const void* qkv, int ld, int nq, int nkv, int hd, const int* cu_dev,
                              int batch, int total, void* out, int ldo) {
  if (total == 0) return;
  int n_blk = (total + AQ - 1) / AQ + batch;   // upper bound on sum_b ceil(L_b / AQ)
  size_t smem = (size_t)(2 * AKV * (hd + 1) + AQ * hd) * sizeof(float);
  dim3 grid(n_blk, nq);
  float scale = 1.f / sqrtf((float)hd);
  ++*ctx.n_launch;
  if (ctx.dtype == 0) {
    cudaFuncSetAttribute(attn_prefill_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    attn_prefill_simt_kernel<float><<<grid, 256, smem, ctx.st>>>((const float*)qkv, ld, nq, nkv, hd, cu_dev, batch, (float*)out, ldo, scale);
  } else {
    cudaFuncSetAttribute(attn_prefill_simt_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    attn_prefill_simt_kernel<bf16><<<grid, 256, smem, ctx.st>>>((const bf16*)qkv, ld, nq, nkv, hd, cu_dev, batch, (bf16*)out, ldo, scale);
  }
}
