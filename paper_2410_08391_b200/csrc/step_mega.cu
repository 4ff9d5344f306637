// The base model's single-token step as ONE persistent cooperative kernel (batch <= 4).
//
// A step is ~170 dependent, bandwidth-bound operations of a few microseconds each; as separate
// kernels their launch and ramp-up latency is several times the time the weights need to stream
// from HBM.  Here one CTA of 16 warps per SM stays resident for the whole step.  The operations
// become phases separated by a grid-wide barrier (one global counter, bounded spin):
//   per layer:  q(kv) projection (RMSNorm fused) | [append k,v] | attention over cache pages |
//               (key-range splits merged by the CTA that finishes a group's last split) | O projection + residual | gate/up + SwiGLU (RMSNorm
//               fused) | down projection + residual;   then LM head (final RMSNorm fused) + argmax.
// Weights never pass through registers on their way from HBM: every warp owns a small ring of
// shared-memory slots that it fills with bulk asynchronous copies (cp.async.bulk, completion on
// an mbarrier) of the weight rows it will need, in schedule order.  The schedule is static, so a
// warp keeps its ring full ACROSS phase boundaries: while the SMs wait at a barrier, or run
// attention, the first rows of the next projection are already landing.  About 190 KB per SM are
// in flight, which is what HBM latency times bandwidth asks for.
#include <math.h>

#include "common.cuh"
#include "tc_ptx.cuh"
#include "step_mega.h"

namespace {
using namespace tcp;

constexpr int NT = 512;                 // threads per CTA, one CTA per SM
constexpr int NW = NT / 32;
constexpr int MAXG = 8;
constexpr int NSLOT = 3;                // ring slots per warp


// Grid-wide barrier: every CTA adds one to *counter and waits until it reaches `target`.
// Returns false when the wait ran out (or some role already gave up): the caller leaves.
__device__ __forceinline__ bool grid_barrier(unsigned* counter, unsigned target, int* status, volatile int* s_abort, int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = *s_abort ? 0 : 1;
    __threadfence();
    atomicAdd(counter, 1u);
    unsigned it = 0;
    while (ok) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
      if (v >= target) break;
      if (++it > SPIN_LIMIT) { dev_flag(status, DEV_TIMEOUT); ok = 0; break; }
      if ((it & 255u) == 0u && *reinterpret_cast<volatile int*>(status) == DEV_TIMEOUT) { ok = 0; break; }
    }
    if (ok && *reinterpret_cast<volatile int*>(status) == DEV_TIMEOUT) ok = 0;
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag != 0;
}

struct GemvDesc {
  const void* W; int N, K;          // rows, row length (= leading dimension)
  int mode;                         // GEMV_STORE / GEMV_RESID / GEMV_SWIGLU
  int G, ffn;                       // SwiGLU row interleave
};

// The projection phases in schedule order: 4 per layer (q(kv), O, gate/up, down), then the LM head.
__device__ __forceinline__ GemvDesc stream_desc(const MegaParams& p, int s) {
  if (s >= 4 * p.n_layers) return GemvDesc{p.lm_head, p.vocab, p.d, GEMV_STORE, 0, 0};
  const MegaLayer& L = p.layers[s >> 2];
  switch (s & 3) {
    case 0: return GemvDesc{L.wqkv, p.generation ? L.nqkv : L.dq, p.d, GEMV_STORE, 0, 0};
    case 1: return GemvDesc{L.wo, p.d, L.dq, GEMV_RESID, 0, 0};
    case 2: return GemvDesc{L.wgu, L.ffn, p.d, GEMV_SWIGLU, L.G, L.ffn};
    default: return GemvDesc{L.wd, p.d, L.ffn, GEMV_RESID, 0, 0};
  }
}

// A warp's weight stream: chunks (pieces of rows, at most `slot_bytes` each) in the order the
// warp consumes them, over all projection phases of the step.  The producer cursor walks the
// static schedule (phase, output row, gate/up half, piece of the row) ahead of the consumer.
struct WarpStream {
  int ps;                              // producer: phase index in the schedule
  const char* base; int row_bytes, mode, G, ffn, N, cpr;   // projection of phase ps
  int n, which, part;                  // producer cursor inside phase ps
  unsigned issued, consumed;
  uint32_t ring, bars;                 // shared-memory addresses of this warp's slots and mbarriers
  int slot_bytes;
};

template <class T>
__device__ __forceinline__ void stream_load_phase(const MegaParams& p, WarpStream& ws, int gw) {
  GemvDesc g = stream_desc(p, ws.ps);
  ws.base = (const char*)g.W; ws.row_bytes = g.K * (int)sizeof(T); ws.mode = g.mode; ws.G = g.G; ws.ffn = g.ffn; ws.N = g.N;
  ws.cpr = (ws.row_bytes + ws.slot_bytes - 1) / ws.slot_bytes;
  ws.n = gw; ws.which = 0; ws.part = 0;
}

// Keep the ring full: issue copies of the next chunks of the schedule into free slots.
template <class T>
__device__ __forceinline__ void stream_fill(const MegaParams& p, WarpStream& ws, int gw, int GW, int lane) {
  const int n_stream = 4 * p.layer_end + (p.do_head ? 1 : 0);     // schedule entries of this launch end here
  while (ws.issued - ws.consumed < (unsigned)NSLOT) {
    while (ws.ps < n_stream && ws.n >= ws.N) {
      if (++ws.ps < n_stream) stream_load_phase<T>(p, ws, gw);
    }
    if (ws.ps >= n_stream) break;
    int row = ws.n;
    if (ws.mode == GEMV_SWIGLU) { RowMap m{ws.which && ws.G == 0 ? ws.ffn : 0, ws.G, ws.which, ws.ffn}; row = map_row(m, ws.n); }
    const int off = ws.part * ws.slot_bytes;
    const int bytes = min(ws.slot_bytes, ws.row_bytes - off);
    const unsigned slot = ws.issued % NSLOT;
    if (lane == 0) {
      mbar_expect_tx(ws.bars + 8u * slot, (uint32_t)bytes);
      bulk_load(ws.ring + slot * ws.slot_bytes, ws.base + (size_t)row * ws.row_bytes + off, (uint32_t)bytes, ws.bars + 8u * slot);
    }
    ++ws.issued;
    if (++ws.part == ws.cpr) {
      ws.part = 0;
      if (++ws.which == (ws.mode == GEMV_SWIGLU ? 2 : 1)) { ws.which = 0; ws.n += GW; }
    }
  }
}

// Staged activations are stored permuted so that a warp's reads are bank-conflict free: within
// every group of 256 elements, lane l's elements 8l..8l+3 sit at [4l, 4l+4) and 8l+4..8l+7 at
// [128 + 4l, 128 + 4l + 4).  (Shared-memory bandwidth, not HBM, bounds these phases otherwise.)
__device__ __forceinline__ int xs_index(int k) {
  return (k & ~255) + ((k & 4) << 5) + (((k & 255) >> 3) << 2) + (k & 3);
}
__device__ __forceinline__ int xs_stride(int K) { return (K + 255) & ~255; }

// 8 consecutive weights (16 bytes for bf16, 32 for fp32) times 8 activations, two partial sums
template <class T> __device__ __forceinline__ float dot_w8(const unsigned char* w, const float* x);
template <> __device__ __forceinline__ float dot_w8<bf16>(const unsigned char* w, const float* x) {
  const uint4 u = *reinterpret_cast<const uint4*>(w);
  const float4 x0 = *reinterpret_cast<const float4*>(x), x1 = *reinterpret_cast<const float4*>(x + 128);
  float a = __uint_as_float(u.x << 16) * x0.x;
  float b = __uint_as_float(u.x & 0xffff0000u) * x0.y;
  a = fmaf(__uint_as_float(u.y << 16), x0.z, a);
  b = fmaf(__uint_as_float(u.y & 0xffff0000u), x0.w, b);
  a = fmaf(__uint_as_float(u.z << 16), x1.x, a);
  b = fmaf(__uint_as_float(u.z & 0xffff0000u), x1.y, b);
  a = fmaf(__uint_as_float(u.w << 16), x1.z, a);
  b = fmaf(__uint_as_float(u.w & 0xffff0000u), x1.w, b);
  return a + b;
}
template <> __device__ __forceinline__ float dot_w8<float>(const unsigned char* w, const float* x) {
  const float4 w0 = *reinterpret_cast<const float4*>(w), w1 = *reinterpret_cast<const float4*>(w + 16);
  const float4 x0 = *reinterpret_cast<const float4*>(x), x1 = *reinterpret_cast<const float4*>(x + 128);
  float a = w0.x * x0.x, b = w0.y * x0.y;
  a = fmaf(w0.z, x0.z, a); b = fmaf(w0.w, x0.w, b);
  a = fmaf(w1.x, x1.x, a); b = fmaf(w1.y, x1.y, b);
  a = fmaf(w1.z, x1.z, a); b = fmaf(w1.w, x1.w, b);
  return a + b;
}

// One projection phase for this warp: y[b, n] (op)= sum_k W[n, k] xs[b, k] over the warp's rows,
// consuming the warp's chunk stream.  xs is the staged (normalised) input in shared memory and
// ring_ptr the address of the warp's first slot.
template <class T, int BB>
__device__ __forceinline__ void gemv_phase(const MegaParams& p, const GemvDesc g, WarpStream& ws, const unsigned char* ring_ptr,
                                           const float* xs, float* y, int ldy, int gw, int GW, int lane,
                                           unsigned long long* best, volatile int* s_abort) {
  const int K = g.K, row_bytes = K * (int)sizeof(T);
  const int cpr = (row_bytes + ws.slot_bytes - 1) / ws.slot_bytes;
  const int R = g.mode == GEMV_SWIGLU ? 2 : 1;
  const bool vec = (K % 8 == 0);
  const int slot_elems = ws.slot_bytes / (int)sizeof(T);
  const int KS = xs_stride(K);
  float acc[BB], accu[BB];
#pragma unroll
  for (int b = 0; b < BB; ++b) { acc[b] = 0.f; accu[b] = 0.f; }
  for (int n = gw; n < g.N; n += GW) {
    for (int which = 0; which < R; ++which) {
      for (int part = 0; part < cpr; ++part) {
        const unsigned slot = ws.consumed % NSLOT;
        const uint32_t bar = ws.bars + 8u * slot, parity = (ws.consumed / NSLOT) & 1u;
        bool got = false;
        if (!*s_abort) {
          for (unsigned it = 0; it < SPIN_LIMIT; ++it) {
            if (mbar_test(bar, parity)) { got = true; break; }
            if ((it & 1023u) == 1023u && *s_abort) break;
          }
          if (!got && !*s_abort) { *s_abort = 1; dev_flag(p.status, DEV_TIMEOUT); }
        }
        got = __all_sync(0xffffffffu, got);
        if (got) {
          const int k0 = part * slot_elems;
          const int ne = min(slot_elems, K - k0);
          const unsigned char* sp = ring_ptr + (size_t)slot * ws.slot_bytes;
          float* a = which ? accu : acc;
          if (vec) {
#pragma unroll 4
            for (int e = lane * 8; e < ne; e += 256) {   // k0 and e - 8 lane are multiples of 256
#pragma unroll
              for (int b = 0; b < BB; ++b) a[b] += dot_w8<T>(sp + (size_t)e * sizeof(T), xs + b * KS + k0 + (e - lane * 8) + lane * 4);
            }
          } else {
            const T* wp = reinterpret_cast<const T*>(sp);
            for (int e = lane; e < ne; e += 32) {
              float wv = to_f(wp[e]);
#pragma unroll
              for (int b = 0; b < BB; ++b) a[b] = fmaf(wv, xs[b * KS + xs_index(k0 + e)], a[b]);
            }
          }
        }
        ++ws.consumed;
        __syncwarp();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (got) stream_fill<T>(p, ws, gw, GW, lane);
      }
    }
    // all pieces of this output are in: reduce, apply, store
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float v = warp_sum(acc[b]);
      float u = R == 2 ? warp_sum(accu[b]) : 0.f;
      if (lane == 0 && b < p.batch && !*s_abort) {
        float* dst = y + (size_t)b * ldy + n;
        if (g.mode == GEMV_SWIGLU) *dst = v / (1.f + __expf(-v)) * u;
        else if (g.mode == GEMV_RESID) *dst = __ldcg(dst) + v;
        else {
          *dst = v;
          if (best) {   // running argmax: larger value wins, then the lower index
            unsigned bits = __float_as_uint(v);
            bits = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
            atomicMax(best + b, ((unsigned long long)bits << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)n));
          }
        }
      }
      acc[b] = 0.f; accu[b] = 0.f;
    }
  }
}

// Stage `batch` activation rows of length K into shared memory, optionally RMS-normalised
// (one pass: the row is held in registers between the sum of squares and the scaled store).
template <int BB>
__device__ __noinline__ void stage_x(const float* x, int ldx, int K, int batch, const float* gain, float eps, float* xs,
                                     float* red) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int KS = xs_stride(K);
  if (gain && K <= 8 * NT) {
    float v[BB][8];
    float ss[BB];
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      ss[b] = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        int k = tid + j * NT;
        v[b][j] = (k < K && b < batch) ? __ldcg(x + (size_t)b * ldx + k) : 0.f;
        ss[b] = fmaf(v[b][j], v[b][j], ss[b]);
      }
    }
#pragma unroll
    for (int b = 0; b < BB; ++b) { float t = warp_sum(ss[b]); if (lane == 0) red[warp * BB + b] = t; }
    __syncthreads();
#pragma unroll
    for (int b = 0; b < BB; ++b) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) t += red[w * BB + b];
      float r = rsqrtf(t / (float)K + eps);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        int k = tid + j * NT;
        if (k < K) xs[b * KS + xs_index(k)] = gain[k] * v[b][j] * r;
      }
    }
  } else {
    float r[BB];
#pragma unroll
    for (int b = 0; b < BB; ++b) r[b] = 1.f;
    if (gain) {
      float ss[BB];
#pragma unroll
      for (int b = 0; b < BB; ++b) ss[b] = 0.f;
      for (int k = tid; k < K; k += NT) {
#pragma unroll
        for (int b = 0; b < BB; ++b)
          if (b < batch) { float t = __ldcg(x + (size_t)b * ldx + k); ss[b] = fmaf(t, t, ss[b]); }
      }
#pragma unroll
      for (int b = 0; b < BB; ++b) { float t = warp_sum(ss[b]); if (lane == 0) red[warp * BB + b] = t; }
      __syncthreads();
#pragma unroll
      for (int b = 0; b < BB; ++b) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) t += red[w * BB + b];
        r[b] = rsqrtf(t / (float)K + eps);
      }
    }
    for (int k = tid; k < K; k += NT) {
      float g = gain ? gain[k] : 1.f;
#pragma unroll
      for (int b = 0; b < BB; ++b) xs[b * KS + xs_index(k)] = b < batch ? g * __ldcg(x + (size_t)b * ldx + k) * r[b] : 0.f;
    }
  }
  __syncthreads();
}

// Attention of one (sequence, kv head, key-range split) over whole cache pages: the K and V page
// (64 keys, contiguous) are copied to shared memory with independent 16-byte loads; scores with
// thread = (key, head), softmax statistics with one warp per head, value sum with thread =
// (dim, head subset).
template <class T>
__device__ __noinline__ void attn_item(const MegaParams& p, const MegaLayer& L, int b, int kvh, int sp, int n_split,
                                       const float* q, int ldq, unsigned char* sm, float* part, float* out) {
  const int hd = p.hd, nq = L.nq, nkv = L.nkv, group = nq / nkv;
  const int row_bytes = hd * (int)sizeof(T) + 16;
  unsigned char* Ks = sm;
  unsigned char* Vs = Ks + PAGE_TOKENS * row_bytes;
  float* qs = reinterpret_cast<float*>(Vs + PAGE_TOKENS * row_bytes);
  float* ps = qs + MAXG * hd;
  float* m_run = ps + MAXG * PAGE_TOKENS;
  float* l_run = m_run + MAXG;
  float* alpha = l_run + MAXG;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_keys = __ldcg(p.seq_lens + b) + (p.generation ? 1 : 0);
  const int pos = n_keys - 1;
  const float scale = rsqrtf((float)hd);
  const int half = hd >> 1;
  __syncthreads();                                   // shared memory free (previous item / phase)
  if (L.q_norm) head_rnorm(q + (size_t)b * ldq + (size_t)kvh * group * hd, group, hd, p.eps, ps);   // ps is free until the first page's scores
  for (int i = tid; i < group * half; i += NT) {
    int h = i / half, c = i - h * half;
    const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * hd;
    float sn, cs;
    rope_sincos(pos, p.inv.f[c], &sn, &cs);
    float x1 = __ldcg(qh + c), x2 = __ldcg(qh + c + half);
    if (L.q_norm) { const float rn = ps[h]; x1 *= rn * L.q_norm[c]; x2 *= rn * L.q_norm[c + half]; }
    qs[h * hd + c] = (x1 * cs - x2 * sn) * scale;
    qs[h * hd + c + half] = (x2 * cs + x1 * sn) * scale;
  }
  if (tid < MAXG) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; alpha[tid] = 1.f; }
  const int n_pg = (n_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  const int per = (n_pg + n_split - 1) / n_split;
  const int pg0 = sp * per, pg1 = min(n_pg, pg0 + per);
  const int key = tid & 63, hh_s = tid >> 6;           // scores: thread = (key, head hh_s)
  const int nhh = NT / hd;                             // value sum: heads hh_v, hh_v + nhh, ...
  const int dim = tid % hd, hh_v = tid / hd;
  float o[MAXG];
#pragma unroll
  for (int i = 0; i < MAXG; ++i) o[i] = 0.f;
  typedef typename KvOf<T>::type KT;                   // cache element: fp32, or 16-bit half in bf16 mode
  const int chunks_per_row = hd * (int)sizeof(KT) / 16;
  const int n_chunks = PAGE_TOKENS * chunks_per_row;
  const KT* kpool = (const KT*)L.kpool;
  const KT* vpool = (const KT*)L.vpool;
  for (int pg = pg0; pg < pg1; ++pg) {
    int page = pg < p.mpps ? p.block_table[(size_t)b * p.mpps + pg] : -1;
    bool page_ok = page >= 0 && page < p.n_pages;
    if (!page_ok && tid == 0) dev_flag(p.status, DEV_BAD_PAGE);
    const int nk = page_ok ? min(PAGE_TOKENS, n_keys - pg * PAGE_TOKENS) : 0;
    __syncthreads();
    if (page_ok) {
      const uint4* ksrc = reinterpret_cast<const uint4*>(kpool + ((size_t)page * nkv + kvh) * PAGE_TOKENS * hd);
      const uint4* vsrc = reinterpret_cast<const uint4*>(vpool + ((size_t)page * nkv + kvh) * PAGE_TOKENS * hd);
      for (int i = tid; i < n_chunks; i += NT) {
        int r = i / chunks_per_row, cc = i - r * chunks_per_row;
        uint4 kx = __ldcg(ksrc + i), vx = __ldcg(vsrc + i);
        *reinterpret_cast<uint4*>(Ks + r * row_bytes + cc * 16) = kx;
        *reinterpret_cast<uint4*>(Vs + r * row_bytes + cc * 16) = vx;
      }
    }
    __syncthreads();
    if (hh_s < group) {
      float sc = 0.f;
      const KT* kr = reinterpret_cast<const KT*>(Ks + key * row_bytes);
      for (int c = 0; c < hd; c += 8) {
        float kf[8];
        if (sizeof(KT) == 2) {
          uint4 u = *reinterpret_cast<const uint4*>(kr + c);
          const __half2* hp = reinterpret_cast<const __half2*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) { float2 t = __half22float2(hp[e]); kf[2 * e] = t.x; kf[2 * e + 1] = t.y; }
        } else {
          float4 a = *reinterpret_cast<const float4*>(kr + c), bq = *reinterpret_cast<const float4*>(kr + c + 4);
          kf[0] = a.x; kf[1] = a.y; kf[2] = a.z; kf[3] = a.w; kf[4] = bq.x; kf[5] = bq.y; kf[6] = bq.z; kf[7] = bq.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) sc = fmaf(kf[e], qs[hh_s * hd + c + e], sc);
      }
      ps[hh_s * PAGE_TOKENS + key] = key < nk ? sc : -INFINITY;
    }
    __syncthreads();
    if (warp < group) {
      const int h = warp;
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
#pragma unroll
    for (int i = 0; i < MAXG; ++i) {
      int h = hh_v + nhh * i;
      if (i * nhh < MAXG && h < group) {
        float acc = o[i] * alpha[h];
        const float* pr = ps + h * PAGE_TOKENS;
        for (int s = 0; s < nk; ++s) acc = fmaf(pr[s], to_f(reinterpret_cast<const KT*>(Vs + s * row_bytes)[dim]), acc);
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

template <class T, int BB>
__global__ void __launch_bounds__(NT, 1) step_mega_kernel(const __grid_constant__ MegaParams p) {
  extern __shared__ __align__(128) unsigned char sm_raw[];
  __shared__ float red[NW * BB];
  __shared__ int s_flag;
  __shared__ int s_last;
  __shared__ int s_abort_mem;
  __shared__ __align__(8) unsigned long long s_bars[NW * NSLOT];
  volatile int* s_abort = &s_abort_mem;
  // dynamic shared memory: [ x staging / attention scratch | per-warp rings ]
  float* xs = reinterpret_cast<float*>(sm_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gw = blockIdx.x * NW + warp, GW = gridDim.x * NW;
  const int batch = p.batch;
  unsigned* counter = reinterpret_cast<unsigned*>(p.status) + 32 + p.counter_idx;
  unsigned long long* best = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(p.status) + 64);
  if (tid == 0) {
    *s_abort = 0;
    for (int i = 0; i < NW * NSLOT; ++i) mbar_init(smem_u32(&s_bars[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  WarpStream ws;
  ws.ps = 4 * p.layer_begin; ws.issued = 0; ws.consumed = 0;
  ws.slot_bytes = p.slot_bytes;
  const unsigned char* ring_ptr = sm_raw + p.stage_bytes + (size_t)warp * NSLOT * p.slot_bytes;
  ws.ring = smem_u32(ring_ptr);
  ws.bars = smem_u32(&s_bars[warp * NSLOT]);
  stream_load_phase<T>(p, ws, gw);
  stream_fill<T>(p, ws, gw, GW, lane);        // the first weight rows start streaming before anything else

  unsigned phase = 0;
#define BARRIER()                                                                                                   \
  do {                                                                                                              \
    ++phase;                                                                                                        \
    if (p.trace && blockIdx.x == 0 && tid == 0 && phase < 900) p.trace[2 * phase] = clock64();                     \
    if (!grid_barrier(counter, phase * gridDim.x, p.status, s_abort, &s_flag)) {                                    \
      for (int i_ = 0; i_ < 2000; ++i_) __nanosleep(1000); /* let copies in flight land before the CTA goes */      \
      return;                                                                                                       \
    }                                                                                                               \
    if (p.trace && blockIdx.x == 0 && tid == 0 && phase < 900) p.trace[2 * phase + 1] = clock64();                 \
  } while (0)

  // embedding gather (+ clear the argmax slots)
  if (p.do_embed)
  for (int i = blockIdx.x * NT + tid; i < batch * p.d; i += gridDim.x * NT) {
    int b = i / p.d, c = i - b * p.d;
    int tok = p.tokens[p.gather_idx ? p.gather_idx[b] : b];
    bool ok = tok >= 0 && tok < p.vocab;
    if (!ok && c == 0) dev_flag(p.status, DEV_BAD_TOKEN);
    p.xb[(size_t)b * p.d + c] = ok ? to_f(((const T*)p.embed)[(size_t)tok * p.d + c]) : 0.f;
  }
  if (blockIdx.x == 0 && tid < BB) best[tid] = 0ull;
  BARRIER();

  for (int i = p.layer_begin; i < p.layer_end; ++i) {
    const MegaLayer& L = p.layers[i];
    const int n_out = p.generation ? L.nqkv : L.dq;
    // ---- q (k, v) projection
    stage_x<BB>(p.xb, p.d, p.d, batch, L.attn_norm, p.eps, xs, red);
    gemv_phase<T, BB>(p, stream_desc(p, 4 * i), ws, ring_ptr, xs, p.qkvb, n_out, gw, GW, lane, nullptr, s_abort);
    BARRIER();
    if (p.generation) {   // append the new key (after RoPE) and value at position seq_lens[b]
      for (int b = blockIdx.x; b < batch; b += gridDim.x) {
        int pos = __ldcg(p.seq_lens + b);
        int pg = pos / PAGE_TOKENS;
        int page = pg < p.mpps ? p.block_table[(size_t)b * p.mpps + pg] : -1;
        if (page < 0 || page >= p.n_pages) { if (tid == 0) dev_flag(p.status, DEV_BAD_PAGE); continue; }
        int row = pos % PAGE_TOKENS, half = p.hd >> 1;
        const float* kin = p.qkvb + (size_t)b * n_out + L.dq;
        const float* vin = kin + (size_t)L.nkv * p.hd;
        float* rk = reinterpret_cast<float*>(sm_raw);     // the staging area is idle in this phase
        __syncthreads();
        if (L.k_norm) head_rnorm(kin, L.nkv, p.hd, p.eps, rk);
        for (int e = tid; e < L.nkv * half; e += NT) {
          int h = e / half, c = e - h * half;
          float sn, cs;
          rope_sincos(pos, p.inv.f[c], &sn, &cs);
          float x1 = __ldcg(kin + h * p.hd + c), x2 = __ldcg(kin + h * p.hd + c + half);
          if (L.k_norm) { x1 *= rk[h] * L.k_norm[c]; x2 *= rk[h] * L.k_norm[c + half]; }
          size_t off = (((size_t)page * L.nkv + h) * PAGE_TOKENS + row) * p.hd;
          typedef typename KvOf<T>::type KT;
          ((KT*)L.kpool)[off + c] = from_f<KT>(x1 * cs - x2 * sn);
          ((KT*)L.kpool)[off + c + half] = from_f<KT>(x2 * cs + x1 * sn);
          ((KT*)L.vpool)[off + c] = from_f<KT>(__ldcg(vin + h * p.hd + c));
          ((KT*)L.vpool)[off + c + half] = from_f<KT>(__ldcg(vin + h * p.hd + c + half));
        }
      }
      BARRIER();
    }
    // ---- attention over the cache.  With split key ranges the CTA that finishes the last split of a
    // (sequence, kv head) merges that group's partial results on the spot (a counter per group tells
    // it so), which saves a separate merge phase and its grid barrier.
    {
      const int n_items = batch * L.nkv * p.n_split;
      const int group = L.nq / L.nkv, ldr = p.hd + 2;
      for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
        const int sp = it % p.n_split, r = it / p.n_split;
        attn_item<T>(p, L, r / L.nkv, r % L.nkv, sp, p.n_split, p.qkvb, n_out, sm_raw, p.part, p.ab);
        if (p.n_split > 1) {
          __threadfence();                       // this CTA's partial results are visible before it counts itself done
          __syncthreads();
          if (tid == 0) {
            const int before = atomicAdd(p.attn_done + r, 1);
            s_last = before == p.n_split - 1;
            if (s_last) atomicExch(p.attn_done + r, 0);      // ready for the next layer
          }
          __syncthreads();
          if (s_last) {
            __threadfence();
            if (warp < group) {                  // one warp per q head of the group
              const int head = (r / L.nkv) * L.nq + (r % L.nkv) * group + warp;
              const float* pr = p.part + (size_t)head * p.n_split * ldr;
              float mm = -INFINITY;
              for (int s = lane; s < p.n_split; s += 32) mm = fmaxf(mm, __ldcg(pr + (size_t)s * ldr + p.hd));
              mm = warp_max(mm);
              // the loads of different splits do not depend on one another: unrolled, they are in flight together
              float ll = 0.f, o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll 8
              for (int s = 0; s < p.n_split; ++s) {
                const float* rr = pr + (size_t)s * ldr;
                const float ms = __ldcg(rr + p.hd);
                const float f = (ms == -INFINITY) ? 0.f : __expf(ms - mm);
                ll = fmaf(__ldcg(rr + p.hd + 1), f, ll);
                if (lane < p.hd) o0 = fmaf(__ldcg(rr + lane), f, o0);
                if (lane + 32 < p.hd) o1 = fmaf(__ldcg(rr + lane + 32), f, o1);
                if (lane + 64 < p.hd) o2 = fmaf(__ldcg(rr + lane + 64), f, o2);
                if (lane + 96 < p.hd) o3 = fmaf(__ldcg(rr + lane + 96), f, o3);
              }
              float* dst = p.ab + (size_t)head * p.hd;
              if (lane < p.hd) dst[lane] = o0 / ll;
              if (lane + 32 < p.hd) dst[lane + 32] = o1 / ll;
              if (lane + 64 < p.hd) dst[lane + 64] = o2 / ll;
              if (lane + 96 < p.hd) dst[lane + 96] = o3 / ll;
            }
          }
        }
      }
    }
    BARRIER();
    // ---- O projection + residual
    stage_x<BB>(p.ab, L.dq, L.dq, batch, nullptr, 0.f, xs, red);
    gemv_phase<T, BB>(p, stream_desc(p, 4 * i + 1), ws, ring_ptr, xs, p.xb, p.d, gw, GW, lane, nullptr, s_abort);
    BARRIER();
    // ---- gate / up + SwiGLU
    stage_x<BB>(p.xb, p.d, p.d, batch, L.ffn_norm, p.eps, xs, red);
    gemv_phase<T, BB>(p, stream_desc(p, 4 * i + 2), ws, ring_ptr, xs, p.actb, L.ffn, gw, GW, lane, nullptr, s_abort);
    BARRIER();
    // ---- down projection + residual
    stage_x<BB>(p.actb, L.ffn, L.ffn, batch, nullptr, 0.f, xs, red);
    gemv_phase<T, BB>(p, stream_desc(p, 4 * i + 3), ws, ring_ptr, xs, p.xb, p.d, gw, GW, lane, nullptr, s_abort);
    BARRIER();
  }
  if (!p.do_head) return;             // a later launch carries on from the residual stream in xb
  // ---- LM head (final RMSNorm fused) with running argmax
  stage_x<BB>(p.xb, p.d, p.d, batch, p.final_norm, p.eps, xs, red);
  gemv_phase<T, BB>(p, stream_desc(p, 4 * p.n_layers), ws, ring_ptr, xs, p.logits, p.vocab, gw, GW, lane,
                    p.token_out ? best : nullptr, s_abort);
  BARRIER();
  if (blockIdx.x == 0 && tid < batch) {
    if (p.token_out) {
      unsigned long long v;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(best + tid) : "memory");
      p.token_out[tid] = (int)(0xFFFFFFFFu - (unsigned)(v & 0xFFFFFFFFull));
    }
    if (p.generation) p.seq_lens[tid] += 1;
  }
#undef BARRIER
}

constexpr int SMEM_LIMIT = 227 * 1024 - 2048;   // dynamic shared memory we allow ourselves per CTA

size_t stage_region_bytes(int batch, int hd, int k_max, int es) {
  int bb = batch <= 1 ? 1 : (batch == 2 ? 2 : 4);
  size_t xs = (size_t)bb * ((k_max + 255) / 256 * 256) * 4;
  size_t at = (size_t)2 * PAGE_TOKENS * (hd * es + 16) + (size_t)(MAXG * hd + MAXG * PAGE_TOKENS + 3 * MAXG) * 4;
  size_t r = xs > at ? xs : at;
  return (r + 127) / 128 * 128;
}

template <class T, int BB>
cudaError_t go(MegaParams& p, size_t smem, cudaStream_t st, int n_sm) {
  auto kern = step_mega_kernel<T, BB>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NT, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  void* args[] = {(void*)&p};
  return cudaLaunchCooperativeKernel((const void*)kern, dim3(n_sm), dim3(NT), args, smem, st);
}

}  // namespace

bool step_mega_supported(int batch, int hd, int k_max, int max_group, int es) {
  if (batch < 1 || batch > 4) return false;
  if (!(hd == 16 || hd == 32 || hd == 64 || hd == 128)) return false;
  if (max_group > MAXG) return false;
  size_t stage = stage_region_bytes(batch, hd, k_max, es);
  return stage + (size_t)NW * NSLOT * 1024 <= (size_t)SMEM_LIMIT;   // at least 1 KiB per ring slot
}

cudaError_t launch_step_mega(MegaParams p, int dtype, int k_max, int n_sm, cudaStream_t st, int64_t* n_launch) {
  const int es = dtype == 0 ? 4 : 2;
  size_t stage = stage_region_bytes(p.batch, p.hd, k_max, es);
  int slot = (int)((SMEM_LIMIT - stage) / (NW * NSLOT));
  slot = slot / 1024 * 1024;      // whole 256-element groups of either element size
  if (slot > 8192) slot = 8192;
  p.stage_bytes = (int)stage;
  p.slot_bytes = slot;
  size_t smem = stage + (size_t)NW * NSLOT * slot;
  ++*n_launch;
  if (dtype == 0) {
    if (p.batch <= 1) return go<float, 1>(p, smem, st, n_sm);
    if (p.batch == 2) return go<float, 2>(p, smem, st, n_sm);
    return go<float, 4>(p, smem, st, n_sm);
  }
  if (p.batch <= 1) return go<bf16, 1>(p, smem, st, n_sm);
  if (p.batch == 2) return go<bf16, 2>(p, smem, st, n_sm);
  return go<bf16, 4>(p, smem, st, n_sm);
}
