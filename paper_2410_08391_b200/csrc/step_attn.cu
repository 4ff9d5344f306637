// Single-query GQA attention of the base step over the paged bf16 cache, bandwidth-bound variant.
//
// grid (key-range split, kv head, sequence); a CTA of 64 * group threads serves the `group` query
// heads that share one kv head and walks its range of cache pages.  A page of one kv head is one
// contiguous block (64 keys x head_dim), so K and V pages are fetched whole with bulk asynchronous
// copies into a ring of shared-memory stages, several pages ahead of the arithmetic: the HBM
// latency is covered by copies in flight, not by resident warps.
//   scores   thread = (key, head): dot product of the key's row with the head's query; the row's
//            16-byte pieces are visited in an order rotated by the key index, which keeps the
//            row-per-thread reads free of bank conflicts without padding the copied page
//   softmax  one warp per head over the page's 64 scores, running max / sum in shared memory
//   values   thread = (head, pair of dims): sum over the page's keys
// With more than one split, partial (o, m, l) per (sequence, q head, split) go to `part`.
// The wait on a page's copies is bounded; on expiry the CTA flags DEV_TIMEOUT and leaves.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int ST = 3;                       // pages in flight per CTA (K and V each)
constexpr int MAXG = 8;
constexpr uint32_t SPIN_LIMIT = 20u * 1000u * 1000u;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <int HD>
__global__ void __launch_bounds__(512) step_attn_ring_kernel(const float* __restrict__ q, int ldq, int nq, int nkv,
                                                             const __grid_constant__ InvFreq inv,
                                                             const bf16* __restrict__ kpool, const bf16* __restrict__ vpool,
                                                             const int* __restrict__ block_table, int mpps, int n_pages,
                                                             const int* __restrict__ seq_lens, int extra, int n_split,
                                                             float* __restrict__ part, float* __restrict__ out, int* status,
                                                             const float* __restrict__ q_gain, float eps) {
  constexpr int PAGE_BYTES = PAGE_TOKENS * HD * 2;       // one K or V page of one kv head
  constexpr int CH = HD / 8;                             // 16-byte pieces per key row
  constexpr int DP = HD / 64;                            // dims per thread in the value sum (1 or 2)
  extern __shared__ __align__(128) unsigned char sm_raw[];
  unsigned char* ring = sm_raw;                                                  // [ST][K page | V page]
  float* qs = reinterpret_cast<float*>(sm_raw + ST * 2 * PAGE_BYTES);            // [MAXG][HD], scaled, after RoPE
  float* ps = qs + MAXG * HD;                                                    // [MAXG][64]
  float* m_run = ps + MAXG * PAGE_TOKENS;
  float* l_run = m_run + MAXG;
  float* alpha = l_run + MAXG;
  __shared__ __align__(8) unsigned long long bars[ST];
  __shared__ int s_ok;
  __shared__ float rq[MAXG];
  const int group = nq / nkv;
  const int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_keys = seq_lens[b] + extra;
  const int pos = n_keys - 1;
  const int n_pg = (n_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  const int per = (n_pg + n_split - 1) / n_split;
  const int pg0 = sp * per, pg1 = min(n_pg, pg0 + per);
  const int n_it = max(pg1 - pg0, 0);

  auto issue = [&](int it) {     // thread 0: start the copies of page pg0 + it into slot it % ST
    const int pg = pg0 + it;
    int page = pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
    const uint32_t bar = smem_u32(&bars[it % ST]);
    if (page < 0 || page >= n_pages) {   // never dereferenced: the slot completes empty and the page is skipped below
      dev_flag(status, DEV_BAD_PAGE);
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
      return;
    }
    const size_t off = ((size_t)page * nkv + kvh) * PAGE_TOKENS * HD;
    const uint32_t dst = smem_u32(ring + (size_t)(it % ST) * 2 * PAGE_BYTES);
    mbar_expect_tx(bar, 2 * PAGE_BYTES);
    bulk_load(dst, kpool + off, PAGE_BYTES, bar);
    bulk_load(dst + PAGE_BYTES, vpool + off, PAGE_BYTES, bar);
  };

  if (tid == 0) {
    for (int s = 0; s < ST; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_ok = 1;
    for (int it = 0; it < min(ST - 1, n_it); ++it) issue(it);
  }
  // queries of the group: (query norm,) RoPE at the last position, scaled by 1/sqrt(hd)
  if (q_gain) head_rnorm(q + (size_t)b * ldq + (size_t)kvh * group * HD, group, HD, eps, rq);
  {
    const float scale = rsqrtf((float)HD);
    constexpr int half = HD / 2;
    for (int i = tid; i < group * half; i += blockDim.x) {
      const int h = i / half, c = i - h * half;
      const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * HD;
      float sn, cs;
      rope_sincos(pos, inv.f[c], &sn, &cs);
      float x1 = qh[c], x2 = qh[c + half];
      if (q_gain) { x1 *= rq[h] * q_gain[c]; x2 *= rq[h] * q_gain[c + half]; }
      qs[h * HD + c] = (x1 * cs - x2 * sn) * scale;
      qs[h * HD + c + half] = (x2 * cs + x1 * sn) * scale;
    }
    if (tid < MAXG) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; alpha[tid] = 1.f; }
  }
  const int key = tid & 63, h = tid >> 6;         // scores: (key, head); values: (pair of dims = key, head)
  float acc[DP];
#pragma unroll
  for (int i = 0; i < DP; ++i) acc[i] = 0.f;
  bool ok = true;
  for (int it = 0; it < n_it; ++it) {
    __syncthreads();                              // slot (it - 1) % ST and ps are free again; qs is staged
    if (tid == 0 && it + ST - 1 < n_it) issue(it + ST - 1);
    // wait for this page's copies (every thread polls the mbarrier; bounded)
    {
      const uint32_t bar = smem_u32(&bars[it % ST]), parity = (it / ST) & 1;
      bool got = false;
      for (uint32_t spin = 0; spin < SPIN_LIMIT; ++spin) {
        if (mbar_test(bar, parity)) { got = true; break; }
        if ((spin & 1023u) == 1023u && *(volatile int*)&s_ok == 0) break;
      }
      if (!got) { s_ok = 0; dev_flag(status, DEV_TIMEOUT); }
    }
    ok = __syncthreads_and(*(volatile int*)&s_ok != 0);
    if (!ok) break;
    const int pg = pg0 + it;
    const int page = pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
    const int nk = (page >= 0 && page < n_pages) ? min(PAGE_TOKENS, n_keys - pg * PAGE_TOKENS) : 0;
    const unsigned char* Ks = ring + (size_t)(it % ST) * 2 * PAGE_BYTES;
    const unsigned char* Vs = Ks + PAGE_BYTES;
    // ---- scores
    {
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;     // four short chains instead of one of HD steps
      const unsigned char* kr = Ks + key * (HD * 2);
      const float* qh = qs + h * HD;
#pragma unroll 4
      for (int i = 0; i < CH; ++i) {
        const int c = (i + key) & (CH - 1);
        const uint4 u = *reinterpret_cast<const uint4*>(kr + c * 16);
        const float4 q0 = *reinterpret_cast<const float4*>(qh + c * 8), q1 = *reinterpret_cast<const float4*>(qh + c * 8 + 4);
        s0 = fmaf(__uint_as_float(u.x << 16), q0.x, s0); s1 = fmaf(__uint_as_float(u.x & 0xffff0000u), q0.y, s1);
        s2 = fmaf(__uint_as_float(u.y << 16), q0.z, s2); s3 = fmaf(__uint_as_float(u.y & 0xffff0000u), q0.w, s3);
        s0 = fmaf(__uint_as_float(u.z << 16), q1.x, s0); s1 = fmaf(__uint_as_float(u.z & 0xffff0000u), q1.y, s1);
        s2 = fmaf(__uint_as_float(u.w << 16), q1.z, s2); s3 = fmaf(__uint_as_float(u.w & 0xffff0000u), q1.w, s3);
      }
      ps[h * PAGE_TOKENS + key] = key < nk ? (s0 + s1) + (s2 + s3) : -INFINITY;
    }
    __syncthreads();
    // ---- running softmax statistics, one warp per head
    if (warp < group) {
      const int hh = warp;
      const float s0 = ps[hh * PAGE_TOKENS + lane], s1 = ps[hh * PAGE_TOKENS + 32 + lane];
      const float mt = warp_max(fmaxf(s0, s1));
      const float m_old = m_run[hh];
      const float mn = fmaxf(m_old, mt);
      const float p0 = (mn == -INFINITY) ? 0.f : __expf(s0 - mn), p1 = (mn == -INFINITY) ? 0.f : __expf(s1 - mn);
      const float sum = warp_sum(p0 + p1);
      ps[hh * PAGE_TOKENS + lane] = p0; ps[hh * PAGE_TOKENS + 32 + lane] = p1;
      if (lane == 0) {
        const float a = (mn == -INFINITY) ? 1.f : __expf(m_old - mn);
        alpha[hh] = a; m_run[hh] = mn; l_run[hh] = l_run[hh] * a + sum;
      }
    }
    __syncthreads();
    // ---- values
    {
      const float a = alpha[h];
      const float* pr = ps + h * PAGE_TOKENS;
      // keys beyond nk carry p = 0 but their rows are not initialised memory: they are not read
      if (DP == 2) {
        float a0 = acc[0] * a, a1 = acc[DP - 1] * a, b0 = 0.f, b1 = 0.f;
        const uint32_t* vr = reinterpret_cast<const uint32_t*>(Vs) + key;
        int s = 0;
#pragma unroll 4
        for (; s + 2 <= nk; s += 2) {
          const uint32_t u = vr[s * (HD / 2)], w = vr[(s + 1) * (HD / 2)];
          const float pu = pr[s], pw = pr[s + 1];
          a0 = fmaf(pu, __uint_as_float(u << 16), a0); a1 = fmaf(pu, __uint_as_float(u & 0xffff0000u), a1);
          b0 = fmaf(pw, __uint_as_float(w << 16), b0); b1 = fmaf(pw, __uint_as_float(w & 0xffff0000u), b1);
        }
        if (s < nk) {
          const uint32_t u = vr[s * (HD / 2)];
          a0 = fmaf(pr[s], __uint_as_float(u << 16), a0); a1 = fmaf(pr[s], __uint_as_float(u & 0xffff0000u), a1);
        }
        acc[0] = a0 + b0; acc[DP - 1] = a1 + b1;
      } else {
        float a0 = acc[0] * a, b0 = 0.f, c0 = 0.f, d0 = 0.f;
        const bf16* vr = reinterpret_cast<const bf16*>(Vs) + key;
        int s = 0;
#pragma unroll 2
        for (; s + 4 <= nk; s += 4) {
          a0 = fmaf(pr[s], __bfloat162float(vr[s * HD]), a0); b0 = fmaf(pr[s + 1], __bfloat162float(vr[(s + 1) * HD]), b0);
          c0 = fmaf(pr[s + 2], __bfloat162float(vr[(s + 2) * HD]), c0); d0 = fmaf(pr[s + 3], __bfloat162float(vr[(s + 3) * HD]), d0);
        }
        for (; s < nk; ++s) a0 = fmaf(pr[s], __bfloat162float(vr[s * HD]), a0);
        acc[0] = (a0 + b0) + (c0 + d0);
      }
    }
  }
  if (!ok) {      // copies may still be landing in this CTA's shared memory
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    return;
  }
  __syncthreads();
  if (h < group) {
    const int qh = kvh * group + h;
    const int ldr = HD + 2;
    if (n_split == 1) {
      const float inv_l = 1.f / l_run[h];
      float* dst = out + (size_t)b * nq * HD + (size_t)qh * HD + key * DP;
#pragma unroll
      for (int i = 0; i < DP; ++i) dst[i] = acc[i] * inv_l;
    } else {
      float* pr = part + (((size_t)b * nq + qh) * n_split + sp) * ldr;
#pragma unroll
      for (int i = 0; i < DP; ++i) pr[key * DP + i] = acc[i];
      if (key == 0) { pr[HD] = m_run[h]; pr[HD + 1] = l_run[h]; }
    }
  }
}

template <int HD>
cudaError_t go(dim3 grid, int threads, cudaStream_t st, const float* q, int ldq, int nq, int nkv, const InvFreq& inv, const bf16* kpool,
               const bf16* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra, int n_split,
               float* part, float* out, int* status, const float* q_gain, float eps) {
  const size_t smem = (size_t)ST * 2 * PAGE_TOKENS * HD * 2 + (size_t)(MAXG * HD + MAXG * PAGE_TOKENS + 3 * MAXG) * sizeof(float);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(step_attn_ring_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  step_attn_ring_kernel<HD><<<grid, threads, smem, st>>>(q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra,
                                                         n_split, part, out, status, q_gain, eps);
  return cudaGetLastError();
}

}  // namespace

bool step_attn_ring_supported(int dtype, int nq, int nkv, int hd, const void* kpool, const void* vpool) {
  const int group = nq / nkv;
  return dtype == 1 && (hd == 64 || hd == 128) && group >= 1 && group <= MAXG && ((uintptr_t)kpool & 15) == 0 && ((uintptr_t)vpool & 15) == 0;
}

cudaError_t launch_step_attn_ring(const LaunchCtx& ctx, const float* q, int ldq, int nq, int nkv, int hd, float theta, const void* kpool,
                                  const void* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra,
                                  int batch, int n_split, float* part, float* out, const float* q_gain, float eps) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  dim3 grid(n_split, nkv, batch);
  const int threads = 64 * (nq / nkv);
  ++*ctx.n_launch;
  if (hd == 64)
    return go<64>(grid, threads, ctx.st, q, ldq, nq, nkv, inv, (const bf16*)kpool, (const bf16*)vpool, block_table, mpps, n_pages, seq_lens,
                  extra, n_split, part, out, ctx.status, q_gain, eps);
  return go<128>(grid, threads, ctx.st, q, ldq, nq, nkv, inv, (const bf16*)kpool, (const bf16*)vpool, block_table, mpps, n_pages, seq_lens,
                 extra, n_split, part, out, ctx.status, q_gain, eps);
}
