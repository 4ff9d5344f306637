// Single-query GQA attention of the base step over the paged 16-bit (half) cache, bandwidth-bound variants.
//
// grid (key-range split, kv head, sequence); a CTA serves the `group` query heads that share one
// kv head and walks its range of cache pages.  A page of one kv head is one contiguous block
// (64 keys x head_dim), so K and V pages are fetched whole with bulk asynchronous copies into a
// ring of shared-memory stages, several pages ahead of the arithmetic: the HBM latency is covered
// by copies in flight, not by resident warps.
//
// step_attn_ring_kernel (up to 4 query heads per kv head): every cached element is read from
// shared memory ONCE and used for all heads of the group, because the shared-memory port, not
// HBM, bounds a kernel that re-reads a page per head.
//   scores   DS lanes share a key: each holds its slice of the group's queries in registers for
//            the whole kernel, reads its 16-byte pieces of the key row (pieces interleaved over
//            the lanes and visited in an order rotated by the key index: conflict-free), and the
//            DS partial dot products per head are added with shuffles
//   softmax  a key's lane takes exp(score - offset) against the head's current exponent offset at
//            once; only when a score exceeds the offset by more than 8 (always on the first page)
//            does the block move the offset to the running maximum and rescale what it has summed
//   values   thread = (pair of dims, block of keys): one 4-byte read of V and one broadcast read
//            of the key's probabilities feed 2 x group multiply-adds; the key blocks are summed
//            through shared memory once, after the last page
//   The page ids of the CTA's range are staged in shared memory once; a page costs one block
//   barrier (the vote on the offset).
// step_attn_ring_wide_kernel (5 to 8 heads per kv head): thread = (key, head) for the scores and
// (pair of dims, head) for the values, one warp per head for a per-page softmax.
// With more than one split, partial (o, m, l) per (sequence, q head, split) go to `part`; given a
// zeroed counter per (sequence, kv head), the CTA of step_attn_ring_kernel that finishes a group's
// last split merges them, otherwise a separate kernel does.
// The wait on a page's copies is bounded; on expiry the CTA flags DEV_TIMEOUT and leaves.
#include <math.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int ST = 3;                       // pages in flight per CTA (K and V each)
constexpr int MAXG = 8;
constexpr int MAX_IDS = 512;                // page ids a CTA keeps in shared memory


template <int HD>
__global__ void __launch_bounds__(512) step_attn_ring_wide_kernel(const float* __restrict__ q, int ldq, int nq, int nkv,
                                                             const __grid_constant__ InvFreq inv,
                                                             const kv16* __restrict__ kpool, const kv16* __restrict__ vpool,
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
        s0 = fmaf(kv_lo(u.x), q0.x, s0); s1 = fmaf(kv_hi(u.x), q0.y, s1);
        s2 = fmaf(kv_lo(u.y), q0.z, s2); s3 = fmaf(kv_hi(u.y), q0.w, s3);
        s0 = fmaf(kv_lo(u.z), q1.x, s0); s1 = fmaf(kv_hi(u.z), q1.y, s1);
        s2 = fmaf(kv_lo(u.w), q1.z, s2); s3 = fmaf(kv_hi(u.w), q1.w, s3);
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
          a0 = fmaf(pu, kv_lo(u), a0); a1 = fmaf(pu, kv_hi(u), a1);
          b0 = fmaf(pw, kv_lo(w), b0); b1 = fmaf(pw, kv_hi(w), b1);
        }
        if (s < nk) {
          const uint32_t u = vr[s * (HD / 2)];
          a0 = fmaf(pr[s], kv_lo(u), a0); a1 = fmaf(pr[s], kv_hi(u), a1);
        }
        acc[0] = a0 + b0; acc[DP - 1] = a1 + b1;
      } else {
        float a0 = acc[0] * a, b0 = 0.f, c0 = 0.f, d0 = 0.f;
        const kv16* vr = reinterpret_cast<const kv16*>(Vs) + key;
        int s = 0;
#pragma unroll 2
        for (; s + 4 <= nk; s += 4) {
          a0 = fmaf(pr[s], __half2float(vr[s * HD]), a0); b0 = fmaf(pr[s + 1], __half2float(vr[(s + 1) * HD]), b0);
          c0 = fmaf(pr[s + 2], __half2float(vr[(s + 2) * HD]), c0); d0 = fmaf(pr[s + 3], __half2float(vr[(s + 3) * HD]), d0);
        }
        for (; s < nk; ++s) a0 = fmaf(pr[s], __half2float(vr[s * HD]), a0);
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

// ---- up to 4 query heads per kv head -------------------------------------------------------
template <int HD, int GP>
struct RingCfg {
  static constexpr int DS = (HD * GP > 256) ? 8 : 4;       // lanes that share one key's dot products
  static constexpr int NT = PAGE_TOKENS * DS;              // threads per CTA
  static constexpr int CH = HD / 8;                        // 16-byte pieces per key row
  static constexpr int CPT = CH / DS;                      // pieces per lane
  static constexpr int NKQ = NT / (HD / 2);                // key blocks of the value sum
  static constexpr int KPT = PAGE_TOKENS / NKQ;            // keys per block
  static constexpr int PAGE_BYTES = PAGE_TOKENS * HD * 2;  // one K or V page of one kv head
  // pages in flight: one 512-thread CTA per SM keeps 5 pages ahead, two 256-thread CTAs 2 or 4 each
  static constexpr int STAGES = NT == 512 ? 6 : (HD == 64 ? 5 : 3);
  static constexpr size_t SMEM = (size_t)STAGES * 2 * PAGE_BYTES + (size_t)(GP * HD + 3 * PAGE_TOKENS * GP + 3 * GP) * sizeof(float);
};

template <int HD, int GP>
__global__ void __launch_bounds__(RingCfg<HD, GP>::NT, RingCfg<HD, GP>::NT == 512 ? 1 : 2)
step_attn_ring_kernel(const float* __restrict__ q, int ldq, int nq, int nkv, const __grid_constant__ InvFreq inv,
                      const kv16* __restrict__ kpool, const kv16* __restrict__ vpool, const int* __restrict__ block_table,
                      int mpps, int n_pages, const int* __restrict__ seq_lens, int extra, int n_split,
                      float* __restrict__ part, float* __restrict__ out, int* status, const float* __restrict__ q_gain,
                      float eps, int* __restrict__ split_done) {
  using Cfg = RingCfg<HD, GP>;
  constexpr int DS = Cfg::DS, NT = Cfg::NT, CPT = Cfg::CPT, NKQ = Cfg::NKQ, KPT = Cfg::KPT, STG = Cfg::STAGES;
  constexpr int PAGE_BYTES = Cfg::PAGE_BYTES;
  extern __shared__ __align__(128) unsigned char sm_raw[];
  unsigned char* ring = sm_raw;                                                  // [STG][K page | V page]
  float* qs = reinterpret_cast<float*>(sm_raw + STG * 2 * PAGE_BYTES);           // [GP][HD], scaled, after RoPE
  float* ps_buf = qs + GP * HD;                                                  // 2 x [64 keys][GP] probabilities (alternating pages)
  float* ss = ps_buf + 2 * PAGE_TOKENS * GP;                                     // [64 keys][GP] scores
  float* m_run = ss + PAGE_TOKENS * GP;                                          // exponent offset of each head
  float* l_run = m_run + GP;
  float* alpha = l_run + GP;
  __shared__ __align__(8) unsigned long long bars[STG];
  __shared__ int s_ok;
  __shared__ float rq[MAXG];
  __shared__ int s_page[MAX_IDS];                  // page ids of this CTA's range (a global load per page would sit on the critical path)
  const int group = nq / nkv;                      // <= GP
  const int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_keys = seq_lens[b] + extra;
  const int pos = n_keys - 1;
  const int n_pg = (n_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  const int per = (n_pg + n_split - 1) / n_split;
  const int pg0 = sp * per, pg1 = min(n_pg, pg0 + per);
  const int n_it = max(pg1 - pg0, 0);

  auto page_of = [&](int it) -> int {
    if (it < MAX_IDS) return s_page[it];
    const int pg = pg0 + it;
    return pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
  };
  auto issue = [&](int it) {     // thread 0: start the copies of page pg0 + it into slot it % STG
    const int page = page_of(it);
    const uint32_t bar = smem_u32(&bars[it % STG]);
    if (page < 0 || page >= n_pages) {   // never dereferenced: the slot completes empty and the page is skipped below
      dev_flag(status, DEV_BAD_PAGE);
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
      return;
    }
    const size_t off = ((size_t)page * nkv + kvh) * PAGE_TOKENS * HD;
    const uint32_t dst = smem_u32(ring + (size_t)(it % STG) * 2 * PAGE_BYTES);
    mbar_expect_tx(bar, 2 * PAGE_BYTES);
    bulk_load(dst, kpool + off, PAGE_BYTES, bar);
    bulk_load(dst + PAGE_BYTES, vpool + off, PAGE_BYTES, bar);
  };

  for (int i = tid; i < min(n_it, MAX_IDS); i += NT) {
    const int pg = pg0 + i;
    s_page[i] = pg < mpps ? block_table[(size_t)b * mpps + pg] : -1;
  }
  if (tid == 0) {
    for (int s = 0; s < STG; ++s) mbar_init(smem_u32(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_ok = 1;
  }
  __syncthreads();
  if (tid == 0)
    for (int it = 0; it < min(STG - 1, n_it); ++it) issue(it);
  // queries of the group: (query norm,) RoPE at the last position, scaled by 1/sqrt(hd); heads beyond the group are zero
  if (q_gain) head_rnorm(q + (size_t)b * ldq + (size_t)kvh * group * HD, group, HD, eps, rq);
  {
    const float scale = rsqrtf((float)HD);
    constexpr int half = HD / 2;
    for (int i = tid; i < GP * half; i += NT) {
      const int h = i / half, c = i - h * half;
      float r1 = 0.f, r2 = 0.f;
      if (h < group) {
        const float* qh = q + (size_t)b * ldq + (size_t)(kvh * group + h) * HD;
        float sn, cs;
        rope_sincos(pos, inv.f[c], &sn, &cs);
        float x1 = qh[c], x2 = qh[c + half];
        if (q_gain) { x1 *= rq[h] * q_gain[c]; x2 *= rq[h] * q_gain[c + half]; }
        r1 = (x1 * cs - x2 * sn) * scale;
        r2 = (x2 * cs + x1 * sn) * scale;
      }
      qs[h * HD + c] = r1;
      qs[h * HD + c + half] = r2;
    }
    if (tid < GP) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; alpha[tid] = 1.f; }
  }
  __syncthreads();
  // scores: lane dq of key `key` visits pieces dq + DS * ((i + key) % CPT), i = 0 .. CPT-1; its queries for
  // exactly those pieces stay in registers, in visiting order
  const int key = tid / DS, dq = tid % DS;
  float qr[GP][CPT][8];
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const int c = dq + DS * ((i + key) % CPT);
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      const float4 a = *reinterpret_cast<const float4*>(qs + g * HD + c * 8), bq = *reinterpret_cast<const float4*>(qs + g * HD + c * 8 + 4);
      qr[g][i][0] = a.x; qr[g][i][1] = a.y; qr[g][i][2] = a.z; qr[g][i][3] = a.w;
      qr[g][i][4] = bq.x; qr[g][i][5] = bq.y; qr[g][i][6] = bq.z; qr[g][i][7] = bq.w;
    }
  }
  // values: thread = (pair of dims d2, key block kq)
  const int d2 = tid % (HD / 2), kq = tid / (HD / 2);
  float acc[GP][2];
#pragma unroll
  for (int g = 0; g < GP; ++g) { acc[g][0] = 0.f; acc[g][1] = 0.f; }
  float l_part = 0.f;                              // lane dq < GP: this key slot's share of head dq's sum of probabilities
  bool ok = true;
  // One block barrier per page: a page's probabilities go to the buffer the page before last used, and the
  // slot of page it - 1 is refilled after the barrier of page it, which every thread passes only once it
  // is through with page it - 1.
  for (int it = 0; it < n_it; ++it) {
    float* ps = ps_buf + (it & 1) * PAGE_TOKENS * GP;
    {                                             // wait for this page's copies (every thread polls; bounded)
      const uint32_t bar = smem_u32(&bars[it % STG]), parity = (it / STG) & 1;
      bool got = false;
      for (uint32_t spin = 0; spin < SPIN_LIMIT; ++spin) {
        if (mbar_test(bar, parity)) { got = true; break; }
        if ((spin & 1023u) == 1023u && *(volatile int*)&s_ok == 0) break;
      }
      if (!got) { s_ok = 0; dev_flag(status, DEV_TIMEOUT); }
    }
    const int pg = pg0 + it;
    const int page = page_of(it);
    const int nk = (page >= 0 && page < n_pages) ? min(PAGE_TOKENS, n_keys - pg * PAGE_TOKENS) : 0;
    const unsigned char* Ks = ring + (size_t)(it % STG) * 2 * PAGE_BYTES;
    const unsigned char* Vs = Ks + PAGE_BYTES;
    // ---- scores
    {
      float s[GP];
#pragma unroll
      for (int g = 0; g < GP; ++g) s[g] = 0.f;
      const unsigned char* kr = Ks + key * (HD * 2);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        const int c = dq + DS * ((i + key) % CPT);
        const uint4 u = *reinterpret_cast<const uint4*>(kr + c * 16);
        const float k0 = kv_lo(u.x), k1 = kv_hi(u.x);
        const float k2 = kv_lo(u.y), k3 = kv_hi(u.y);
        const float k4 = kv_lo(u.z), k5 = kv_hi(u.z);
        const float k6 = kv_lo(u.w), k7 = kv_hi(u.w);
#pragma unroll
        for (int g = 0; g < GP; ++g) {
          float t0 = fmaf(k0, qr[g][i][0], s[g]), t1 = k1 * qr[g][i][1];
          t0 = fmaf(k2, qr[g][i][2], t0); t1 = fmaf(k3, qr[g][i][3], t1);
          t0 = fmaf(k4, qr[g][i][4], t0); t1 = fmaf(k5, qr[g][i][5], t1);
          t0 = fmaf(k6, qr[g][i][6], t0); t1 = fmaf(k7, qr[g][i][7], t1);
          s[g] = t0 + t1;
        }
      }
      float mine = 0.f;                            // lane dq < GP keeps head dq's sum
#pragma unroll
      for (int g = 0; g < GP; ++g) {
#pragma unroll
        for (int off = 1; off < DS; off <<= 1) s[g] += __shfl_xor_sync(0xffffffffu, s[g], off);
        if (dq == g) mine = s[g];
      }
      // Probabilities are taken against the head's current offset m_run straight away.  Only when a score
      // exceeds the offset by more than 8 (always on the first page) does the block take the slow path
      // below: new offset = running maximum, everything accumulated so far rescaled.
      float pr = 0.f;
      bool grow = false;
      if (dq < GP) {
        if (key >= nk) mine = -INFINITY;
        const float mr = m_run[dq];
        grow = mine > mr + 8.f;
        pr = (mine == -INFINITY || grow) ? 0.f : __expf(mine - mr);
        ss[key * GP + dq] = mine;
        ps[key * GP + dq] = pr;
      }
      const int any_grow = __syncthreads_or(grow);
      if (*(volatile int*)&s_ok == 0) { ok = false; break; }      // a wait ran out (same answer in every thread: read after the barrier)
      if (tid == 0 && it + STG - 1 < n_it) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the block's reads of that slot come before the copy's writes
        issue(it + STG - 1);
      }
      if (any_grow) {
        if (warp < GP) {
          const int hh = warp;
          const float mt = warp_max(fmaxf(ss[lane * GP + hh], ss[(32 + lane) * GP + hh]));
          if (lane == 0) {
            const float m_old = m_run[hh], mn = fmaxf(m_old, mt);
            alpha[hh] = (m_old == -INFINITY) ? (mn == -INFINITY ? 1.f : 0.f) : __expf(m_old - mn);
            m_run[hh] = mn;
          }
        }
        __syncthreads();
        if (dq < GP) {
          pr = (mine == -INFINITY) ? 0.f : __expf(mine - m_run[dq]);
          ps[key * GP + dq] = pr;
          l_part *= alpha[dq];
        }
#pragma unroll
        for (int g = 0; g < GP; ++g) { const float al = alpha[g]; acc[g][0] *= al; acc[g][1] *= al; }
        __syncthreads();
      }
      l_part += pr;
    }
    // ---- values: keys beyond nk carry p = 0 but their rows are not initialised memory: they are not read
    {
      const uint32_t* vr = reinterpret_cast<const uint32_t*>(Vs) + d2;
      const int s1 = min(nk, (kq + 1) * KPT);
#pragma unroll 4
      for (int s = kq * KPT; s < s1; ++s) {
        const uint32_t u = vr[s * (HD / 2)];
        const float v0 = kv_lo(u), v1 = kv_hi(u);
        float pv[4];
        if constexpr (GP == 4) {
          const float4 t = *reinterpret_cast<const float4*>(ps + s * 4);
          pv[0] = t.x; pv[1] = t.y; pv[2] = t.z; pv[3] = t.w;
        } else if constexpr (GP == 2) {
          const float2 t = *reinterpret_cast<const float2*>(ps + s * 2);
          pv[0] = t.x; pv[1] = t.y;
        } else {
          pv[0] = ps[s];
        }
#pragma unroll
        for (int g = 0; g < GP; ++g) { acc[g][0] = fmaf(pv[g], v0, acc[g][0]); acc[g][1] = fmaf(pv[g], v1, acc[g][1]); }
      }
    }
  }
  if (!ok) {      // copies may still be landing in this CTA's shared memory
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    return;
  }
  __syncthreads();
  if (dq < GP) ps_buf[key * GP + dq] = l_part;     // the heads' sums of probabilities
  __syncthreads();
  if (tid < GP) {
    float l = 0.f;
    for (int i = 0; i < PAGE_TOKENS; ++i) l += ps_buf[i * GP + tid];
    l_run[tid] = l;
  }
  // the key blocks' sums meet in shared memory (the ring is idle: every copy issued was waited for)
  float* red = reinterpret_cast<float*>(ring);                                   // [NKQ][GP][HD]
#pragma unroll
  for (int g = 0; g < GP; ++g)
    *reinterpret_cast<float2*>(red + ((size_t)(kq * GP + g) * HD + 2 * d2)) = make_float2(acc[g][0], acc[g][1]);
  __syncthreads();
  const int ldr = HD + 2;
  for (int o = tid; o < group * HD; o += NT) {
    const int g = o / HD, d = o - g * HD;
    float v = 0.f;
#pragma unroll
    for (int k = 0; k < NKQ; ++k) v += red[(size_t)(k * GP + g) * HD + d];
    const int qh = kvh * group + g;
    if (n_split == 1) out[(size_t)b * nq * HD + (size_t)qh * HD + d] = v / l_run[g];
    else part[(((size_t)b * nq + qh) * n_split + sp) * ldr + d] = v;
  }
  if (n_split > 1 && tid < group) {
    float* pr = part + (((size_t)b * nq + kvh * group + tid) * n_split + sp) * ldr;
    pr[HD] = m_run[tid]; pr[HD + 1] = l_run[tid];
  }
  // With a counter per (sequence, kv head) (zero at launch) the CTA that finishes the group's last split merges the
  // partial results on the spot; without one a separate kernel does it.
  if (n_split > 1 && split_done) {
    __shared__ int s_last;
    __threadfence();                               // this CTA's partial results are visible before it counts itself done
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(split_done + b * nkv + kvh, 1) == n_split - 1;
    __syncthreads();
    if (s_last) {
      __threadfence();
      for (int o = tid; o < group * HD; o += NT) {
        const int g = o / HD, d = o - g * HD;
        const int qh = kvh * group + g;
        const float* pr = part + ((size_t)b * nq + qh) * n_split * ldr;
        float mm = -INFINITY;
        for (int s = 0; s < n_split; ++s) mm = fmaxf(mm, __ldcg(pr + (size_t)s * ldr + HD));
        float ll = 0.f, v = 0.f;
        for (int s = 0; s < n_split; ++s) {
          const float* r = pr + (size_t)s * ldr;
          const float ms = __ldcg(r + HD);
          const float f = (ms == -INFINITY) ? 0.f : __expf(ms - mm);
          ll = fmaf(__ldcg(r + HD + 1), f, ll);
          v = fmaf(__ldcg(r + d), f, v);
        }
        out[(size_t)b * nq * HD + (size_t)qh * HD + d] = v / ll;
      }
    }
  }
}

template <int HD, int GP>
cudaError_t go_ring(dim3 grid, cudaStream_t st, const float* q, int ldq, int nq, int nkv, const InvFreq& inv, const kv16* kpool,
                    const kv16* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra, int n_split,
                    float* part, float* out, int* status, const float* q_gain, float eps, int* split_done) {
  using Cfg = RingCfg<HD, GP>;
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(step_attn_ring_kernel<HD, GP>, (int)Cfg::SMEM, raised);
  if (e != cudaSuccess) return e;
  step_attn_ring_kernel<HD, GP><<<grid, Cfg::NT, Cfg::SMEM, st>>>(q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens,
                                                                  extra, n_split, part, out, status, q_gain, eps, split_done);
  return cudaGetLastError();
}

template <int HD>
cudaError_t go_ring_hd(int group, dim3 grid, cudaStream_t st, const float* q, int ldq, int nq, int nkv, const InvFreq& inv,
                       const kv16* kpool, const kv16* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens,
                       int extra, int n_split, float* part, float* out, int* status, const float* q_gain, float eps, int* split_done) {
  if (group == 1)
    return go_ring<HD, 1>(grid, st, q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, status, q_gain, eps, split_done);
  if (group == 2)
    return go_ring<HD, 2>(grid, st, q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, status, q_gain, eps, split_done);
  return go_ring<HD, 4>(grid, st, q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, status, q_gain, eps, split_done);
}

template <int HD>
cudaError_t go(dim3 grid, int threads, cudaStream_t st, const float* q, int ldq, int nq, int nkv, const InvFreq& inv, const kv16* kpool,
               const kv16* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra, int n_split,
               float* part, float* out, int* status, const float* q_gain, float eps) {
  const size_t smem = (size_t)ST * 2 * PAGE_TOKENS * HD * 2 + (size_t)(MAXG * HD + MAXG * PAGE_TOKENS + 3 * MAXG) * sizeof(float);
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(step_attn_ring_wide_kernel<HD>, (int)smem, raised);
  if (e != cudaSuccess) return e;
  step_attn_ring_wide_kernel<HD><<<grid, threads, smem, st>>>(q, ldq, nq, nkv, inv, kpool, vpool, block_table, mpps, n_pages, seq_lens, extra,
                                                         n_split, part, out, status, q_gain, eps);
  return cudaGetLastError();
}

}  // namespace

// Key-range splits for the ring kernels: at most `upper` (what the partial-result buffer was sized
// for), chosen so that the CTAs fill whole waves of the SMs' resident slots: the cost of a launch is
// waves x (pages per split + about two pages' worth of start-up).
int step_attn_ring_splits(int nq, int nkv, int hd, int batch, int max_keys, int upper) {
  const int group = nq / nkv;
  int per_sm = 2;
  if (group > 4) per_sm = 2;
  else if (hd == 128 && group > 2) per_sm = 1;         // the 512-thread configuration
  const int slots = 148 * per_sm, items = batch * nkv;
  const int n_pg = (max_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  int best = 1; long long best_cost = -1;
  for (int n = 1; n <= upper; ++n) {
    const long long waves = ((long long)items * n + slots - 1) / slots;
    const long long cost = waves * ((n_pg + n - 1) / n + 2);
    if (best_cost < 0 || cost < best_cost) { best = n; best_cost = cost; }
  }
  return best;
}

bool step_attn_ring_supported(int dtype, int nq, int nkv, int hd, const void* kpool, const void* vpool) {
  const int group = nq / nkv;
  return dtype == 1 && (hd == 64 || hd == 128) && group >= 1 && group <= MAXG && ((uintptr_t)kpool & 15) == 0 && ((uintptr_t)vpool & 15) == 0;
}

cudaError_t launch_step_attn_ring(const LaunchCtx& ctx, const float* q, int ldq, int nq, int nkv, int hd, float theta, const void* kpool,
                                  const void* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra,
                                  int batch, int n_split, float* part, float* out, const float* q_gain, float eps, int* split_done) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  dim3 grid(n_split, nkv, batch);
  const int threads = 64 * (nq / nkv);
  ++*ctx.n_launch;
  const int group = nq / nkv;
  if (group <= 4) {
    if (hd == 64)
      return go_ring_hd<64>(group, grid, ctx.st, q, ldq, nq, nkv, inv, (const kv16*)kpool, (const kv16*)vpool, block_table, mpps, n_pages,
                            seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps, split_done);
    return go_ring_hd<128>(group, grid, ctx.st, q, ldq, nq, nkv, inv, (const kv16*)kpool, (const kv16*)vpool, block_table, mpps, n_pages,
                           seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps, split_done);
  }
  if (hd == 64)
    return go<64>(grid, threads, ctx.st, q, ldq, nq, nkv, inv, (const kv16*)kpool, (const kv16*)vpool, block_table, mpps, n_pages, seq_lens,
                  extra, n_split, part, out, ctx.status, q_gain, eps);
  return go<128>(grid, threads, ctx.st, q, ldq, nq, nkv, inv, (const kv16*)kpool, (const kv16*)vpool, block_table, mpps, n_pages, seq_lens,
                 extra, n_split, part, out, ctx.status, q_gain, eps);
}
