// Single-query GQA attention of the base step over the paged half-precision cache on the warp-level
// tensor-core path (mma.sync m16n8k16, fp32 accumulation).
//
// The CUDA-core kernels of step_attn.cu spend about 300 instructions per thread and page and are bound by
// instruction issue at a third of the HBM rate.  Here the arithmetic per cached element is almost free:
//   grid (key-range split, kv head, sequence); a CTA serves the group's query heads (up to 8) and walks its
//   range of cache pages.  Warp 4 fetches pages with TMA through a tensor map over the layer's pool (64 x 64
//   boxes, 128-byte swizzle, so that the matrix loads below are free of bank conflicts) into a ring of stages;
//   warps 0-3 each take 16 of a page's 64 keys:
//   scores   S[16 x 16] = Q K^T: rows g / g + 8 of the A operand carry the half-precision value / remainder of
//            query head g (the two accumulator rows are added), K fragments by ldmatrix
//   softmax  per warp, online, on the 4 lanes that own a head's row; the rescale of what has been accumulated
//            happens only when a row maximum grows
//   values   O[16 x hd] += P V with P as value / remainder rows like Q, V fragments by transposing ldmatrix
//   The four warps' (max, sum, O) meet in shared memory after the last page; key-range splits are merged by the
//   CTA that finishes a group's last split (counter per (sequence, kv head)), as in step_attn.cu.
// Every wait is bounded (DEV_TIMEOUT, the CTA leaves); page ids are checked before they are used as coordinates.
#include <math.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int NW = 4;                       // consumer warps
constexpr int NT = (NW + 1) * 32;
constexpr int BOX_BYTES = 64 * 128;         // one 64-key x 64-dim box

template <int HD> struct MmaCfg {
  static constexpr int PAGE_BYTES = PAGE_TOKENS * HD * 2;
  static constexpr int STAGES = HD == 64 ? 5 : 3;          // two CTAs per SM
  static constexpr int RING = STAGES * 2 * PAGE_BYTES;
  // after the ring: q [8][HD] fp32, then the warps' partial results [NW][8][HD + 2] fp32 (reuses the ring when it is idle)
  static constexpr int SMEM = 1024 + RING + 8 * HD * 4 + 256;
};

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (value, remainder) of two floats as packed halves
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(x, y);
  const float2 f = __half22float2(h);
  const __half2 l = __floats2half2_rn(x - f.x, y - f.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}
// byte offset of the 16-byte piece `c` (8 dims) of key `k` inside a page stored as 64 x 64 boxes with the 128-byte swizzle
__device__ __forceinline__ uint32_t piece(int k, int c) { return (uint32_t)((c >> 3) * BOX_BYTES + k * 128 + (((c & 7) ^ (k & 7)) << 4)); }

struct MmaParams {
  const float* q; int ldq, nq, nkv;
  const int* block_table; int mpps, n_pages;
  const int* seq_lens; int extra, n_split;
  float* part; float* out; int* status;
  const float* q_gain; float eps;
  int* split_done;
  int per_pages;            // pages per CTA
};

template <int HD>
__global__ void __launch_bounds__(NT, 2)
step_attn_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const __grid_constant__ InvFreq inv, const MmaParams p) {
  using Cfg = MmaCfg<HD>;
  constexpr int STG = Cfg::STAGES, PB = Cfg::PAGE_BYTES, KS = HD / 16, NTL = HD / 8;
  extern __shared__ uint8_t sm_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(sm_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t ring = smem_u32(smem);
  float* qs = reinterpret_cast<float*>(smem + Cfg::RING);                        // [8][HD], scaled, after RoPE
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::RING + 8 * HD * 4);   // full[STG], empty[STG]
  __shared__ int s_abort_mem;
  __shared__ float rq[8];
  __shared__ int s_last;
  volatile int* abort_flag = &s_abort_mem;
  const uint32_t bar_base = smem_u32(bars);
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (STG + s); };
  const int group = p.nq / p.nkv;                  // <= 8
  const int sp = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_keys = p.seq_lens[b] + p.extra;
  const int pos = n_keys - 1;
  const int n_pg = (n_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  // every CTA walks at most `per_pages` pages, so a short sequence takes fewer CTAs instead of shorter ranges:
  // its surplus CTAs leave at once and the launch is as long as per_pages pages, not as the longest sequence's share
  // (a sequence that has grown since the launch shape was chosen, as in a replayed generation step, leaves its surplus
  // pages to the last CTA)
  const int my_splits = min(p.n_split, max(1, (n_pg + p.per_pages - 1) / p.per_pages));
  if (sp >= my_splits) return;
  const int pg0 = sp * p.per_pages, pg1 = sp == my_splits - 1 ? n_pg : pg0 + p.per_pages;
  const int n_it = max(pg1 - pg0, 0);
  if (tid == 0) {
    for (int s = 0; s < STG; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), NW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid == 32) { prefetch_tensormap(&map_k); prefetch_tensormap(&map_v); }
  // queries of the group: (query norm,) RoPE at the last position, scaled by 1/sqrt(hd); rows beyond the group are zero
  if (p.q_gain) head_rnorm(p.q + (size_t)b * p.ldq + (size_t)kvh * group * HD, group, HD, p.eps, rq);
  {
    const float scale = rsqrtf((float)HD);
    constexpr int half = HD / 2;
    for (int i = tid; i < 8 * half; i += NT) {
      const int h = i / half, c = i - h * half;
      float r1 = 0.f, r2 = 0.f;
      if (h < group) {
        const float* qh = p.q + (size_t)b * p.ldq + (size_t)(kvh * group + h) * HD;
        float sn, cs;
        rope_sincos(pos, inv.f[c], &sn, &cs);
        float x1 = qh[c], x2 = qh[c + half];
        if (p.q_gain) { x1 *= rq[h] * p.q_gain[c]; x2 *= rq[h] * p.q_gain[c + half]; }
        r1 = (x1 * cs - x2 * sn) * scale;
        r2 = (x2 * cs + x1 * sn) * scale;
      }
      qs[h * HD + c] = r1;
      qs[h * HD + c + half] = r2;
    }
  }
  __syncthreads();

  const int g = lane >> 2, qd = lane & 3;          // this lane's row (query head) and position in the row's quad
  float o[NTL][4];                                  // O fragments: [dims 8j..8j+7]: rows g (from P's value part), g + 8 (remainder part)
#pragma unroll
  for (int j = 0; j < NTL; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_run = -INFINITY, l_run = 0.f;
  bool ok = true;

  if (warp == NW) {
    // ---------------- producer: pages of the range through the ring ----------------
    if (lane == 0) {
      for (int it = 0; it < n_it && ok; ++it) {
        const int s = it % STG;
        if (it >= STG) ok = mbar_wait(empty(s), ((it / STG) - 1) & 1u, abort_flag, p.status);
        if (!ok) break;
        const int pg = pg0 + it;
        const int page = pg < p.mpps ? p.block_table[(size_t)b * p.mpps + pg] : -1;
        if (page < 0 || page >= p.n_pages) {       // never used as a coordinate: the stage completes empty, consumers skip the page
          dev_flag(p.status, DEV_BAD_PAGE);
          mbar_arrive(full(s));
          continue;
        }
        const int row0 = (page * p.nkv + kvh) * PAGE_TOKENS;
        const uint32_t dst = ring + s * 2 * PB;
        mbar_expect_tx(full(s), 2 * PB);
#pragma unroll
        for (int x = 0; x < HD / 64; ++x) {
          tma_load_2d(dst + x * BOX_BYTES, &map_k, x * 64, row0, full(s));
          tma_load_2d(dst + PB + x * BOX_BYTES, &map_v, x * 64, row0, full(s));
        }
      }
      if (!ok) drain_after_abort();
    }
  } else {
    // ---------------- consumers: warp w takes keys 16 w .. 16 w + 15 of every page ----------------
    uint32_t qa[KS][4];                             // A fragments of Q: rows g = value part, g + 8 = remainder part
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const float* qrow = qs + g * HD + ks * 16 + 2 * qd;
      split2(qrow[0], qrow[1], qa[ks][0], qa[ks][1]);
      split2(qrow[8], qrow[9], qa[ks][2], qa[ks][3]);
    }
    const int k_lane = warp * 16 + (lane & 7);      // key row this lane addresses in matrix loads (+ 8 for the second key block)
    const int mi = lane >> 3;                        // which of the four 8 x 8 matrices of a load this lane addresses
    for (int it = 0; it < n_it; ++it) {
      const int s = it % STG;
      ok = mbar_wait(full(s), (it / STG) & 1u, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int pg = pg0 + it;
      const int page = pg < p.mpps ? p.block_table[(size_t)b * p.mpps + pg] : -1;
      const int nk = (page >= 0 && page < p.n_pages) ? min(PAGE_TOKENS, n_keys - pg * PAGE_TOKENS) : 0;
      if (warp * 16 < nk) {
        const uint32_t sk = ring + s * 2 * PB, sv = sk + PB;
        // ---- scores of this warp's 16 keys: two 8-key blocks
        float sc[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) { sc[t][0] = sc[t][1] = sc[t][2] = sc[t][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          uint32_t kb[4];        // matrices: (keys 0-7, dims 16ks..+7), (keys 0-7, dims +8..+15), (keys 8-15, ..), (keys 8-15, ..)
          ldsm4(sk + piece(k_lane + (mi >> 1) * 8, 2 * ks + (mi & 1)), kb);
          mma16816(sc[0], qa[ks], kb[0], kb[1]);
          mma16816(sc[1], qa[ks], kb[2], kb[3]);
        }
        // value row + remainder row of head g: this lane holds keys 2 qd, 2 qd + 1 of each 8-key block
        float sv4[4];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          sv4[2 * t] = sc[t][0] + sc[t][2];
          sv4[2 * t + 1] = sc[t][1] + sc[t][3];
          const int key0 = warp * 16 + t * 8 + 2 * qd;
          if (key0 >= nk) sv4[2 * t] = -INFINITY;
          if (key0 + 1 >= nk) sv4[2 * t + 1] = -INFINITY;
        }
        float mt = fmaxf(fmaxf(sv4[0], sv4[1]), fmaxf(sv4[2], sv4[3]));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
        if (mt > m_run) {                             // the row's maximum grows: rescale what this lane holds of the row
          const float a = (m_run == -INFINITY) ? 0.f : __expf(m_run - mt);
          l_run *= a;
#pragma unroll
          for (int j = 0; j < NTL; ++j) { o[j][0] *= a; o[j][1] *= a; o[j][2] *= a; o[j][3] *= a; }
          m_run = mt;
        }
        float pr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { pr[i] = (sv4[i] == -INFINITY) ? 0.f : __expf(sv4[i] - m_run); l_run += pr[i]; }
        uint32_t pa[4];          // A fragment of P: (row g, keys 2qd..) value, (row g + 8) remainder, then the second key block
        split2(pr[0], pr[1], pa[0], pa[1]);
        split2(pr[2], pr[3], pa[2], pa[3]);
        // ---- values: O[16 x HD] += P[16 x 16 keys] V[16 keys x HD]
#pragma unroll
        for (int j = 0; j < NTL; j += 2) {
          uint32_t vb[4];        // matrices: (keys 0-7, dims 8j..), (keys 8-15, dims 8j..), (keys 0-7, dims 8(j+1)..), (keys 8-15, ..)
          ldsm4_t(sv + piece(k_lane + (mi & 1) * 8, j + (mi >> 1)), vb);
          mma16816(o[j], pa, vb[0], vb[1]);
          mma16816(o[j + 1], pa, vb[2], vb[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty(s));           // this warp is through with the stage
    }
  }
  // every thread learns whether some wait ran out (copies may then still be landing in this CTA's shared memory)
  if (!__syncthreads_and(ok && *abort_flag == 0)) {
    drain_after_abort();
    return;
  }
  // ---- the four warps' partial results meet in shared memory (the ring is idle: every copy issued was waited for)
  constexpr int LDR = HD + 2;
  float* red = reinterpret_cast<float*>(smem);                                   // [NW][8][HD + 2]
  if (warp < NW) {
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    float* r = red + (size_t)(warp * 8 + g) * LDR;
#pragma unroll
    for (int j = 0; j < NTL; ++j)
      *reinterpret_cast<float2*>(r + 8 * j + 2 * qd) = make_float2(o[j][0] + o[j][2], o[j][1] + o[j][3]);
    if (qd == 0) { r[HD] = m_run; r[HD + 1] = l_run; }
  }
  __syncthreads();
  const int ldr = HD + 2;
  for (int e = tid; e < group * HD; e += NT) {
    const int gg = e / HD, d = e - gg * HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) mm = fmaxf(mm, red[(size_t)(w * 8 + gg) * LDR + HD]);
    float v = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float* r = red + (size_t)(w * 8 + gg) * LDR;
      const float f = (r[HD] == -INFINITY) ? 0.f : __expf(r[HD] - mm);
      v = fmaf(r[d], f, v);
      l = fmaf(r[HD + 1], f, l);
    }
    const int qh = kvh * group + gg;
    if (my_splits == 1) {
      p.out[(size_t)b * p.nq * HD + (size_t)qh * HD + d] = v / l;
    } else {
      float* pr = p.part + (((size_t)b * p.nq + qh) * p.n_split + sp) * ldr;
      pr[d] = v;
      if (d == 0) { pr[HD] = mm; pr[HD + 1] = l; }
    }
  }
  // With more than one split the CTA that finishes the group's last split merges the partial results on the spot
  // (counter per (sequence, kv head), zero at launch).
  if (my_splits > 1) {
    __threadfence();                               // this CTA's partial results are visible before it counts itself done
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(p.split_done + b * p.nkv + kvh, 1) == my_splits - 1;
    __syncthreads();
    if (s_last) {
      __threadfence();
      for (int e = tid; e < group * HD; e += NT) {
        const int gg = e / HD, d = e - gg * HD;
        const int qh = kvh * group + gg;
        const float* pr = p.part + ((size_t)b * p.nq + qh) * p.n_split * ldr;
        float mm = -INFINITY;
        for (int s = 0; s < my_splits; ++s) mm = fmaxf(mm, __ldcg(pr + (size_t)s * ldr + HD));
        float ll = 0.f, v = 0.f;
        for (int s = 0; s < my_splits; ++s) {
          const float* r = pr + (size_t)s * ldr;
          const float ms = __ldcg(r + HD);
          const float f = (ms == -INFINITY) ? 0.f : __expf(ms - mm);
          ll = fmaf(__ldcg(r + HD + 1), f, ll);
          v = fmaf(__ldcg(r + d), f, v);
        }
        p.out[(size_t)b * p.nq * HD + (size_t)qh * HD + d] = v / ll;
      }
    }
  }
}

// fp16 pool [rows, hd] row-major; box = 64 dims x 64 keys, 128-byte swizzle
bool make_pool_map(CUtensorMap* m, const void* pool, long long rows, int hd) {
  return tc_make_map_bf16(m, pool, rows, hd, hd, 64);      // halves are 2-byte elements like bf16 for the copy engine
}

template <int HD>
cudaError_t go_mma(const CUtensorMap& mk, const CUtensorMap& mv, const InvFreq& inv, const MmaParams& p, dim3 grid, cudaStream_t st) {
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(step_attn_mma_kernel<HD>, MmaCfg<HD>::SMEM, raised);
  if (e != cudaSuccess) return e;
  step_attn_mma_kernel<HD><<<grid, NT, MmaCfg<HD>::SMEM, st>>>(mk, mv, inv, p);
  return cudaGetLastError();
}

}  // namespace

// Key-range splits: at most `upper`, chosen so that the CTAs fill whole waves of the two resident slots per SM.
int step_attn_mma_splits(int batch, int nkv, int max_keys, int upper) {
  const int slots = 148 * 2, items = batch * nkv;
  const int n_pg = (max_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  int best = 1; long long best_cost = -1;
  for (int n = 1; n <= upper; ++n) {
    const long long waves = ((long long)items * n + slots - 1) / slots;
    const long long cost = waves * ((n_pg + n - 1) / n + 3);
    if (best_cost < 0 || cost < best_cost) { best = n; best_cost = cost; }
  }
  return best;
}

bool step_attn_mma_supported(int dtype, int nq, int nkv, int hd, const void* kpool, const void* vpool, int n_pages) {
  const int group = nq / nkv;
  return dtype == 1 && (hd == 64 || hd == 128) && group >= 1 && group <= 8 && ((uintptr_t)kpool & 15) == 0 && ((uintptr_t)vpool & 15) == 0 &&
         (long long)n_pages * nkv * PAGE_TOKENS < (1LL << 31) && tc_encode_fn() != nullptr;
}

cudaError_t launch_step_attn_mma(const LaunchCtx& ctx, const float* q, int ldq, int nq, int nkv, int hd, float theta, const void* kpool,
                                 const void* vpool, const int* block_table, int mpps, int n_pages, const int* seq_lens, int extra,
                                 int batch, int n_split, int max_keys, float* part, float* out, const float* q_gain, float eps,
                                 int* split_done) {
  if (n_split > 1 && !split_done) return cudaErrorInvalidValue;
  const int max_pg = (max_keys + PAGE_TOKENS - 1) / PAGE_TOKENS;
  const int per_pages = (max_pg + n_split - 1) / n_split > 0 ? (max_pg + n_split - 1) / n_split : 1;
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  CUtensorMap mk, mv;
  const long long rows = (long long)n_pages * nkv * PAGE_TOKENS;
  if (!make_pool_map(&mk, kpool, rows, hd) || !make_pool_map(&mv, vpool, rows, hd)) return cudaErrorInvalidValue;
  MmaParams p{q, ldq, nq, nkv, block_table, mpps, n_pages, seq_lens, extra, n_split, part, out, ctx.status, q_gain, eps, split_done, per_pages};
  dim3 grid(n_split, nkv, batch);
  ++*ctx.n_launch;
  return hd == 64 ? go_mma<64>(mk, mv, inv, p, grid, ctx.st) : go_mma<128>(mk, mv, inv, p, grid, ctx.st);
}
