// K/V projection of one auxiliary layer with the KV predictor as its epilogue (Sec. 4.2 of the paper:
// K_hat_i = K_A,j FK_i^T, V_hat_i = V_A,j FV_i^T for every base layer i with j_i = j), sm_100a.
//
// One work item = 128 tokens x (K or V).  A persistent CTA per SM:
//   phase 1  acc1[128, d_kvA] = h_hi Wkv^T + h_lo Wkv^T  (bf16 operands by TMA, fp32 accumulator in tensor memory)
//   epilogue 1 (4 warps, a thread per token row): 1 / rms of the folded RMSNorm, key norm, RoPE; the result goes
//            (a) as bf16 to the layer's q|k|v buffer (the auxiliary attention reads it) and
//            (b) as IEEE halves into shared memory in the swizzled operand layout: the A operand of phase 2,
//                which therefore never travels through global memory
//   phase 2  for every 128 columns of the stacked predictor matrices of the base layers this auxiliary layer feeds:
//            acc2[128, 128] = A2[128, d_kvA] F_chunk^T (halves, one pass), four accumulators in rotation
//   epilogue 2: (+ bias) -> halves, 64-byte stores straight into the cache pages of the base layer a column belongs to.
// The operand ring in shared memory serves both phases (48-64 KiB stages in phase 1, 16 KiB slots in phase 2).
// Warp 0 loads h (phase 1) and F (phase 2), warp 2 loads Wkv, warp 1 issues the MMAs, warps 3-6 are the epilogue.
// Every mbarrier wait is bounded (DEV_TIMEOUT; all roles leave, tensor memory is freed).
#include <math.h>

#include "kvpred_tc.h"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int BM = 128, BK = 64;
constexpr int N_THREADS = 224;
constexpr int NC = 128;                   // predictor output columns per accumulator
constexpr int A_BYTES = BM * BK * 2;      // 16 KiB: a k block of the token tile
constexpr int SLOT2 = NC * BK * 2;        // 16 KiB: a k block of one output chunk of F
constexpr int MAX_S1 = 4, MAX_S2 = 10, N_ACC2 = 4;
constexpr int SMEM_TOTAL = 227 * 1024;
constexpr int BAR_BYTES = 512;

struct Params {
  int M, K, dkv, n_tot, hd, kv_begin, kv_end;
  int stages1, slots2, stage1_bytes, a2_bytes;
  int has_lo;
  const float* ss_in; float rms_eps;
  const float2* rope_tab; int tab_stride; const int* tok_pos;
  const float* k_gain; float eps;
  bf16* C; int ldc; int k_col;
  PagedOut paged[2];
  int* status;
};

__device__ __forceinline__ uint32_t idesc_f16(int m, int n) {     // IEEE half operands, fp32 accumulator, both K-major
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ uint4 halves8(const float* v) {
  uint4 u;
  uint32_t* w = &u.x;
#pragma unroll
  for (int i = 0; i < 4; ++i) w[i] = half2_sat(v[2 * i], v[2 * i + 1]);
  return u;
}
__device__ __forceinline__ uint4 bf16x8(const float* v) {
  uint4 u;
  uint32_t* w = &u.x;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  return u;
}

// 32 values of token row r, columns n .. n + 31 of K_A or V_A: bf16 to the q|k|v buffer, halves into the phase-2 operand
__device__ __forceinline__ void put32(const Params& p, uint32_t sA2, int r, int m, bool row_ok, int col0, int n, const float* v) {
  const uint32_t base = sA2 + (uint32_t)(n >> 6) * A_BYTES + r * 128;
  const int c16 = (n & 63) >> 3;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const uint4 u = halves8(v + g * 8);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + (((c16 + g) ^ (r & 7)) << 4)), "r"(u.x), "r"(u.y), "r"(u.z), "r"(u.w) : "memory");
  }
  if (row_ok) {
    bf16* dst = p.C + (size_t)m * p.ldc + col0 + n;
#pragma unroll
    for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(dst + g * 8) = bf16x8(v + g * 8);
  }
}

__global__ void __launch_bounds__(N_THREADS, 1)
kvpred_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a2,
                 const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_fk,
                 const __grid_constant__ CUtensorMap map_fv, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sA2 = smem_u32(smem);                       // phase-2 A operand: dkv / 64 k blocks of 16 KiB
  const uint32_t ring = sA2 + p.a2_bytes;
  const int ring_bytes = p.stages1 * p.stage1_bytes > p.slots2 * SLOT2 ? p.stages1 * p.stage1_bytes : p.slots2 * SLOT2;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.a2_bytes + ring_bytes);
  const uint32_t bar_base = smem_u32(bars);
  // full1[4] empty1[4] full2[10] empty2[10] acc2_full[4] acc2_empty[4] acc1_full a2_ready p2_done
  auto full1 = [&](int s) { return bar_base + 8u * s; };
  auto empty1 = [&](int s) { return bar_base + 8u * (MAX_S1 + s); };
  auto full2 = [&](int s) { return bar_base + 8u * (2 * MAX_S1 + s); };
  auto empty2 = [&](int s) { return bar_base + 8u * (2 * MAX_S1 + MAX_S2 + s); };
  auto acc2_full = [&](int b) { return bar_base + 8u * (2 * MAX_S1 + 2 * MAX_S2 + b); };
  auto acc2_empty = [&](int b) { return bar_base + 8u * (2 * MAX_S1 + 2 * MAX_S2 + N_ACC2 + b); };
  const uint32_t acc1_full = bar_base + 8u * (2 * MAX_S1 + 2 * MAX_S2 + 2 * N_ACC2);
  const uint32_t a2_ready = acc1_full + 8u, p2_done = acc1_full + 16u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_S1 + 2 * MAX_S2 + 2 * N_ACC2 + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();
  if (threadIdx.x == 32) {
    prefetch_tensormap(&map_a); prefetch_tensormap(&map_w); prefetch_tensormap(&map_fk); prefetch_tensormap(&map_fv);
    if (p.has_lo) prefetch_tensormap(&map_a2);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_S1; ++s) { mbar_init(full1(s), 2); mbar_init(empty1(s), 1); }
    for (int s = 0; s < MAX_S2; ++s) { mbar_init(full2(s), 1); mbar_init(empty2(s), 1); }
    for (int b = 0; b < N_ACC2; ++b) { mbar_init(acc2_full(b), 1); mbar_init(acc2_empty(b), 4); }
    mbar_init(acc1_full, 1); mbar_init(a2_ready, 4); mbar_init(p2_done, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();

  const int m_blocks = (p.M + BM - 1) / BM;
  const int n_kv = p.kv_end - p.kv_begin;
  const int n_items = m_blocks * n_kv;
  const int nkb1 = (p.K + BK - 1) / BK, n_it1 = (p.has_lo ? 2 : 1) * nkb1;
  const int nkb2 = p.dkv / BK;
  const int n_chunks = (p.n_tot + NC - 1) / NC;
  const int w_bytes = p.dkv * BK * 2;

  if (warp == 0 || warp == 2) {
    // ---------------- loaders ----------------
    if (lane == 0) {
      const bool is_a = warp == 0;
      int st1 = 0, sl2 = 0; uint32_t ph1 = 0, ph2 = 0, item_par = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        const int m0 = (it / n_kv) * BM, kv = p.kv_begin + it % n_kv;
        for (int i = 0; i < n_it1 && ok; ++i) {
          ok = mbar_wait(empty1(st1), ph1 ^ 1u, abort_flag, p.status);
          if (!ok) break;
          const int kb = i < nkb1 ? i : i - nkb1;
          const uint32_t sa = ring + st1 * p.stage1_bytes;
          if (is_a) {
            mbar_expect_tx(full1(st1), A_BYTES);
            tma_load_2d(sa, i < nkb1 ? &map_a : &map_a2, kb * BK, m0, full1(st1));
          } else {
            mbar_expect_tx(full1(st1), w_bytes);
            for (int r = 0; r < p.dkv; r += 64) tma_load_2d(sa + A_BYTES + r * 128, &map_w, kb * BK, kv * p.dkv + r, full1(st1));
          }
          if (++st1 == p.stages1) { st1 = 0; ph1 ^= 1u; }
        }
        if (!ok) break;
        if (is_a) {     // phase 2: the ring is free of phase-1 reads once the projection's accumulator is complete
          ok = mbar_wait(acc1_full, item_par, abort_flag, p.status);
          for (int c = 0; c < n_chunks && ok; ++c) {
            const int rows = min(NC, p.n_tot - c * NC);
            for (int kb = 0; kb < nkb2 && ok; ++kb) {
              ok = mbar_wait(empty2(sl2), ph2 ^ 1u, abort_flag, p.status);
              if (!ok) break;
              mbar_expect_tx(full2(sl2), rows * 128);
              for (int r = 0; r < rows; r += 64)
                tma_load_2d(ring + sl2 * SLOT2 + r * 128, kv ? &map_fv : &map_fk, kb * BK, c * NC + r, full2(sl2));
              if (++sl2 == p.slots2) { sl2 = 0; ph2 ^= 1u; }
            }
          }
        }
        // the next item's projection operands overwrite the ring: every phase-2 MMA must have read its slot
        if (ok) ok = mbar_wait(p2_done, item_par, abort_flag, p.status);
        item_par ^= 1u;
      }
      if (!ok) drain_after_abort();
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int st1 = 0, sl2 = 0; uint32_t ph1 = 0, ph2 = 0, item_par = 0;
      uint32_t acc_uses = 0;        // chunks issued so far (accumulator c % 4, parity from the use count)
      bool ok = true;
      const int n_lo = p.dkv > 256 ? 256 : p.dkv, n_hi = p.dkv - n_lo;
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        // phase 1 writes columns [0, dkv): every phase-2 accumulator of the previous item must have been drained
        for (int b = 0; b < N_ACC2 && ok; ++b) {
          const uint32_t uses = (acc_uses + N_ACC2 - 1 - b) / N_ACC2;     // times accumulator b has been filled
          if (uses > 0) ok = mbar_wait(acc2_empty(b), (uses - 1) & 1u, abort_flag, p.status);
        }
        if (!ok) break;
        tc_fence_after();
        for (int i = 0; i < n_it1 && ok; ++i) {
          ok = mbar_wait(full1(st1), ph1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = ring + st1 * p.stage1_bytes, sw = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint32_t accum = (i > 0 || k > 0) ? 1u : 0u;
            tc_mma_bf16(tmem_base, desc_kmajor(sa) + 2u * k, desc_kmajor(sw) + 2u * k, idesc_bf16(BM, n_lo), accum);
            if (n_hi > 0)
              tc_mma_bf16(tmem_base + 256, desc_kmajor(sa) + 2u * k, desc_kmajor(sw + 256 * 128) + 2u * k, idesc_bf16(BM, n_hi), accum);
          }
          tc_commit(empty1(st1));
          if (++st1 == p.stages1) { st1 = 0; ph1 ^= 1u; }
        }
        if (!ok) break;
        tc_commit(acc1_full);
        // phase 2
        ok = mbar_wait(a2_ready, item_par, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        for (int c = 0; c < n_chunks && ok; ++c) {
          const int b = acc_uses % N_ACC2;
          const uint32_t uses = acc_uses / N_ACC2;
          // within an item the first four chunks find their accumulators free (checked above); later ones wait for the epilogue
          if (c >= N_ACC2) ok = mbar_wait(acc2_empty(b), (uses - 1) & 1u, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const int rows = min(NC, p.n_tot - c * NC);
          for (int kb = 0; kb < nkb2 && ok; ++kb) {
            ok = mbar_wait(full2(sl2), ph2, abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sf = ring + sl2 * SLOT2;
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              tc_mma_bf16(tmem_base + b * NC, desc_kmajor(sA2 + kb * A_BYTES) + 2u * k, desc_kmajor(sf) + 2u * k, idesc_f16(BM, rows),
                          (kb > 0 || k > 0) ? 1u : 0u);
            tc_commit(empty2(sl2));
            if (++sl2 == p.slots2) { sl2 = 0; ph2 ^= 1u; }
          }
          if (ok) tc_commit(acc2_full(b));
          ++acc_uses;
        }
        if (ok) tc_commit(p2_done);
        item_par ^= 1u;
      }
      if (!ok) drain_after_abort();
    }
  } else {
    // ---------------- epilogue ----------------
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t tlane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    uint32_t item_par = 0, acc_uses = 0;
    bool ok = true;
    for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
      const int m0 = (it / n_kv) * BM, kv = p.kv_begin + it % n_kv;
      const int m = m0 + r;
      const bool row_ok = m < p.M;
      ok = mbar_wait(acc1_full, item_par, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const float rinv = (p.ss_in && row_ok) ? rsqrtf(p.ss_in[m] / (float)p.K + p.rms_eps) : 1.f;
      const int col0 = p.k_col + kv * p.dkv;
      if (kv == 0) {      // keys: (key norm,) RoPE on the pairs (c, c + hd / 2) of every head
        const int half = p.hd >> 1;
        const float4* tab = reinterpret_cast<const float4*>(p.rope_tab) + (row_ok ? p.tok_pos[m] : 0);
#pragma unroll 1
        for (int h0 = 0; h0 < p.dkv; h0 += p.hd) {
          float rn = rinv;
          if (p.k_gain) {
            float ss = 0.f;
#pragma unroll 1
            for (int j = 0; j < p.hd; j += 32) {
              float a[32];
              tmem_ld32(tlane + h0 + j, a);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) ss = fmaf(a[i], a[i], ss);
            }
            rn = rinv * rsqrtf(ss * rinv * rinv / (float)p.hd + p.eps);
          }
#pragma unroll 1
          for (int j = 0; j < half; j += 32) {
            float a[32], b[32];
            tmem_ld32(tlane + h0 + j, a);
            tmem_ld32(tlane + h0 + half + j, b);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              a[i] *= rn; b[i] *= rn;
              if (p.k_gain) { a[i] *= p.k_gain[j + i]; b[i] *= p.k_gain[half + j + i]; }
            }
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float4 cs = tab[(size_t)((j + i) >> 1) * p.tab_stride];     // (cos, sin) of two frequencies
              float x1 = a[i], x2 = b[i];
              a[i] = x1 * cs.x - x2 * cs.y; b[i] = x2 * cs.x + x1 * cs.y;
              x1 = a[i + 1]; x2 = b[i + 1];
              a[i + 1] = x1 * cs.z - x2 * cs.w; b[i + 1] = x2 * cs.z + x1 * cs.w;
            }
            put32(p, sA2, r, m, row_ok, col0, h0 + j, a);
            put32(p, sA2, r, m, row_ok, col0, h0 + half + j, b);
          }
        }
      } else {            // values
#pragma unroll 1
        for (int n = 0; n < p.dkv; n += 32) {
          float a[32];
          tmem_ld32(tlane + n, a);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) a[i] *= rinv;
          put32(p, sA2, r, m, row_ok, col0, n, a);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the operand is read by the tensor core
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(a2_ready);
      // epilogue 2: predicted columns into cache pages
      const PagedOut& q = p.paged[kv];
      const int slot = row_ok ? q.tok_slot[m] : -1;
      const int page = slot / PAGE_TOKENS, prow = slot - page * PAGE_TOKENS;
      for (int c = 0; c < n_chunks; ++c) {
        const int b = acc_uses % N_ACC2;
        ok = mbar_wait(acc2_full(b), (acc_uses / N_ACC2) & 1u, abort_flag, p.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const int cols = min(NC, p.n_tot - c * NC);
#pragma unroll 1
        for (int cc = 0; cc < cols; cc += 32) {
          float v[32];
          tmem_ld32(tlane + b * NC + cc, v);
          tmem_ld_wait();
          if (slot < 0) continue;
          const int n = c * NC + cc;
          int s = 0;
          while (s + 1 < q.n_seg && n >= q.col0[s + 1]) ++s;
          const int in_seg = n - q.col0[s];
          const int head = in_seg / q.head_dim, dim = in_seg - head * q.head_dim;
          if (q.bias) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] += q.bias[n + i];
          }
          kv16* dst = (kv16*)q.pool[s] + (((size_t)page * q.n_kv[s] + head) * PAGE_TOKENS + prow) * q.head_dim + dim;
#pragma unroll
          for (int g = 0; g < 4; ++g) *reinterpret_cast<uint4*>(dst + g * 8) = halves8(v + g * 8);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc2_empty(b));
        ++acc_uses;
      }
      if (!ok) break;
      item_par ^= 1u;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool kvpred_tc_supported(const KvPred& g) {
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (g.M <= 0 || g.K <= 0 || g.K % 8 || g.lda % 8 || g.ldw % 8 || !al16(g.A) || !al16(g.Wkv)) return false;
  if (g.A_lo && (g.lda_lo % 8 || !al16(g.A_lo))) return false;
  if (g.dkv % 64 || g.dkv < 64 || g.dkv > 384 || (g.hd != 64 && g.hd != 128) || g.dkv % g.hd) return false;
  if (g.ldc % 8 || !al16(g.C) || g.k_col % 8 || !g.rope_tab || !g.tok_pos) return false;
  for (int kv = g.kv_begin; kv < g.kv_end; ++kv) {
    const PagedOut& q = g.paged[kv];
    if (q.n_seg < 1 || q.head_dim % 32 || q.col0[q.n_seg] != g.n_tot || !q.tok_slot) return false;
    for (int s = 0; s <= q.n_seg; ++s) if (q.col0[s] % 32) return false;
  }
  if (g.n_tot % 64 || g.n_tot < 64 || !al16(g.FK) || !al16(g.FV)) return false;
  return g.kv_begin >= 0 && g.kv_end <= 2 && g.kv_begin < g.kv_end;
}

cudaError_t launch_kvpred_tc(const KvPred& g, int* status, cudaStream_t st, int64_t* n_launch) {
  if (!tc_encode_fn()) return cudaErrorNotSupported;
  CUtensorMap ma, ma2, mw, mfk, mfv;
  if (!tc_make_map_bf16(&ma, g.A, g.M, g.K, g.lda, BM)) return cudaErrorInvalidValue;
  if (g.A_lo) { if (!tc_make_map_bf16(&ma2, g.A_lo, g.M, g.K, g.lda_lo, BM)) return cudaErrorInvalidValue; }
  else ma2 = ma;
  if (!tc_make_map_bf16(&mw, g.Wkv, 2LL * g.dkv, g.K, g.ldw, 64)) return cudaErrorInvalidValue;
  // (the predictor matrices hold IEEE halves: for the copy engine they are 2-byte elements like bf16)
  if (!tc_make_map_bf16(&mfk, g.FK, g.n_tot, g.dkv, g.dkv, 64)) return cudaErrorInvalidValue;
  if (!tc_make_map_bf16(&mfv, g.FV, g.n_tot, g.dkv, g.dkv, 64)) return cudaErrorInvalidValue;
  Params p{};
  p.M = g.M; p.K = g.K; p.dkv = g.dkv; p.n_tot = g.n_tot; p.hd = g.hd; p.kv_begin = g.kv_begin; p.kv_end = g.kv_end;
  p.has_lo = g.A_lo != nullptr;
  p.ss_in = g.ss_in; p.rms_eps = g.rms_eps; p.rope_tab = g.rope_tab; p.tab_stride = g.tab_stride; p.tok_pos = g.tok_pos; p.k_gain = g.k_gain; p.eps = g.eps;
  p.C = g.C; p.ldc = g.ldc; p.k_col = g.k_col; p.paged[0] = g.paged[0]; p.paged[1] = g.paged[1]; p.status = status;
  p.a2_bytes = (g.dkv / BK) * A_BYTES;
  p.stage1_bytes = A_BYTES + g.dkv * BK * 2;
  const int ring = (SMEM_TOTAL - 1024 - BAR_BYTES - p.a2_bytes) / 1024 * 1024;
  p.stages1 = ring / p.stage1_bytes;
  if (p.stages1 > MAX_S1) p.stages1 = MAX_S1;
  p.slots2 = ring / SLOT2;
  if (p.slots2 > MAX_S2) p.slots2 = MAX_S2;
  if (p.stages1 < 2 || p.slots2 < 2) return cudaErrorInvalidValue;
  const int ring_used = p.stages1 * p.stage1_bytes > p.slots2 * SLOT2 ? p.stages1 * p.stage1_bytes : p.slots2 * SLOT2;
  const int smem = 1024 + p.a2_bytes + ring_used + BAR_BYTES;
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(kvpred_tc_kernel, SMEM_TOTAL, raised);
  if (e != cudaSuccess) return e;
  const int items = ((g.M + BM - 1) / BM) * (g.kv_end - g.kv_begin);
  const int grid = items < g.n_sm ? items : g.n_sm;
  ++*n_launch;
  return launch_overlapped(kvpred_tc_kernel, dim3(grid), dim3(N_THREADS), (size_t)smem, st, ma, ma2, mw, mfk, mfv, p);
}
