// Tensor-core GEMM for sm_100a:  D[M,N] = A[M,K] W[N,K]^T (+ A_lo W^T on split tiles), bf16
// operands, fp32 accumulation in tensor memory.
//
// One persistent CTA per SM walks output tiles of 128 x BN (BN = 256, or 128 when the problem
// has too few wide tiles to fill the SMs).  Operand tiles travel through a ring of shared-
// memory stages (128-byte swizzle, 64 k-elements per stage) filled by TMA.  A thread that
// issues a tensor copy is held for a few hundred cycles per copy, which caps one issuing thread
// at about 120 GB/s; a 128 x 256 tile needs 48 KiB per 512 tensor-pipe cycles (about 180 GB/s),
// so the A and the W tile of a stage are issued by two different warps (0 and 2).  Warp 1
// issues tcgen05.mma (one elected thread) into one of two BN-column accumulators in tensor
// memory; warps 3-6 drain the other accumulator with tcgen05.ld and run the fused epilogue
// (bf16 store / fp32 residual add / RoPE + hi-lo split / SwiGLU / scatter into cache pages),
// so the epilogue of tile i overlaps the main loop of tile i+1.
// Tiles are visited in groups of 16 row blocks so that a wave's A and W tiles stay in L2.
// The residual GEMMs (x += A W^T) add with red.global, so when they have fewer tiles than
// two per SM their k loops are cut into equal contiguous shares, one per CTA (stream-K).
// Every mbarrier wait is bounded: on expiry the kernel records DEV_TIMEOUT, all roles leave
// their loops, in-flight copies are given time to land, tensor memory is freed.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <math.h>

#include "common.cuh"
#include "gemm_tc.h"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int BM = 128, BK = 64;
constexpr int GROUP_M = 16;                                // row blocks per rasterisation group
constexpr int N_THREADS = 224;                             // warps: 0 A loads, 1 MMA, 2 W loads, 3-6 epilogue
constexpr int N_THREADS_NORM = 352;                        // fused-norm residual kernel: 8 epilogue warps (3-10), two per lane quarter
constexpr int TC_RESID_NORM = 100;                         // internal: TC_RESID with the folded RMSNorm producer (own shared-memory plan)
template <int BN, int EPI = TC_STORE> struct Tile {
  // the fused-norm residual epilogue needs a deeper prefetch ring for the old values of X: one operand stage less
  static constexpr int STAGES = (BN == 256 ? 4 : 6) - (EPI == TC_RESID_NORM ? 1 : 0);
  static constexpr int XS = (EPI == TC_PAGED || EPI == TC_QKV) ? 1 : 2;        // 4 KiB slots per epilogue warp
  // epilogues that move every element through shared memory get eight warps (two per tensor-memory lane quarter)
  static constexpr int EPI_WARPS = (EPI == TC_RESID_NORM || EPI == TC_PAGED || EPI == TC_QKV || EPI == TC_SWIGLU) ? 8 : 4;
  static constexpr int THREADS = EPI_WARPS == 8 ? N_THREADS_NORM : N_THREADS;
  static constexpr int XRING = (EPI == TC_RESID || EPI == TC_RESID_NORM || EPI == TC_PAGED || EPI == TC_QKV) ? EPI_WARPS * XS * 4096 : 0;
  static constexpr int A_BYTES = BM * BK * 2, W_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;    // 48 KiB / 32 KiB
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + XRING + 1024 /*align*/ + 512 /*barriers*/;
};
// Fused-norm residual epilogue: each epilogue warp prefetches the residual stream's old values of its 32 rows,
// 32 columns at a time, into a private ring of XS slots (TMA, 128-byte swizzle) while the main loop of the next
// tile runs, so the read-modify-write of X never waits on memory.
constexpr int X_SLOT_BYTES = 32 * 32 * 4;
__device__ __forceinline__ uint4 pack8(const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 u;
  u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
  u.z = *reinterpret_cast<uint32_t*>(&c); u.w = *reinterpret_cast<uint32_t*>(&d);
  return u;
}
// 8 values as IEEE halves (saturating)
__device__ __forceinline__ uint4 pack8_half(const float* v) {
  uint4 u;
  uint32_t* w = &u.x;
#pragma unroll
  for (int i = 0; i < 4; ++i) w[i] = half2_sat(v[2 * i], v[2 * i + 1]);
  return u;
}
// bf16 rounding remainders of 8 values
__device__ __forceinline__ uint4 pack8_lo(const float* v) {
  float r[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) r[i] = v[i] - __bfloat162float(__float2bfloat16_rn(v[i]));
  return pack8(r);
}
__device__ __forceinline__ void store32_bf16(bf16* dst, const float* v, int n_valid) {
#pragma unroll
  for (int g = 0; g < 4; ++g)
    if (g * 8 < n_valid) *reinterpret_cast<uint4*>(dst + g * 8) = pack8(v + g * 8);
}

struct Params {
  int M, N, K;
  int split_begin;       // tiles with n0 + BN > split_begin run the k loop a second time over A2
  int has_a2;
  int stream_k;          // residual GEMM only: CTAs take equal shares of all k blocks
  int* status;
  // epilogue
  bf16* C; int ldc;
  float* X; int ldx;
  bf16* C_lo; int ld_lo; int lo_col_begin;
  int lo_is_half;        // C_lo receives the whole value as an IEEE half instead of the bf16 remainder
  int h_is_half;         // H is written as IEEE halves
  int c_is_half;         // TC_QKV: C itself is written as IEEE halves (attention with half operands)
  int f16_operands;      // A and W hold IEEE halves (both operands of one MMA have the same type)
  int rot_cols; int hd;
  const float2* rope_tab; int tab_stride; const int* tok_pos;
  int ffn;               // SwiGLU: output width
  const float* q_gain; const float* k_gain; int q_cols; float eps;   // TC_QKV: query / key norm (null = off)
  PagedOut paged;
  int paged_wide;        // TC_PAGED: head_dim and every segment boundary are multiples of 64 (128-byte row pieces)
  // RMSNorm folded into its neighbours.  Producer (TC_RESID with H; every tile owned by one CTA): the epilogue
  // reads the old X (prefetched by TMA), stores X + acc, and also writes the next GEMM's operand
  // H = bf16(X * gain_next) (+ its bf16 remainder H_lo) and adds the row's share of sum X^2 to ss_out[m].  Consumer (TC_QKV / TC_SWIGLU with ss_in): every row of the accumulator is scaled by
  // rsqrt(ss_in[m] / K + rms_eps), which is the norm's 1 / rms applied after the product instead of before it.
  bf16* H; bf16* H_lo; int ldh; const float* gain_next; float* ss_out;
  const float* ss_in; float rms_eps;
};

// ---- work list: every role of a CTA walks the same sequence of (tile, k-block range) ---------
struct Work { int m0, n0, kb0, kb1, tile; };

template <int BN>
struct Sched {
  int tiles_m, tiles_n, n_tiles, num_kb;
  int tile;                 // tile mode: next tile of this CTA
  long long g, g_end;       // stream-K mode: this CTA's share of the global k-block sequence
  const Params& p;
  __device__ __forceinline__ explicit Sched(const Params& p_) : p(p_) {
    tiles_m = (p.M + BM - 1) / BM; tiles_n = (p.N + BN - 1) / BN;
    n_tiles = tiles_m * tiles_n;
    num_kb = (p.K + BK - 1) / BK;
    tile = blockIdx.x;
    long long total = (long long)n_tiles * num_kb;
    g = total * blockIdx.x / gridDim.x;
    g_end = total * (blockIdx.x + 1) / gridDim.x;
  }
  __device__ __forceinline__ void coords(int t, Work& w) const {
    const int per_group = GROUP_M * tiles_n;
    const int grp = t / per_group, r = t - grp * per_group;
    const int gm = min(GROUP_M, tiles_m - grp * GROUP_M);
    w.m0 = (grp * GROUP_M + r % gm) * BM;
    w.n0 = (r / gm) * BN;
    w.tile = t;
  }
  __device__ __forceinline__ bool next(Work& w) {
    if (p.stream_k) {
      if (g >= g_end) return false;
      const int t = (int)(g / num_kb);
      coords(t, w);
      w.kb0 = (int)(g - (long long)t * num_kb);
      w.kb1 = (int)min((long long)num_kb, w.kb0 + (g_end - g));
      g += w.kb1 - w.kb0;
      return true;
    }
    if (tile >= n_tiles) return false;
    coords(tile, w);
    w.kb0 = 0;
    w.kb1 = ((p.has_a2 && w.n0 + BN > p.split_begin) ? 2 : 1) * num_kb;
    tile += gridDim.x;
    return true;
  }
};

// ---- epilogues: one thread owns one output row of the tile ---------------------------------
// `part` of `n_parts`: the warps that share a lane quarter take turns over the blocks of 32 columns (TC_QKV: over the heads)
template <int EPI, int BN>
__device__ __forceinline__ void epilogue_tile(const Params& p, uint32_t tmem_acc, int m, int n0, bool row_ok, int part, int n_parts, uint32_t slot, int row_base) {
  // tmem_acc already carries this warp's lane quarter in its upper half
  if (EPI == TC_STORE) {
#pragma unroll 1
    for (int c = part * 32; c < BN; c += 32 * n_parts) {
      int n = n0 + c;
      int n_valid = p.N - n;
      if (n_valid <= 0) break;           // uniform over the warp
      float v[32];
      tmem_ld32(tmem_acc + c, v);
      tmem_ld_wait();
      if (row_ok) store32_bf16(p.C + (size_t)m * p.ldc + n, v, n_valid);
    }
  } else if (EPI == TC_SWIGLU) {
    // every 128 columns of the tile: [0, 64) gate rows, [64, 128) the matching up rows
    const float rinv = (p.ss_in && row_ok) ? rsqrtf(p.ss_in[m] / (float)p.K + p.rms_eps) : 1.f;
#pragma unroll 1
    for (int c = part * 32; c < BN / 2; c += 32 * n_parts) {
      int grp = c >> 6, cc = c & 63;
      int n = ((n0 + grp * 128) >> 1) + cc;
      int n_valid = p.ffn - n;
      if (n_valid <= 0) break;
      float g[32], u[32];
      tmem_ld32(tmem_acc + grp * 128 + cc, g);
      tmem_ld32(tmem_acc + grp * 128 + 64 + cc, u);
      tmem_ld_wait();
      if (!row_ok) continue;
#pragma unroll
      for (int i = 0; i < 32; ++i) { const float gi = g[i] * rinv; g[i] = __fdividef(gi, 1.f + __expf(-gi)) * (u[i] * rinv); }
      store32_bf16(p.C + (size_t)m * p.ldc + n, g, n_valid);
      if (p.C_lo) {        // bf16 remainder of the activation, for a down projection that takes both parts
        bf16* lo = p.C_lo + (size_t)m * p.ld_lo + n;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (q * 8 < n_valid) *reinterpret_cast<uint4*>(lo + q * 8) = pack8_lo(g + q * 8);
      }
    }
  } else {  // TC_QKV: RoPE on columns < rot_cols, hi part to C, lo part of columns >= lo_col_begin to C_lo
    int half = p.hd >> 1;
    const int lane = threadIdx.x & 31;
    // (cos, sin) of two neighbouring frequencies per 16-byte entry, entries of consecutive POSITIONS next to each other: the 32
    // rows of a warp (consecutive tokens) read 512 contiguous bytes per load
    const float4* tab = row_ok ? reinterpret_cast<const float4*>(p.rope_tab) + p.tok_pos[m] : nullptr;
    const float rinv = (p.ss_in && row_ok) ? rsqrtf(p.ss_in[m] / (float)p.K + p.rms_eps) : 1.f;
#pragma unroll 1
    for (int h0 = part * p.hd; h0 < BN; h0 += p.hd * n_parts) {
      if (n0 + h0 >= p.N) break;
      // query / key norm: this thread's row of the head is scaled by 1 / rms and the head's gain before RoPE
      const float* gain = (n0 + h0 < p.rot_cols) ? (n0 + h0 < p.q_cols ? p.q_gain : p.k_gain) : nullptr;
      float rn = 1.f;
      if (gain) {          // (uniform over the warp) first pass over the head's columns: mean square
        float ss = 0.f;
#pragma unroll 1
        for (int j = 0; j < p.hd; j += 32) {
          float a[32];
          tmem_ld32(tmem_acc + h0 + j, a);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ss = fmaf(a[i], a[i], ss);
        }
        rn = rsqrtf(ss * rinv * rinv / (float)p.hd + p.eps);
      }
#pragma unroll 1
      for (int j = 0; j < half; j += 32) {
        float a[32], b[32];
        tmem_ld32(tmem_acc + h0 + j, a);
        tmem_ld32(tmem_acc + h0 + half + j, b);
        tmem_ld_wait();
        int n = n0 + h0 + j;
        if (row_ok) {
          if (p.ss_in) {
#pragma unroll
            for (int i = 0; i < 32; ++i) { a[i] *= rinv; b[i] *= rinv; }
          }
          if (gain) {
#pragma unroll
            for (int i = 0; i < 32; ++i) { a[i] *= rn * gain[j + i]; b[i] *= rn * gain[half + j + i]; }
          }
          if (n < p.rot_cols) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float4 cs = tab[(size_t)((j + i) >> 1) * p.tab_stride];   // (cos, sin) of two frequencies
              float x1 = a[i], x2 = b[i];
              a[i] = x1 * cs.x - x2 * cs.y; b[i] = x2 * cs.x + x1 * cs.y;
              x1 = a[i + 1]; x2 = b[i + 1];
              a[i + 1] = x1 * cs.z - x2 * cs.w; b[i + 1] = x2 * cs.z + x1 * cs.w;
            }
          }
        }
        // A thread owns a ROW here, and 16-byte stores of 32 different rows cost four times the memory transactions of
        // 64-byte row pieces: the two 32 x 32 blocks (first and second half of the head) go through this warp's
        // shared-memory slot as 16-bit values (16-byte pieces swizzled by the row) and leave as 8 rows x 64 bytes per store.
        auto stage_and_store = [&](bool as_half, bool remainder, bf16* base, int ld, int col) {
          __syncwarp();                        // the slot's previous contents have been read
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const uint32_t off = lane * 64 + ((g ^ ((lane >> 1) & 3)) << 4);
            const uint4 ua = as_half ? pack8_half(a + g * 8) : (remainder ? pack8_lo(a + g * 8) : pack8(a + g * 8));
            const uint4 ub = as_half ? pack8_half(b + g * 8) : (remainder ? pack8_lo(b + g * 8) : pack8(b + g * 8));
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slot + off), "r"(ua.x), "r"(ua.y), "r"(ua.z), "r"(ua.w) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slot + 2048 + off), "r"(ub.x), "r"(ub.y), "r"(ub.z), "r"(ub.w) : "memory");
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int r = 8 * i + (lane >> 2), cq = lane & 3;
            if (row_base + r < p.M) {
              const uint32_t off = r * 64 + ((cq ^ ((r >> 1) & 3)) << 4);
              uint4 ua, ub;
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(ua.x), "=r"(ua.y), "=r"(ua.z), "=r"(ua.w) : "r"(slot + off));
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(ub.x), "=r"(ub.y), "=r"(ub.z), "=r"(ub.w) : "r"(slot + 2048 + off));
              bf16* dst = base + (size_t)(row_base + r) * ld + col + 8 * cq;
              *reinterpret_cast<uint4*>(dst) = ua;
              *reinterpret_cast<uint4*>(dst + half) = ub;
            }
          }
        };
        stage_and_store(p.c_is_half != 0, false, p.C, p.ldc, n);
        if (p.C_lo && n >= p.lo_col_begin) stage_and_store(p.lo_is_half != 0, p.lo_is_half == 0, p.C_lo, p.ld_lo, n - p.lo_col_begin);
      }
    }
  }
}

template <int EPI, int BN>
__global__ void __launch_bounds__((Tile<BN, EPI>::THREADS), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a2,
               const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const Params p) {
  using T = Tile<BN, EPI>;
  constexpr int STAGES = T::STAGES, STAGE_BYTES = T::STAGE_BYTES, XS = T::XS;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int XR = T::XRING;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES + XR);
  // bars: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], x_full[epilogue warps][XS]; then tmem base, abort flag
  constexpr int EW = T::EPI_WARPS;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4 + EW * XS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  auto xfull_bar = [&](int q, int s) { return bar_base + 8u * (2 * STAGES + 4 + q * XS + s); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();      // the next kernel's CTAs may take SMs as this kernel's CTAs leave them
  if (threadIdx.x == 32) {   // tensor maps on their way while the barriers and tensor memory are set up
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_w);
    if (p.has_a2) prefetch_tensormap(&map_a2);
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // two loaders per stage
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), EW); }
    for (int q = 0; q < EW; ++q) for (int x = 0; x < XS; ++x) mbar_init(xfull_bar(q, x), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor memory: two accumulators of BN columns
    tmem_alloc(smem_u32(tmem_slot), 2 * BN);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int num_kb = (p.K + BK - 1) / BK;
  pdl_wait();         // set-up above overlapped the previous kernel's tail; its results are needed from here on

  if (warp == 0 || warp == 2) {
    // ---------------- TMA producers: warp 0 loads the A tile of every stage, warp 2 the W tile ----------------
    if (lane == 0) {
      const bool is_a = warp == 0;
      Sched<BN> sched(p);
      Work w;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      while (ok && sched.next(w)) {
        for (int it = w.kb0; it < w.kb1 && ok; ++it) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status);
          if (!ok) break;
          const int kb = it < num_kb ? it : it - num_kb;
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          if (is_a) {
            mbar_expect_tx(full_bar(stage), T::A_BYTES);
            tma_load_2d(sa, it < num_kb ? &map_a : &map_a2, kb * BK, w.m0, full_bar(stage));
          } else {
            mbar_expect_tx(full_bar(stage), T::W_BYTES);
            tma_load_2d(sa + T::A_BYTES, &map_w, kb * BK, w.n0, full_bar(stage));
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) drain_after_abort();
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // operand formats: bits 7-9 (A) and 10-12 (B): 1 = bf16, 0 = IEEE half
      const uint32_t fmt = p.f16_operands ? 0u : ((1u << 7) | (1u << 10));
      const uint32_t idesc = (1u << 4) | fmt | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      Sched<BN> sched(p);
      Work w;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      while (ok && sched.next(w)) {
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int it = w.kb0; it < w.kb1 && ok; ++it) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES, sb = sa + T::A_BYTES;
          const uint64_t da = desc_kmajor(sa), db = desc_kmajor(sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            tc_mma_bf16(d_tmem, da + 2u * k, db + 2u * k, idesc, (it > w.kb0 || k > 0) ? 1u : 0u);
          tc_commit(empty_bar(stage));        // the slot is free once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));    // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) drain_after_abort();
    }
  } else {
    // ---------------- epilogue: 4 warps, each owns the 32 tensor-memory lanes of its quarter ----------------
    const int quarter = warp & 3;                 // tensor-memory lanes this warp may read
    const int ew = warp - 3;                      // epilogue warp index
    constexpr int NH = EW / 4;                    // warps per lane quarter: each takes every NH-th block of 32 columns
    const int half = ew >> 2;
    Sched<BN> sched(p);
    Work w;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    // fused norm (TC_RESID with H, every tile owned by one CTA): the old values of X arrive through this warp's ring
    constexpr bool fused = EPI == TC_RESID_NORM;
    const uint32_t xring = smem_base + STAGES * STAGE_BYTES + ew * (XS * X_SLOT_BYTES);
    Sched<BN> pre(p);
    Work pw;
    bool pre_ok = fused && pre.next(pw);
    int pre_c = half;
    while (pre_ok && pw.n0 + pre_c * 32 >= p.N) { pre_ok = pre.next(pw); pre_c = half; }     // (a tile without a block for this warp)
    uint32_t x_issued = 0, x_used = 0;
    auto prefetch_x = [&]() {      // this warp's next 32 x 32 block of X in (tile, column) order into the slot just freed
      if (!pre_ok) return;
      const int slot = x_issued % XS;
      if (lane == 0) {
        mbar_expect_tx(xfull_bar(ew, slot), X_SLOT_BYTES);
        tma_load_2d(xring + slot * X_SLOT_BYTES, &map_x, pw.n0 + pre_c * 32, pw.m0 + quarter * 32, xfull_bar(ew, slot));
      }
      ++x_issued;
      pre_c += NH;
      while (pre_ok && (pw.n0 + pre_c * 32 >= p.N || pre_c * 32 >= BN)) { pre_ok = pre.next(pw); pre_c = half; }
    };
    if (fused) for (int i = 0; i < XS; ++i) prefetch_x();
    while (sched.next(w)) {
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int m = w.m0 + quarter * 32 + lane;
      const uint32_t tmem_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
      if (fused) {
        float row_ss = 0.f;
#pragma unroll 1
        for (int c = half * 32; c < BN && ok; c += 32 * NH) {
          const int n = w.n0 + c, n_valid = p.N - n;
          if (n_valid <= 0) break;
          const int slot = x_used % XS;
          ok = mbar_wait(xfull_bar(ew, slot), (x_used / XS) & 1u, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          float v[32];
          tmem_ld32(tmem_acc + c, v);
          const uint32_t xrow = xring + slot * X_SLOT_BYTES + lane * 128;
#pragma unroll
          for (int g = 0; g < 8; ++g) {          // this thread's row of the slot: 16-byte pieces swizzled by the row
            float4 o;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(o.x), "=f"(o.y), "=f"(o.z), "=f"(o.w)
                         : "r"(xrow + ((g ^ (lane & 7)) << 4)));
            if (g == 0) tmem_ld_wait();
            v[4 * g] += o.x; v[4 * g + 1] += o.y; v[4 * g + 2] += o.z; v[4 * g + 3] += o.w;
          }
          // The new values leave through the slot: every thread owns a ROW here, and 16-byte stores of 32 different rows
          // cost eight times the memory transactions of whole 128-byte lines.  Each thread puts its row back into the slot,
          // then the warp reads the slot line by line and stores it coalesced; the operand rows (bf16 value, remainder) follow
          // through the same 4 KiB.
          const uint32_t sl = xring + slot * X_SLOT_BYTES;
          const int row_base = w.m0 + quarter * 32;
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 8; ++g)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(xrow + ((g ^ (lane & 7)) << 4)), "f"(v[4 * g]), "f"(v[4 * g + 1]),
                         "f"(v[4 * g + 2]), "f"(v[4 * g + 3]) : "memory");
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i) {            // 4 rows x 128 bytes per instruction
            const int r = 4 * i + (lane >> 3), j = lane & 7;
            float4 o;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(o.x), "=f"(o.y), "=f"(o.z), "=f"(o.w)
                         : "r"(sl + r * 128 + ((j ^ (r & 7)) << 4)));
            if (row_base + r < p.M && n + 4 * j < p.N) *reinterpret_cast<float4*>(p.X + (size_t)(row_base + r) * p.ldx + n + 4 * j) = o;
          }
          // operand of the next GEMM and the row's sum of squares
          float ssq = 0.f;
          if (n_valid >= 32) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const float4 gn = __ldg(reinterpret_cast<const float4*>(p.gain_next + n) + g);
              ssq = fmaf(v[4 * g], v[4 * g], ssq); ssq = fmaf(v[4 * g + 1], v[4 * g + 1], ssq);
              ssq = fmaf(v[4 * g + 2], v[4 * g + 2], ssq); ssq = fmaf(v[4 * g + 3], v[4 * g + 3], ssq);
              v[4 * g] *= gn.x; v[4 * g + 1] *= gn.y; v[4 * g + 2] *= gn.z; v[4 * g + 3] *= gn.w;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const bool in = i < n_valid;
              ssq = fmaf(in ? v[i] : 0.f, v[i], ssq);
              v[i] = in ? v[i] * p.gain_next[n + i] : 0.f;
            }
          }
          row_ss += ssq;
          __syncwarp();                            // the slot has been read back by every lane
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const uint4 hi = p.h_is_half ? pack8_half(v + g * 8) : pack8(v + g * 8);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sl + lane * 64 + g * 16), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
            if (p.H_lo) {
              const uint4 lo = pack8_lo(v + g * 8);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sl + 2048 + lane * 64 + g * 16), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
            }
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 4; ++i) {            // 8 rows x 64 bytes per instruction
            const int r = 8 * i + (lane >> 2), c = lane & 3;
            if (row_base + r < p.M && n + 8 * c < p.N) {
              uint4 u;
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(sl + r * 64 + c * 16));
              *reinterpret_cast<uint4*>(p.H + (size_t)(row_base + r) * p.ldh + n + 8 * c) = u;
              if (p.H_lo) {
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(sl + 2048 + r * 64 + c * 16));
                *reinterpret_cast<uint4*>(p.H_lo + (size_t)(row_base + r) * p.ldh + n + 8 * c) = u;
              }
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // this warp's own writes to the slot come before the copy engine's
          __syncwarp();                            // the slot is free: the next block of X may land in it
          ++x_used;
          prefetch_x();
        }
        if (!ok) break;
        if (m < p.M) atomicAdd(p.ss_out + m, row_ss);
      } else if (EPI == TC_RESID || EPI == TC_RESID_NORM) {
        // X += acc through the copy engine: a 32 x 32 block of the accumulator goes into one of this warp's slots
        // (swizzled like a tensor tile) and leaves as ONE reduce-add of whole 128-byte rows, instead of 256 separate
        // 16-byte atomics.  Rows and columns beyond the matrix are clipped by the tensor map.
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          const int n = w.n0 + c;
          if (n >= p.N) break;
          const int slot = x_used % XS;
          if (x_used >= XS) {          // the reduce issued from this slot two blocks ago has read it
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(XS - 1) : "memory");
            __syncwarp();
          }
          float v[32];
          tmem_ld32(tmem_acc + c, v);
          tmem_ld_wait();
          const uint32_t xrow = xring + slot * X_SLOT_BYTES + lane * 128;
#pragma unroll
          for (int g = 0; g < 8; ++g)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(xrow + ((g ^ (lane & 7)) << 4)), "f"(v[4 * g]), "f"(v[4 * g + 1]),
                         "f"(v[4 * g + 2]), "f"(v[4 * g + 3]) : "memory");
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(&map_x), "r"(n), "r"(w.m0 + quarter * 32), "r"(xring + slot * X_SLOT_BYTES) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          ++x_used;
        }
      } else if (EPI == TC_PAGED) {
        // Predicted columns into cache pages.  A thread owns a token ROW of the accumulator, but 16-byte stores of 32
        // different rows cost four times the memory transactions of 64-byte row pieces: the 32 x 32 block goes through
        // this warp's shared-memory slot as halves and leaves as 8 rows x 64 bytes per store instruction.
        const PagedOut& q = p.paged;
        const uint32_t sl = xring;
        const int row_base = w.m0 + quarter * 32;
        if (p.paged_wide) {
          // head_dim and every segment boundary are multiples of 64: 64 columns at a time (half a head_dim-128 row or a
          // whole head_dim-64 row of a token), staged as 32 rows x 128 bytes (16-byte pieces swizzled by the row) and
          // stored as 4 rows x 128 bytes per instruction.
          int slot8[8];            // cache slots of the eight rows this lane writes in the read-back pattern
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int mr = row_base + 4 * i + (lane >> 3);
            slot8[i] = mr < p.M ? q.tok_slot[mr] : -1;
          }
#pragma unroll 1
          for (int c = half * 64; c < BN; c += 64 * NH) {
            const int n = w.n0 + c;
            if (n >= p.N) break;
            float v[64];
            tmem_ld32(tmem_acc + c, v);
            tmem_ld32(tmem_acc + c + 32, v + 32);
            tmem_ld_wait();
            if (q.bias) {
#pragma unroll
              for (int i = 0; i < 64; ++i) v[i] += q.bias[n + i];
            }
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const uint4 u = pack8_half(v + g * 8);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sl + lane * 128 + ((g ^ (lane & 7)) << 4)), "r"(u.x), "r"(u.y), "r"(u.z), "r"(u.w) : "memory");
            }
            __syncwarp();
            int sg = 0;
            while (sg + 1 < q.n_seg && n >= q.col0[sg + 1]) ++sg;
            const int in_seg = n - q.col0[sg];
            const int head = in_seg / q.head_dim, dim = in_seg - head * q.head_dim;
            kv16* pool = (kv16*)q.pool[sg];
            const int nkv_s = q.n_kv[sg];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = 4 * i + (lane >> 3), cq = lane & 7;
              if (slot8[i] >= 0) {
                uint4 u;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(sl + r * 128 + ((cq ^ (r & 7)) << 4)));
                const int page = slot8[i] / PAGE_TOKENS, prow = slot8[i] - page * PAGE_TOKENS;
                *reinterpret_cast<uint4*>(pool + (((size_t)page * nkv_s + head) * PAGE_TOKENS + prow) * q.head_dim + dim + 8 * cq) = u;
              }
            }
            __syncwarp();
          }
        } else {
          int slot4[4];              // cache slots of the four rows this lane writes in the read-back pattern
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int mr = row_base + 8 * i + (lane >> 2);
            slot4[i] = mr < p.M ? q.tok_slot[mr] : -1;
          }
#pragma unroll 1
          for (int c = half * 32; c < BN; c += 32 * NH) {
            const int n = w.n0 + c;
            if (n >= p.N) break;
            float v[32];
            tmem_ld32(tmem_acc + c, v);
            tmem_ld_wait();
            if (q.bias) {
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] += q.bias[n + i];
            }
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const uint4 u = pack8_half(v + g * 8);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sl + lane * 64 + g * 16), "r"(u.x), "r"(u.y), "r"(u.z), "r"(u.w) : "memory");
            }
            __syncwarp();
            int sg = 0;
            while (sg + 1 < q.n_seg && n >= q.col0[sg + 1]) ++sg;
            const int in_seg = n - q.col0[sg];
            const int head = in_seg / q.head_dim, dim = in_seg - head * q.head_dim;
            kv16* pool = (kv16*)q.pool[sg];
            const int nkv_s = q.n_kv[sg];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int r = 8 * i + (lane >> 2), cq = lane & 3;
              if (slot4[i] >= 0) {
                uint4 u;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(sl + r * 64 + cq * 16));
                const int page = slot4[i] / PAGE_TOKENS, prow = slot4[i] - page * PAGE_TOKENS;
                *reinterpret_cast<uint4*>(pool + (((size_t)page * nkv_s + head) * PAGE_TOKENS + prow) * q.head_dim + dim + 8 * cq) = u;
              }
            }
            __syncwarp();
          }
        }
      } else {
        epilogue_tile<EPI, BN>(p, tmem_acc, m, w.n0, m < p.M, half, NH, xring, w.m0 + quarter * 32);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if ((EPI == TC_RESID || EPI == TC_RESID_NORM) && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");    // this warp's reduces have completed
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ---- host side ----------------------------------------------------------------------------
// bf16 [rows, cols] row-major with row stride ld elements; box = 64 columns x box_rows rows, 128B swizzle
bool make_map(CUtensorMap* m, const void* base, int rows, int cols, int ld, int box_rows) {
  return tc_make_map_bf16(m, base, rows, cols, ld, box_rows);
}

template <int EPI, int BN>
cudaError_t go(const CUtensorMap& a, const CUtensorMap& a2, const CUtensorMap& w, const CUtensorMap& x, const Params& p, int grid, cudaStream_t st) {
  constexpr int SMEM = Tile<BN, EPI>::SMEM_BYTES;
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(gemm_tc_kernel<EPI, BN>, SMEM, raised);
  if (e != cudaSuccess) return e;
  return launch_overlapped(gemm_tc_kernel<EPI, BN>, dim3(grid), dim3(Tile<BN, EPI>::THREADS), SMEM, st, a, a2, w, x, p);
}

template <int BN>
cudaError_t go_epi(int epi, const CUtensorMap& a, const CUtensorMap& a2, const CUtensorMap& w, const CUtensorMap& x, const Params& p, int grid, cudaStream_t st) {
  switch (epi) {
    case TC_STORE: return go<TC_STORE, BN>(a, a2, w, x, p, grid, st);
    case TC_RESID: return p.H ? go<TC_RESID_NORM, BN>(a, a2, w, x, p, grid, st) : go<TC_RESID, BN>(a, a2, w, x, p, grid, st);
    case TC_SWIGLU: return go<TC_SWIGLU, BN>(a, a2, w, x, p, grid, st);
    case TC_QKV: return go<TC_QKV, BN>(a, a2, w, x, p, grid, st);
    default: return go<TC_PAGED, BN>(a, a2, w, x, p, grid, st);
  }
}

// Relative time of a launch with tile width bn on n_sm SMs: waves of tiles, each tile costing
// the larger of its tensor-pipe time and its operand-feed time (two issuing threads deliver
// about 100 bytes per cycle).
double tile_cost(const TcGemm& g, int bn, bool stream_k) {
  const double tiles = (double)((g.M + BM - 1) / BM) * ((g.N + bn - 1) / bn);
  const double mma = 2.0 * bn, feed = (BM + bn) * 128.0 / 100.0;      // cycles per k block
  const double per_tile = mma > feed ? mma : feed;
  const double waves = stream_k ? tiles / g.n_sm : (double)(((long long)tiles + g.n_sm - 1) / g.n_sm);
  return waves * per_tile;
}

}  // namespace

bool tc_gemm_resid_can_fuse(int M, int N, int n_sm) {
  // with fewer than two 128 x 128 tiles per SM the k loops are shared among CTAs and no CTA sees a final value
  return ((M + BM - 1) / BM) * ((N + 127) / 128) >= 2 * n_sm;
}

bool tc_gemm_supported(const TcGemm& g) {
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
  if (g.K % 8 || g.lda % 8 || g.ldw % 8 || !al16(g.A) || !al16(g.W)) return false;
  if (g.A2 && (g.lda2 % 8 || !al16(g.A2))) return false;
  switch (g.epi) {
    case TC_STORE: return g.N % 8 == 0 && g.ldc % 8 == 0 && al16(g.C);
    case TC_RESID:
      if (g.H && (g.N % 8 || g.ldh % 8 || !al16(g.H) || (g.H_lo && !al16(g.H_lo)) || !g.gain_next || !g.ss_out || g.A2 ||
                  !tc_gemm_resid_can_fuse(g.M, g.N, g.n_sm))) return false;
      return g.N % 4 == 0 && g.ldx % 4 == 0 && al16(g.X);
    case TC_SWIGLU:
      return g.ffn % 64 == 0 && g.N == 2 * g.ffn && g.ldc % 8 == 0 && al16(g.C) && (!g.C_lo || (g.ld_lo % 8 == 0 && al16(g.C_lo)));
    case TC_QKV:
      return (g.hd == 64 || g.hd == 128) && g.N % g.hd == 0 && g.rot_cols % g.hd == 0 && g.lo_col_begin % g.hd == 0 &&
             g.ldc % 8 == 0 && al16(g.C) && (!g.C_lo || (g.ld_lo % 8 == 0 && al16(g.C_lo))) && g.rope_tab && g.tok_pos;
    case TC_PAGED: {
      const PagedOut& q = g.paged;
      if (q.head_dim % 32 || q.n_seg < 1) return false;
      for (int s = 0; s <= q.n_seg; ++s) if (q.col0[s] % 32) return false;
      return g.N == q.col0[q.n_seg];
    }
  }
  return false;
}

cudaError_t launch_gemm_tc(const TcGemm& g, int* status, cudaStream_t st, int64_t* n_launch) {
  if (!tc_encode_fn()) return cudaErrorNotSupported;
  const int tiles128 = ((g.M + BM - 1) / BM) * ((g.N + 127) / 128);
  const bool stream_k = g.epi == TC_RESID && !g.A2 && tiles128 < 2 * g.n_sm;
  int bn = g.bn;
  if (bn != 128 && bn != 256) bn = tile_cost(g, 256, stream_k) <= tile_cost(g, 128, stream_k) ? 256 : 128;
  CUtensorMap ma, ma2, mw, mx;
  if (g.H && (stream_k || g.epi != TC_RESID)) return cudaErrorInvalidValue;     // see tc_gemm_resid_can_fuse()
  if (!make_map(&ma, g.A, g.M, g.K, g.lda, BM)) return cudaErrorInvalidValue;
  if (!make_map(&mw, g.W, g.N, g.K, g.ldw, bn)) return cudaErrorInvalidValue;
  if (g.A2) { if (!make_map(&ma2, g.A2, g.M, g.K, g.lda2, BM)) return cudaErrorInvalidValue; }
  else ma2 = ma;
  if (g.epi == TC_RESID) { if (!tc_make_map_f32(&mx, g.X, g.M, g.N, g.ldx, 32)) return cudaErrorInvalidValue; }
  else mx = ma;
  Params p{};
  p.M = g.M; p.N = g.N; p.K = g.K; p.split_begin = g.split_begin; p.has_a2 = g.A2 != nullptr; p.status = status;
  p.stream_k = stream_k ? 1 : 0;
  p.C = g.C; p.ldc = g.ldc; p.X = g.X; p.ldx = g.ldx; p.C_lo = g.C_lo; p.ld_lo = g.ld_lo; p.lo_col_begin = g.lo_col_begin;
  p.q_gain = g.q_gain; p.k_gain = g.k_gain; p.q_cols = g.q_cols; p.eps = g.eps;
  p.rot_cols = g.rot_cols; p.hd = g.hd; p.rope_tab = g.rope_tab; p.tab_stride = g.tab_stride; p.tok_pos = g.tok_pos; p.ffn = g.ffn; p.paged = g.paged;
  p.H = g.H; p.H_lo = g.H_lo; p.ldh = g.ldh; p.gain_next = g.gain_next; p.ss_out = g.ss_out;
  p.ss_in = g.ss_in; p.rms_eps = g.rms_eps;
  p.paged_wide = 0;
  if (g.epi == TC_PAGED) {
    p.paged_wide = g.paged.head_dim % 64 == 0 && g.N % 64 == 0;
    for (int sg = 0; sg <= g.paged.n_seg; ++sg) if (g.paged.col0[sg] % 64) p.paged_wide = 0;
  }
  p.lo_is_half = g.lo_is_half; p.f16_operands = g.f16_operands; p.c_is_half = g.c_is_half; p.h_is_half = g.h_is_half;
  const int tiles = ((g.M + BM - 1) / BM) * ((g.N + bn - 1) / bn);
  const long long kblocks = (long long)tiles * ((g.K + BK - 1) / BK);
  int grid = stream_k ? (int)(kblocks < g.n_sm ? kblocks : g.n_sm) : (tiles < g.n_sm ? tiles : g.n_sm);
  ++*n_launch;
  return bn == 256 ? go_epi<256>(g.epi, ma, ma2, mw, mx, p, grid, st) : go_epi<128>(g.epi, ma, ma2, mw, mx, p, grid, st);
}

// ---- RoPE table: entry [c / 2][pos] = (cos, sin)(pos * theta^(-2c/hd)) for c and c + 1 (16 bytes), positions contiguous ----
__global__ void rope_table_kernel(float2* tab, int n_pos, int half, const __grid_constant__ InvFreq inv) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pos * half) return;
  int c = i / n_pos, pos = i - c * n_pos;
  float s, co;
  rope_sincos(pos, inv.f[c], &s, &co);
  tab[((size_t)(c >> 1) * n_pos + pos) * 2 + (c & 1)] = make_float2(co, s);
}

void launch_rope_table(const LaunchCtx& ctx, float2* tab, int n_pos, int hd, float theta) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  int n = n_pos * (hd / 2);
  ++*ctx.n_launch;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, ctx.st>>>(tab, n_pos, hd / 2, inv);
}
