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

namespace {

constexpr int BM = 128, BK = 64;
constexpr int GROUP_M = 16;                                // row blocks per rasterisation group
constexpr int N_THREADS = 224;                             // warps: 0 A loads, 1 MMA, 2 W loads, 3-6 epilogue
template <int BN> struct Tile {
  static constexpr int STAGES = BN == 256 ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2, W_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;    // 48 KiB / 32 KiB
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};
constexpr uint32_t SPIN_LIMIT = 20u * 1000u * 1000u;      // ~1-2 s of polling

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the kernel is aborting (this or another role gave up).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
    if (mbar_test(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      __nanosleep(64);
    }
  }
  *abort_flag = 1;
  dev_flag(status, DEV_TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 lanes x 32 columns of fp32: thread i of the warp gets row i, register j = column j.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored with the 128-byte swizzle:
// rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  uint64_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);             // start address, leading offset (unused)
  uint64_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);                 // stride offset, version 1, 128B swizzle
  return lo | (hi << 32);
}

__device__ __forceinline__ uint4 pack8(const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 u;
  u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
  u.z = *reinterpret_cast<uint32_t*>(&c); u.w = *reinterpret_cast<uint32_t*>(&d);
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
  int rot_cols; int hd;
  const float2* rope_tab; const int* tok_pos;
  int ffn;               // SwiGLU: output width
  const float* q_gain; const float* k_gain; int q_cols; float eps;   // TC_QKV: query / key norm (null = off)
  PagedOut paged;
};

// ---- work list: every role of a CTA walks the same sequence of (tile, k-block range) ---------
struct Work { int m0, n0, kb0, kb1; };

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

__device__ __forceinline__ void red_add4(float* dst, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// ---- epilogues: one thread owns one output row of the tile ---------------------------------
template <int EPI, int BN>
__device__ __forceinline__ void epilogue_tile(const Params& p, uint32_t tmem_acc, int m, int n0, bool row_ok) {
  // tmem_acc already carries this warp's lane quarter in its upper half
  if (EPI == TC_STORE || EPI == TC_RESID || EPI == TC_PAGED) {
    int slot = -1;
    if (EPI == TC_PAGED && row_ok) slot = p.paged.tok_slot[m];
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      int n = n0 + c;
      int n_valid = p.N - n;
      if (n_valid <= 0) break;           // uniform over the warp
      float v[32];
      tmem_ld32(tmem_acc + c, v);
      tmem_ld_wait();
      if (!row_ok) continue;
      if (EPI == TC_STORE) {
        store32_bf16(p.C + (size_t)m * p.ldc + n, v, n_valid);
      } else if (EPI == TC_RESID) {
        float* x = p.X + (size_t)m * p.ldx + n;
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (g * 4 < n_valid) red_add4(x + 4 * g, v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
      } else {
        if (slot < 0) continue;
        const PagedOut& q = p.paged;
        int s = 0;
        while (s + 1 < q.n_seg && n >= q.col0[s + 1]) ++s;
        int cc = n - q.col0[s];
        int head = cc / q.head_dim, dim = cc - head * q.head_dim;
        if (q.bias) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] += q.bias[n + i];
        }
        int page = slot / PAGE_TOKENS, row = slot - page * PAGE_TOKENS;
        bf16* dst = (bf16*)q.pool[s] + (((size_t)page * q.n_kv[s] + head) * PAGE_TOKENS + row) * q.head_dim + dim;
        store32_bf16(dst, v, n_valid);
      }
    }
  } else if (EPI == TC_SWIGLU) {
    // every 128 columns of the tile: [0, 64) gate rows, [64, 128) the matching up rows
#pragma unroll 1
    for (int c = 0; c < BN / 2; c += 32) {
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
      for (int i = 0; i < 32; ++i) g[i] = __fdividef(g[i], 1.f + __expf(-g[i])) * u[i];
      store32_bf16(p.C + (size_t)m * p.ldc + n, g, n_valid);
    }
  } else {  // TC_QKV: RoPE on columns < rot_cols, hi part to C, lo part of columns >= lo_col_begin to C_lo
    int half = p.hd >> 1;
    const float2* tab = row_ok ? p.rope_tab + (size_t)p.tok_pos[m] * half : nullptr;
#pragma unroll 1
    for (int h0 = 0; h0 < BN; h0 += p.hd) {
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
        rn = rsqrtf(ss / (float)p.hd + p.eps);
      }
#pragma unroll 1
      for (int j = 0; j < half; j += 32) {
        float a[32], b[32];
        tmem_ld32(tmem_acc + h0 + j, a);
        tmem_ld32(tmem_acc + h0 + half + j, b);
        tmem_ld_wait();
        int n = n0 + h0 + j;
        if (!row_ok) continue;
        if (gain) {
#pragma unroll
          for (int i = 0; i < 32; ++i) { a[i] *= rn * gain[j + i]; b[i] *= rn * gain[half + j + i]; }
        }
        if (n < p.rot_cols) {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float4 cs = *reinterpret_cast<const float4*>(tab + j + i);   // (cos, sin) of two frequencies
            float x1 = a[i], x2 = b[i];
            a[i] = x1 * cs.x - x2 * cs.y; b[i] = x2 * cs.x + x1 * cs.y;
            x1 = a[i + 1]; x2 = b[i + 1];
            a[i + 1] = x1 * cs.z - x2 * cs.w; b[i + 1] = x2 * cs.z + x1 * cs.w;
          }
        }
        bf16* dst = p.C + (size_t)m * p.ldc + n;
        store32_bf16(dst, a, 32);
        store32_bf16(dst + half, b, 32);
        if (p.C_lo && n >= p.lo_col_begin) {
          bf16* lo = p.C_lo + (size_t)m * p.ld_lo + (n - p.lo_col_begin);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            *reinterpret_cast<uint4*>(lo + g * 8) = pack8_lo(a + g * 8);
            *reinterpret_cast<uint4*>(lo + half + g * 8) = pack8_lo(b + g * 8);
          }
        }
      }
    }
  }
}

template <int EPI, int BN>
__global__ void __launch_bounds__(N_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a2,
               const __grid_constant__ CUtensorMap map_w, const Params p) {
  using T = Tile<BN>;
  constexpr int STAGES = T::STAGES, STAGE_BYTES = T::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  // bars: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]; then tmem base, abort flag
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();      // the next kernel's CTAs may take SMs as this kernel's CTAs leave them
  if (threadIdx.x == 32) {   // tensor maps on their way while the barriers and tensor memory are set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    if (p.has_a2) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a2) : "memory");
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // two loaders per stage
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor memory: two accumulators of BN columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
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
      if (!ok) {   // aborting: give copies already issued time to land before the CTA's memory goes away
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
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
          const uint64_t da = make_desc(sa), db = make_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            tc_mma_bf16(d_tmem, da + 2u * k, db + 2u * k, idesc, (it > w.kb0 || k > 0) ? 1u : 0u);
          tc_commit(empty_bar(stage));        // the slot is free once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));    // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else {
    // ---------------- epilogue: 4 warps, each owns the 32 tensor-memory lanes of its quarter ----------------
    const int quarter = warp & 3;
    Sched<BN> sched(p);
    Work w;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    while (sched.next(w)) {
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int m = w.m0 + quarter * 32 + lane;
      const uint32_t tmem_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
      epilogue_tile<EPI, BN>(p, tmem_acc, m, w.n0, m < p.M);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
  }
}

// ---- host side ----------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

bool get_encode() {
  if (g_encode) return true;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return false;
  g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  return true;
}

// bf16 [rows, cols] row-major with row stride ld elements; box = 64 columns x box_rows rows, 128B swizzle
bool make_map(CUtensorMap* m, const void* base, int rows, int cols, int ld, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int EPI, int BN>
cudaError_t go(const CUtensorMap& a, const CUtensorMap& a2, const CUtensorMap& w, const Params& p, int grid, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<EPI, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<BN>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return launch_overlapped(gemm_tc_kernel<EPI, BN>, dim3(grid), dim3(N_THREADS), Tile<BN>::SMEM_BYTES, st, a, a2, w, p);
}

template <int BN>
cudaError_t go_epi(int epi, const CUtensorMap& a, const CUtensorMap& a2, const CUtensorMap& w, const Params& p, int grid, cudaStream_t st) {
  switch (epi) {
    case TC_STORE: return go<TC_STORE, BN>(a, a2, w, p, grid, st);
    case TC_RESID: return go<TC_RESID, BN>(a, a2, w, p, grid, st);
    case TC_SWIGLU: return go<TC_SWIGLU, BN>(a, a2, w, p, grid, st);
    case TC_QKV: return go<TC_QKV, BN>(a, a2, w, p, grid, st);
    default: return go<TC_PAGED, BN>(a, a2, w, p, grid, st);
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

bool tc_gemm_supported(const TcGemm& g) {
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
  if (g.K % 8 || g.lda % 8 || g.ldw % 8 || !al16(g.A) || !al16(g.W)) return false;
  if (g.A2 && (g.lda2 % 8 || !al16(g.A2))) return false;
  switch (g.epi) {
    case TC_STORE: return g.N % 8 == 0 && g.ldc % 8 == 0 && al16(g.C);
    case TC_RESID: return g.N % 4 == 0 && g.ldx % 4 == 0 && al16(g.X);
    case TC_SWIGLU: return g.ffn % 64 == 0 && g.N == 2 * g.ffn && g.ldc % 8 == 0 && al16(g.C);
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
  if (!get_encode()) return cudaErrorNotSupported;
  const int tiles128 = ((g.M + BM - 1) / BM) * ((g.N + 127) / 128);
  const bool stream_k = g.epi == TC_RESID && !g.A2 && tiles128 < 2 * g.n_sm;
  int bn = g.bn;
  if (bn != 128 && bn != 256) bn = tile_cost(g, 256, stream_k) <= tile_cost(g, 128, stream_k) ? 256 : 128;
  CUtensorMap ma, ma2, mw;
  if (!make_map(&ma, g.A, g.M, g.K, g.lda, BM)) return cudaErrorInvalidValue;
  if (!make_map(&mw, g.W, g.N, g.K, g.ldw, bn)) return cudaErrorInvalidValue;
  if (g.A2) { if (!make_map(&ma2, g.A2, g.M, g.K, g.lda2, BM)) return cudaErrorInvalidValue; }
  else ma2 = ma;
  Params p{};
  p.M = g.M; p.N = g.N; p.K = g.K; p.split_begin = g.split_begin; p.has_a2 = g.A2 != nullptr; p.status = status;
  p.stream_k = stream_k ? 1 : 0;
  p.C = g.C; p.ldc = g.ldc; p.X = g.X; p.ldx = g.ldx; p.C_lo = g.C_lo; p.ld_lo = g.ld_lo; p.lo_col_begin = g.lo_col_begin;
  p.q_gain = g.q_gain; p.k_gain = g.k_gain; p.q_cols = g.q_cols; p.eps = g.eps;
  p.rot_cols = g.rot_cols; p.hd = g.hd; p.rope_tab = g.rope_tab; p.tok_pos = g.tok_pos; p.ffn = g.ffn; p.paged = g.paged;
  const int tiles = ((g.M + BM - 1) / BM) * ((g.N + bn - 1) / bn);
  const long long kblocks = (long long)tiles * ((g.K + BK - 1) / BK);
  int grid = stream_k ? (int)(kblocks < g.n_sm ? kblocks : g.n_sm) : (tiles < g.n_sm ? tiles : g.n_sm);
  ++*n_launch;
  return bn == 256 ? go_epi<256>(g.epi, ma, ma2, mw, p, grid, st) : go_epi<128>(g.epi, ma, ma2, mw, p, grid, st);
}

// ---- RoPE table: tab[pos][c] = (cos, sin)(pos * theta^(-2c/hd)) -----------------------------
__global__ void rope_table_kernel(float2* tab, int n_pos, int half, const __grid_constant__ InvFreq inv) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pos * half) return;
  int pos = i / half, c = i - pos * half;
  float s, co;
  rope_sincos(pos, inv.f[c], &s, &co);
  tab[i] = make_float2(co, s);
}

void launch_rope_table(const LaunchCtx& ctx, float2* tab, int n_pos, int hd, float theta) {
  InvFreq inv;
  fill_inv_freq(&inv, hd, theta);
  int n = n_pos * (hd / 2);
  ++*ctx.n_launch;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, ctx.st>>>(tab, n_pos, hd / 2, inv);
}
