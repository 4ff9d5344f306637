// Projections of the single-token step on the tensor cores, for batches of more than a few rows.
//
// y[b, n] = sum_k W[n, k] x[b, k] with W streamed once from HBM is bandwidth-bound only while
// the multiply keeps up; beyond about 8 rows the CUDA cores do not.  Here the roles of the
// operands are swapped: a tile of 128 weight rows is the M side of tcgen05.mma, the activations
// are the N side (2 * Bp columns: each row as a bf16 hi part and a bf16 lo part of its fp32
// value, so that the activations lose nothing that matters), and the 128 x 2Bp accumulator
// lives in tensor memory.  All k blocks of all row tiles form one sequence that is cut into
// equal contiguous shares, one per SM, so every SM streams weights for the whole launch
// whatever the number of row tiles; a share's partial sums are added to the fp32 output with
// red.global (lanes = consecutive n: 128 contiguous bytes per instruction).
// Warp 0 feeds a ring of shared-memory stages with TMA, warp 1 issues the MMAs, warps 2-5 drain
// accumulators.  Every wait is bounded (DEV_TIMEOUT, all roles leave, tensor memory is freed).
#include "step_tc.h"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int BM = 128, BK = 64;
constexpr int W_BYTES = BM * BK * 2;
constexpr int N_THREADS = 192;
constexpr int SMEM_LIMIT = 220 * 1024;
constexpr size_t STEP_PREFETCH_MAX = 32u << 20;   // bytes of the next weight matrix asked into L2 (L2 holds 126 MB; this kernel streams through it too)

struct Params {
  int N, K, batch, Bp;
  int stages, x_bytes;      // ring depth; bytes of the activation tile of a stage (multiple of 1024)
  int acc_stride;           // tensor-memory columns between the two accumulators
  float* Y; int ldy;
  int* status;
  // The weights the NEXT projection will stream (null = none): once this kernel has requested all of its own tiles, every CTA
  // asks for its share of them to be brought into L2, so HBM keeps streaming through this kernel's tail, the operand
  // preparation and the launch gap.
  const char* next_w; long long next_bytes;
};

__device__ __forceinline__ void red_add(float* dst, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst), "f"(v) : "memory");
}

struct Work { int n0, kb0, kb1; };
struct Sched {
  int num_kb; long long g, g_end;
  __device__ __forceinline__ explicit Sched(const Params& p) {
    num_kb = (p.K + BK - 1) / BK;
    long long total = (long long)((p.N + BM - 1) / BM) * num_kb;
    g = total * blockIdx.x / gridDim.x;
    g_end = total * (blockIdx.x + 1) / gridDim.x;
  }
  __device__ __forceinline__ bool next(Work& w) {
    if (g >= g_end) return false;
    const int t = (int)(g / num_kb);
    w.n0 = t * BM;
    w.kb0 = (int)(g - (long long)t * num_kb);
    w.kb1 = (int)min((long long)num_kb, w.kb0 + (g_end - g));
    g += w.kb1 - w.kb0;
    return true;
  }
};

__global__ void __launch_bounds__(N_THREADS, 1)
step_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = W_BYTES + p.x_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.stages * stage_bytes);
  // bars: full[stages], empty[stages], tmem_full[2], tmem_empty[2]; then tmem base, abort flag
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(bars);
  const int S = p.stages;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_cols = max(32, 2 * p.acc_stride);
  pdl_trigger();      // the next kernel's CTAs may take SMs as this kernel's CTAs leave them

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      Sched sched(p);
      Work w;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      const uint32_t tx = W_BYTES + 2 * p.Bp * BK * 2;
      // The weights do not depend on the kernel before this one: the W tiles of the first S k-blocks are
      // requested before the wait for that kernel, so they stream in while it finishes (all stages are free,
      // in order, on a fresh pipeline).  The activation tiles of those k-blocks follow after the wait.
      int pre = 0;
      {
        Sched ahead(p);
        Work wa;
        while (pre < S && ahead.next(wa)) {
          for (int kb = wa.kb0; kb < wa.kb1 && pre < S; ++kb, ++pre) {
            mbar_expect_tx(full_bar(pre), tx);
            tma_load_2d(smem_base + pre * stage_bytes, &map_w, kb * BK, wa.n0, full_bar(pre));
          }
        }
      }
      pdl_wait();
      int issued = 0;
      while (ok && sched.next(w)) {
        for (int kb = w.kb0; kb < w.kb1 && ok; ++kb, ++issued) {
          const uint32_t sw = smem_base + stage * stage_bytes;
          if (issued >= pre) {
            ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status);
            if (!ok) break;
            mbar_expect_tx(full_bar(stage), tx);
            tma_load_2d(sw, &map_w, kb * BK, w.n0, full_bar(stage));
          }
          tma_load_2d(sw + W_BYTES, &map_x, kb * BK, 0, full_bar(stage));
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
      if (ok && p.next_w) {
        constexpr long long CHUNK = 64 * 1024;
        const long long n_chunks = (p.next_bytes + CHUNK - 1) / CHUNK;
        for (long long c = blockIdx.x; c < n_chunks; c += gridDim.x) {
          const long long off = c * CHUNK, len = min(CHUNK, p.next_bytes - off) & ~15ll;
          if (len > 0) bulk_prefetch_l2(p.next_w + off, (uint32_t)len);
        }
      }
      if (!ok) drain_after_abort();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(BM, 2 * p.Bp);
      Sched sched(p);
      Work w;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      while (ok && sched.next(w)) {
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * p.acc_stride;
        for (int kb = w.kb0; kb < w.kb1 && ok; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sw = smem_base + stage * stage_bytes;
          const uint64_t da = desc_kmajor(sw), db = desc_kmajor(sw + W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) tc_mma_bf16(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
          tc_commit(empty_bar(stage));
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) drain_after_abort();
    }
  } else {
    const int quarter = warp & 3;
    Sched sched(p);
    Work w;
    int acc = 0; uint32_t acc_phase = 0;
    pdl_wait();       // the output was cleared by the kernel before this one
    while (sched.next(w)) {
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int n = w.n0 + quarter * 32 + lane;
      const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.acc_stride;
#pragma unroll 1
      for (int c = 0; c < p.batch; c += 8) {
        float hi[8], lo[8];
        tmem_ld8(t_acc + c, hi);
        tmem_ld8(t_acc + p.Bp + c, lo);
        tmem_ld_wait();
        if (n < p.N) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (c + i < p.batch) red_add(p.Y + (size_t)(c + i) * p.ldy + n, hi[i] + lo[i]);
        }
      }
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
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// grid (operand row incl. pad rows, chunk of PREP_CHUNK elements); 8 elements per thread and step.
// Every CTA of a row recomputes the row's sum of squares (the row is a few KB in L2), so the
// chunks need no second kernel.
constexpr int PREP_CHUNK = 2048;

__global__ void __launch_bounds__(256) step_prep_kernel(int mode, const float* __restrict__ x, int ldx, int K, int batch, int Bp,
                                                        const float* __restrict__ gain, float eps, RowMap mg, RowMap mu,
                                                        bf16* __restrict__ XB, float* zero_ptr, int zero_ld, int zero_n) {
  __shared__ float red[8];
  pdl_trigger();
  pdl_wait();         // everything below reads or overwrites what earlier kernels of the step use
  const int b = blockIdx.x, tid = threadIdx.x;
  const int k_begin = blockIdx.y * PREP_CHUNK, k_end = min(K, k_begin + PREP_CHUNK);
  bf16* hi = XB + (size_t)b * K;
  bf16* lo = XB + (size_t)(Bp + b) * K;
  if (b >= batch) {
    for (int k = k_begin + tid * 8; k < k_end; k += 2048) {
      *reinterpret_cast<uint4*>(hi + k) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(lo + k) = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  const float* xr = x + (size_t)b * ldx;
  float r = 1.f;
  if (mode == PREP_NORM) {
    float ss = 0.f;
    for (int k = tid * 4; k < K; k += 1024) {
      const float4 v = *reinterpret_cast<const float4*>(xr + k);
      ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
    ss = warp_sum(ss);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += red[w];
    r = rsqrtf(t / (float)K + eps);
  }
  for (int k = k_begin + tid * 8; k < k_end; k += 2048) {
    float v[8];
    if (mode == PREP_SWIGLU) {
      // gate and up rows of 8 consecutive outputs are 8 consecutive elements each (interleave blocks are multiples of 8)
      const float* g = xr + map_row(mg, k);
      const float* u = xr + map_row(mu, k);
      const float4 g0 = *reinterpret_cast<const float4*>(g), g1 = *reinterpret_cast<const float4*>(g + 4);
      const float4 u0 = *reinterpret_cast<const float4*>(u), u1 = *reinterpret_cast<const float4*>(u + 4);
      const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w}, uv[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __fdividef(gv[i], 1.f + __expf(-gv[i])) * uv[i];
    } else {
      const float4 a0 = *reinterpret_cast<const float4*>(xr + k), a1 = *reinterpret_cast<const float4*>(xr + k + 4);
      v[0] = a0.x; v[1] = a0.y; v[2] = a0.z; v[3] = a0.w; v[4] = a1.x; v[5] = a1.y; v[6] = a1.z; v[7] = a1.w;
      if (mode == PREP_NORM) {
        const float4 c0 = *reinterpret_cast<const float4*>(gain + k), c1 = *reinterpret_cast<const float4*>(gain + k + 4);
        const float gg[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = gg[i] * v[i] * r;
      }
    }
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      const float2 hf = __bfloat1622float2(hh);
      const __nv_bfloat162 ll = __floats2bfloat162_rn(v[2 * i] - hf.x, v[2 * i + 1] - hf.y);
      h[i] = *reinterpret_cast<const uint32_t*>(&hh);
      l[i] = *reinterpret_cast<const uint32_t*>(&ll);
    }
    *reinterpret_cast<uint4*>(hi + k) = make_uint4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<uint4*>(lo + k) = make_uint4(l[0], l[1], l[2], l[3]);
  }
  if (zero_ptr) {
    const int n_chunks = gridDim.y;
    for (int i = blockIdx.y * 256 + tid; i < zero_n; i += n_chunks * 256) zero_ptr[(size_t)b * zero_ld + i] = 0.f;
  }
}

int pow2_ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }

}  // namespace

bool step_tc_supported(int batch, int K, int ldw, const void* W, const void* XB) {
  return batch >= 1 && step_tc_rows(batch) <= 128 && K % 8 == 0 && ldw % 8 == 0 && ((uintptr_t)W & 15) == 0 &&
         ((uintptr_t)XB & 15) == 0;
}

void launch_step_prep(const LaunchCtx& ctx, int mode, const float* x, int ldx, int K, int batch, const float* gain, float eps,
                      int G, bf16* XB, float* zero_ptr, int zero_ld, int zero_n) {
  const int Bp = step_tc_rows(batch);
  RowMap mg{0, G, 0, K}, mu{G == 0 ? K : 0, G, 1, K};
  ++*ctx.n_launch;
  launch_overlapped(step_prep_kernel, dim3(Bp, (K + PREP_CHUNK - 1) / PREP_CHUNK), dim3(256), 0, ctx.st, mode, x, ldx, K, batch, Bp, gain, eps,
                    mg, mu, XB, zero_ptr, zero_ld, zero_n);
}

cudaError_t launch_step_gemm_tc(const bf16* W, int ldw, int N, int K, const bf16* XB, int batch, float* Y, int ldy, int n_sm,
                                int* status, cudaStream_t st, int64_t* n_launch, const void* next_w, size_t next_bytes) {
  const int Bp = step_tc_rows(batch);
  CUtensorMap mw, mx;
  if (!tc_make_map_bf16(&mw, W, N, K, ldw, BM)) return cudaErrorInvalidValue;
  if (!tc_make_map_bf16(&mx, XB, 2 * Bp, K, K, 2 * Bp)) return cudaErrorInvalidValue;
  Params p{};
  p.N = N; p.K = K; p.batch = batch; p.Bp = Bp; p.Y = Y; p.ldy = ldy; p.status = status;
  p.next_w = (((uintptr_t)next_w & 15) == 0) ? (const char*)next_w : nullptr;
  p.next_bytes = (long long)(next_bytes < STEP_PREFETCH_MAX ? next_bytes : STEP_PREFETCH_MAX);
  p.x_bytes = (2 * Bp * BK * 2 + 1023) / 1024 * 1024;
  p.stages = (SMEM_LIMIT - 2048) / (W_BYTES + p.x_bytes);
  if (p.stages > 12) p.stages = 12;
  p.acc_stride = pow2_ceil(2 * Bp < 16 ? 16 : 2 * Bp);
  const int smem = p.stages * (W_BYTES + p.x_bytes) + 1024 + 8 * (2 * p.stages + 4) + 64;
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(step_gemm_kernel, SMEM_LIMIT, raised);
  if (e != cudaSuccess) return e;
  const long long total = (long long)((N + BM - 1) / BM) * ((K + BK - 1) / BK);
  const int grid = (int)(total < n_sm ? total : n_sm);
  ++*n_launch;
  return launch_overlapped(step_gemm_kernel, dim3(grid), dim3(N_THREADS), (size_t)smem, st, mw, mx, p);
}
