// Causal grouped-query attention over a ragged batch on the sm_100a tensor cores.
//
// One CTA = 128 consecutive queries of one sequence and one query head.  Warp 0 streams K and
// V tiles (128 keys) of the matching kv head with TMA straight out of the packed [T, q|k|v]
// projection buffer; warp 1 issues S = Q K^T and PV = P V with tcgen05.mma into tensor memory
// (two S buffers, one PV buffer); warps 2-5 own one query row per thread: they read S from
// tensor memory, keep the running max / sum in fp32, write P as bf16 into shared memory in the
// swizzled operand layout, and accumulate O in registers from the per-tile PV products, so
// no rescaling ever touches tensor memory.  S of tile j+1 is computed while the softmax of
// tile j runs.  Key tiles above the diagonal are skipped; the diagonal tile is masked.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <math.h>

#include "attn_tc.h"
#include "common.cuh"

namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int N_THREADS = 192;
constexpr uint32_t SPIN_LIMIT = 20u * 1000u * 1000u;
constexpr int P_BYTES = BQ * BKV * 2;

template <int HD> struct Cfg {
  static constexpr int TILE_BYTES = 128 * HD * 2;       // a Q, K or V tile
  static constexpr int STAGES = HD == 64 ? 3 : 2;
  static constexpr int SMEM = TILE_BYTES + P_BYTES + STAGES * 2 * TILE_BYTES + 1024 + 256;
};

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
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
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
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
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
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
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
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// K-major operand tile (rows of 128 bytes, 128B swizzle, 8-row groups 1024 B apart)
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
  uint64_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);
  uint64_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return lo | (hi << 32);
}
// MN-major operand tile: 64 contiguous MN elements per 128-byte row, rows = K index, 8-row groups
// 1024 B apart (stride offset), next 64 MN elements `lbo` bytes away (leading offset)
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr, uint32_t lbo) {
  uint64_t lo = ((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16);
  uint64_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return lo | (hi << 32);
}

struct Params {
  const int* cu; int batch; int nq, nkv;
  bf16* out; int ldo;
  float scale_log2e;
  int* status;
};

template <int HD>
__global__ void __launch_bounds__(N_THREADS, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap map_qkv, const Params p) {
  using C = Cfg<HD>;
  constexpr int ST = C::STAGES, TB = C::TILE_BYTES, NBOX = HD / 64;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int s_b, s_q0;
  // which (sequence, query tile): tiles are numbered sequence by sequence, last tile of a sequence first
  if (threadIdx.x == 0) {
    int blk = blockIdx.y, b = 0;
    for (; b < p.batch; ++b) {
      int nb = (p.cu[b + 1] - p.cu[b] + BQ - 1) / BQ;
      if (blk < nb) { blk = nb - 1 - blk; break; }
      blk -= nb;
    }
    s_b = b; s_q0 = blk * BQ;
  }
  __syncthreads();
  const int b = s_b, q0 = s_q0;
  if (b >= p.batch) return;
  const int base = p.cu[b], L = p.cu[b + 1] - base;
  const int head = blockIdx.x, kvh = head / (p.nq / p.nkv);
  const int n_kv = (min(L, q0 + BQ) + BKV - 1) / BKV;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sQ = smem_u32(smem), sP = sQ + TB, sKV = sP + P_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + TB + P_BYTES + ST * 2 * TB);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * ST + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar_base = smem_u32(bars);
  auto kv_full = [&](int s) { return bar_base + 8u * s; };
  auto kv_empty = [&](int s) { return bar_base + 8u * (ST + s); };
  auto s_full = [&](int i) { return bar_base + 8u * (2 * ST + i); };
  const uint32_t q_full = bar_base + 8u * (2 * ST + 2), p_ready = bar_base + 8u * (2 * ST + 3), pv_full = bar_base + 8u * (2 * ST + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < ST; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), 1); }
    mbar_init(s_full(0), 1); mbar_init(s_full(1), 1);
    mbar_init(q_full, 1); mbar_init(p_ready, 4); mbar_init(pv_full, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor memory: S0 at column 0, S1 at 128, PV at 256
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(q_full, TB);
#pragma unroll
      for (int x = 0; x < NBOX; ++x) tma_load_2d(sQ + x * 16384, &map_qkv, head * HD + x * 64, base + q0, q_full);
      const int kcol = (p.nq + kvh) * HD, vcol = (p.nq + p.nkv + kvh) * HD;
      int stage = 0; uint32_t phase = 0;
      for (int j = 0; j < n_kv && ok; ++j) {
        ok = mbar_wait(kv_empty(stage), phase ^ 1u, abort_flag, p.status);
        if (!ok) break;
        uint32_t sk = sKV + stage * 2 * TB, sv = sk + TB;
        mbar_expect_tx(kv_full(stage), 2 * TB);
#pragma unroll
        for (int x = 0; x < NBOX; ++x) {
          tma_load_2d(sk + x * 16384, &map_qkv, kcol + x * 64, base + j * BKV, kv_full(stage));
          tma_load_2d(sv + x * 16384, &map_qkv, vcol + x * 64, base + j * BKV, kv_full(stage));
        }
        if (++stage == ST) { stage = 0; phase ^= 1u; }
      }
      if (!ok) for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // S = Q K^T: M = 128 queries, N = 128 keys, both operands K-major over head_dim
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BKV >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
      // PV = P V: A = P (K-major over keys), B = V as stored [key][dim] = MN-major, N = head_dim
      const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
      bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
      int stage_qk = 0; uint32_t phase_qk = 0;      // stage of the next QK to issue
      int stage_pv = 0;                             // stage of the next PV to issue
      auto issue_qk = [&](int j) -> bool {
        if (!mbar_wait(kv_full(stage_qk), phase_qk, abort_flag, p.status)) return false;
        tc_fence_after();
        uint32_t sk = sKV + stage_qk * 2 * TB;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;
          tc_mma_bf16(tmem_base + (j & 1) * 128, desc_kmajor(sQ + off), desc_kmajor(sk + off), idesc_s, kk > 0 ? 1u : 0u);
        }
        tc_commit(s_full(j & 1));
        if (++stage_qk == ST) { stage_qk = 0; phase_qk ^= 1u; }
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int j = 0; j < n_kv && ok; ++j) {
        if (j + 1 < n_kv) { ok = issue_qk(j + 1); if (!ok) break; }
        ok = mbar_wait(p_ready, j & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        uint32_t sv = sKV + stage_pv * 2 * TB + TB;
#pragma unroll
        for (int kk = 0; kk < BKV / 16; ++kk) {
          uint64_t da = desc_kmajor(sP + (kk >> 2) * 16384 + (kk & 3) * 32);
          uint64_t db = desc_mnmajor(sv + kk * 2048, 16384);
          tc_mma_bf16(tmem_base + 256, da, db, idesc_pv, kk > 0 ? 1u : 0u);
        }
        tc_commit(pv_full);
        tc_commit(kv_empty(stage_pv));
        if (++stage_pv == ST) stage_pv = 0;
      }
      if (!ok) for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
  } else {
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;          // row of the query tile owned by this thread
    const int q_pos = q0 + r;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float c = p.scale_log2e;
    float m = -INFINITY, l = 0.f;
    float o[HD];
#pragma unroll
    for (int i = 0; i < HD; ++i) o[i] = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(s_full(j & 1), (j >> 1) & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tS = tmem_base + lane_off + (j & 1) * 128;
      const int kbase = j * BKV;
      const bool diag = kbase + BKV - 1 > q0;    // some key of this tile may lie above some query of the tile
      // pass 1: row maximum over the visible keys
      float mt = -INFINITY;
#pragma unroll 1
      for (int cc = 0; cc < BKV; cc += 32) {
        float v[32];
        tmem_ld32(tS + cc, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (!diag || kbase + cc + i <= q_pos) mt = fmaxf(mt, v[i]);
      }
      const float m_new = fmaxf(m, mt);
      const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2((m - m_new) * c);
      // fold in the previous tile's PV product (this also tells us that P may be overwritten)
      if (j > 0) {
        ok = mbar_wait(pv_full, (j - 1) & 1, abort_flag, p.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int cc = 0; cc < HD; cc += 32) {
          float v[32];
          tmem_ld32(tmem_base + lane_off + 256 + cc, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[cc + i] = (o[cc + i] + v[i]) * alpha;
        }
      }
      l *= alpha;
      // pass 2: probabilities, written as the bf16 A operand of the PV product
      const float mc = (m_new == -INFINITY) ? 0.f : m_new * c;
      float rowsum = 0.f;
#pragma unroll 1
      for (int cc = 0; cc < BKV; cc += 32) {
        float v[32];
        tmem_ld32(tS + cc, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float e = (!diag || kbase + cc + i <= q_pos) ? fast_exp2(v[i] * c - mc) : 0.f;
          rowsum += e;
          v[i] = e;
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          int k0 = cc + g * 8;
          uint32_t addr = sP + (k0 >> 6) * 16384 + r * 128 + ((((k0 & 63) >> 3) ^ (r & 7)) << 4);
          __nv_bfloat162 a0 = __floats2bfloat162_rn(v[g * 8], v[g * 8 + 1]), a1 = __floats2bfloat162_rn(v[g * 8 + 2], v[g * 8 + 3]);
          __nv_bfloat162 a2 = __floats2bfloat162_rn(v[g * 8 + 4], v[g * 8 + 5]), a3 = __floats2bfloat162_rn(v[g * 8 + 6], v[g * 8 + 7]);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t*>(&a0)),
                       "r"(*reinterpret_cast<uint32_t*>(&a1)), "r"(*reinterpret_cast<uint32_t*>(&a2)),
                       "r"(*reinterpret_cast<uint32_t*>(&a3)) : "memory");
        }
      }
      l += rowsum;
      m = m_new;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P visible to the tensor core's reads
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready);
    }
    if (ok) {
      ok = mbar_wait(pv_full, (n_kv - 1) & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l;
      bf16* dst = p.out + (size_t)(base + q_pos) * p.ldo + (size_t)head * HD;
#pragma unroll
      for (int cc = 0; cc < HD; cc += 32) {
        float v[32];
        tmem_ld32(tmem_base + lane_off + 256 + cc, v);
        tmem_ld_wait();
        if (q_pos < L) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float t[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) t[i] = (o[cc + g * 8 + i] + v[g * 8 + i]) * inv;
            __nv_bfloat162 a0 = __floats2bfloat162_rn(t[0], t[1]), a1 = __floats2bfloat162_rn(t[2], t[3]);
            __nv_bfloat162 a2 = __floats2bfloat162_rn(t[4], t[5]), a3 = __floats2bfloat162_rn(t[6], t[7]);
            uint4 u;
            u.x = *reinterpret_cast<uint32_t*>(&a0); u.y = *reinterpret_cast<uint32_t*>(&a1);
            u.z = *reinterpret_cast<uint32_t*>(&a2); u.w = *reinterpret_cast<uint32_t*>(&a3);
            *reinterpret_cast<uint4*>(dst + cc + g * 8) = u;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
bool get_encode() {
  if (g_encode) return true;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return false;
  g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  return true;
}

template <int HD>
cudaError_t go(const CUtensorMap& map, const Params& p, dim3 grid, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<HD>::SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  attn_tc_kernel<HD><<<grid, N_THREADS, Cfg<HD>::SMEM, st>>>(map, p);
  return cudaGetLastError();
}
}  // namespace

bool attn_tc_supported(int hd, int ld, const void* qkv, int ldo, const void* out) {
  return (hd == 64 || hd == 128) && ld % 8 == 0 && ((uintptr_t)qkv & 15) == 0 && ldo % 8 == 0 && ((uintptr_t)out & 15) == 0;
}

cudaError_t launch_attn_tc(const bf16* qkv, int ld, int total, int nq, int nkv, int hd, const int* cu_dev, int batch,
                           bf16* out, int ldo, int* status, cudaStream_t st, int64_t* n_launch) {
  if (!get_encode()) return cudaErrorNotSupported;
  CUtensorMap map;
  cuuint64_t dims[2] = {(cuuint64_t)((nq + 2 * nkv) * hd), (cuuint64_t)total};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, 128};
  cuuint32_t estr[2] = {1, 1};
  if (g_encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(qkv), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  Params p{cu_dev, batch, nq, nkv, out, ldo, (1.f / sqrtf((float)hd)) * 1.4426950408889634f, status};
  dim3 grid(nq, (total + BQ - 1) / BQ + batch);
  ++*n_launch;
  return hd == 64 ? go<64>(map, p, grid, st) : go<128>(map, p, grid, st);
}
