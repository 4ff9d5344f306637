// Causal grouped-query attention over a ragged batch on the sm_100a tensor cores.
//
// One CTA = 256 consecutive queries of one sequence (two tiles of 128) and one query head.
// Warp 0 streams K and V tiles (128 keys) of the matching kv head with TMA straight out of the
// packed [T, q|k|v] projection buffer, K and V through rings of their own (the K tile of the next
// S product is wanted long before the V tile of this P V product); both query tiles use them.
// S = Q K^T and O += P V run on tcgen05.mma with S, P and O in tensor memory.  Two groups of four
// warps, one per query tile, own one query row per thread: a thread copies its row of S into
// registers in one go (which frees the S columns at once), keeps the running max / sum in fp32
// and writes P as packed 16-bit values into tensor-memory columns of its own, from where the P V
// product takes it as its A operand (P never touches shared memory).  So S of the next key tile
// is computed while the softmax of this one runs, and a group never waits for its own products.
//   head_dim 64: every tile has its S, P and O columns (2 x (128 + 64 + 64) = 512); one warp
//     issues the products of both tiles.
//   head_dim 128: the two O take half of tensor memory, so both tiles share ONE S buffer, used in
//     turns (S0(0), S1(0), S0(1), ...), and each has an issuing warp of its own.
// The issuing warps are event loops: whichever product has its inputs is issued, all 32 lanes
// running the loop so that its state stays warp-uniform and one elected lane issuing.
// O is accumulated by the tensor core itself and only touched when a row's maximum has grown
// by more than 2^8 since the exponent offset was last fixed; then the group rescales its O in
// tensor memory (tcgen05.ld / st).  Key tiles above the diagonal are skipped; tiles touching it
// are masked.  Work is ordered so that, over the whole batch, CTAs with the most key tiles start first.
#include <math.h>

#include "attn_tc.h"
#include "tc_ptx.cuh"

namespace {
using namespace tcp;

constexpr int BQ = 128;                 // queries per tile; a CTA has two tiles
constexpr int N_THREADS = 384;          // warps: 0 TMA, 1 / 2 issuers of tile 0 / 1, 3 idle, 4-7 softmax of tile 0, 8-11 of tile 1
// Registers move from the loader / issuer warp group to the two softmax groups once the roles split (setmaxnreg): the
// kernel is launched with 168 per thread, 128 x REGS_LOW + 256 x REGS_HIGH = 384 x 168.  The launcher refuses the kernel
// if it was compiled with fewer (the raise would wait for registers that do not exist).
constexpr int REGS_LAUNCH = 168, REGS_LOW = 56, REGS_HIGH = 224;
static_assert(128 * REGS_LOW + 256 * REGS_HIGH <= 384 * REGS_LAUNCH, "register split exceeds the launch's registers");
constexpr float RESCALE_LOG2 = 8.f;     // tolerated growth of a row maximum before O is rescaled

template <int HD> struct Cfg {
  static constexpr int BKV = 128;                       // keys per tile
  static constexpr int K_STAGES = HD == 64 ? 4 : 3;     // K tiles in flight (16 / 32 KiB each)
  static constexpr int V_STAGES = HD == 64 ? 4 : 2;     // V tiles in flight
  static constexpr int Q_BYTES = BQ * HD * 2;
  static constexpr int KV_BYTES = BKV * HD * 2;         // a K or a V tile
  static constexpr int SMEM = 2 * Q_BYTES + (K_STAGES + V_STAGES) * KV_BYTES + 1024 + 256;
  // Tensor-memory columns.  head_dim 64: S of tile g, O of tile g, P of tile g (packed 16-bit: 64 columns for 128 keys).
  // head_dim 128: the two O take half of the 512 columns, so both query tiles share ONE S buffer (a group copies its S
  // into registers at once, then the buffer is free for the other group) and each has P columns of its own.
  static constexpr bool S_SHARED = HD == 128;
  static constexpr bool TWO_ISSUERS = HD == 128;      // one issuing warp per query tile, or one for both
  // head_dim 64 is bound by the exp unit (one exponential per 2 x 64 MACs): one pair of exponentials in eight is computed on the
  // FMA pipe instead (+5 %; larger shares, and any share at head_dim 128, cost more issue slots than they save)
  static constexpr bool FMA_EXP2 = HD == 64;
  static constexpr int S_COL0 = 0, S_STRIDE = S_SHARED ? 0 : 128;
  static constexpr int P_COL0 = S_SHARED ? 128 : 384, P_STRIDE = 64;
  static constexpr int O_COL0 = 256, O_STRIDE = HD;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for a pair on the FMA pipe: x = n + f with n = round(x), |f| <= 1/2; a cubic for 2^f (relative error 7.5e-5),
// n added into the exponent field.  x <= 127; anything below -126 (masked scores included) gives 2^-126.
__device__ __forceinline__ float2 exp2_fma(float2 x) {
  x.x = fmaxf(x.x, -126.f); x.y = fmaxf(x.y, -126.f);
  const float2 magic = make_float2(12582912.f, 12582912.f);          // 1.5 * 2^23: the sum's low mantissa bits hold round(x)
  const float2 r = __fadd2_rn(x, magic);
  const float2 n = __fadd2_rn(r, make_float2(-12582912.f, -12582912.f));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(f, make_float2(0.0551714076f, 0.0551714076f), make_float2(0.2426107455f, 0.2426107455f));
  p = __ffma2_rn(p, f, make_float2(0.6932609900f, 0.6932609900f));
  p = __ffma2_rn(p, f, make_float2(0.9999280967f, 0.9999280967f));
  p.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(r.x) << 23));
  p.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(r.y) << 23));
  return p;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// MN-major operand tile: 64 contiguous MN elements per 128-byte row, rows = K index, 8-row groups
// 1024 B apart (stride offset), next 64 MN elements `lbo` bytes away (leading offset)
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr, uint32_t lbo) {
  uint64_t lo = ((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16);
  uint64_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return lo | (hi << 32);
}

// one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
  uint32_t is_leader;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(is_leader));
  return is_leader != 0;
}
// D (+)= A B.  The matrix descriptors of one tile differ only in the start-address field (low word), so they are passed
// as two words and the issuing loop only adds to the low one.  mma_ts: A from tensor memory (row i of A in lane i, two
// 16-bit elements per 32-bit column).
template <bool ACC>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}
template <bool ACC>
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}

// 32 lanes x 128 columns of fp32 in one instruction: thread i of the warp gets lane (row) i, register j = column j.
__device__ __forceinline__ void tmem_ld128(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x128.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64, %65, %66, %67, %68, %69, %70, %71, %72, %73, %74, %75, %76, %77, %78, %79, %80, %81, %82, %83, %84, %85, %86, %87, %88, %89, %90, %91, %92, %93, %94, %95, %96, %97, %98, %99, %100, %101, %102, %103, %104, %105, %106, %107, %108, %109, %110, %111, %112, %113, %114, %115, %116, %117, %118, %119, %120, %121, %122, %123, %124, %125, %126, %127}, [%128];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
               : "r"(taddr) : "memory");
}

struct Params {
  const int* cu; const int2* sched;     // sched[i] = (sequence, first query of the pair of tiles)
  int nq, nkv;
  bf16* out; int ldo;
  float scale_log2e;
  int* status;
  int tiles;                            // query tiles per CTA: 2, or 1 when pairs would leave SMs idle
  bf16* out_lo;                         // bf16 remainder of the output (same layout as out), or null
};

// F16: q, k, v hold IEEE halves instead of bf16 (and P is packed as halves): same kernel, other operand format bits
template <int HD, bool F16>
__global__ void __launch_bounds__(N_THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv, const Params p) {
  using C = Cfg<HD>;
  constexpr int BKV = C::BKV, QB = C::Q_BYTES, KB = C::KV_BYTES, NBOX = HD / 64, KS = C::K_STAGES, VS = C::V_STAGES;
  constexpr int KV_BOX = BKV * 128;     // bytes of one 64-column box of a K or V tile
  extern __shared__ uint8_t smem_raw[];
  pdl_trigger();
  if (threadIdx.x == 32) { prefetch_tensormap(&map_q); prefetch_tensormap(&map_kv); }
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sQ = smem_u32(smem), sK = sQ + 2 * QB, sV = sK + KS * KB;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * QB + (KS + VS) * KB);
  constexpr int N_BARS = 2 * KS + 2 * VS + 9;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar_base = smem_u32(bars);
  auto k_full = [&](int s) { return bar_base + 8u * s; };
  auto k_empty = [&](int s) { return bar_base + 8u * (KS + s); };
  auto v_full = [&](int s) { return bar_base + 8u * (2 * KS + s); };
  auto v_empty = [&](int s) { return bar_base + 8u * (2 * KS + VS + s); };
  constexpr int B0 = 2 * KS + 2 * VS;
  auto s_full = [&](int g) { return bar_base + 8u * (B0 + g); };
  auto s_free = [&](int g) { return bar_base + 8u * (B0 + 2 + g); };
  auto p_ready = [&](int g) { return bar_base + 8u * (B0 + 4 + g); };
  auto pv_done = [&](int g) { return bar_base + 8u * (B0 + 6 + g); };
  const uint32_t q_full = bar_base + 8u * (B0 + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    // a K (V) stage goes back to the loader when BOTH query tiles are through with it: one arrival per issuer warp
    for (int s = 0; s < KS; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), C::TWO_ISSUERS ? 2 : 1); }
    for (int s = 0; s < VS; ++s) { mbar_init(v_full(s), 1); mbar_init(v_empty(s), C::TWO_ISSUERS ? 2 : 1); }
    for (int g = 0; g < 2; ++g) { mbar_init(s_full(g), 1); mbar_init(s_free(g), 4); mbar_init(p_ready(g), 4); mbar_init(pv_done(g), 1); }
    mbar_init(q_full, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();         // set-up above overlapped the previous kernel's tail; its results are needed from here on
  const int2 item = p.sched[blockIdx.y];
  const int b = item.x, q0 = item.y;
  const int base = p.cu[b], L = p.cu[b + 1] - base;
  const int head = blockIdx.x, kvh = head / (p.nq / p.nkv);
  // key tiles each query tile needs (tile 1 may lie beyond the end of the sequence)
  int n_kv[2];
  n_kv[0] = (min(L, q0 + BQ) + BKV - 1) / BKV;
  n_kv[1] = (p.tiles == 2 && q0 + BQ < L) ? (min(L, q0 + 2 * BQ) + BKV - 1) / BKV : 0;
  const int n_max = max(n_kv[0], n_kv[1]);

  if (warp < 4) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_LOW));
  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(q_full, 2 * QB);
#pragma unroll
      for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int x = 0; x < NBOX; ++x) tma_load_2d(sQ + g * QB + x * 16384, &map_q, head * HD + x * 64, base + q0 + g * BQ, q_full);
      const int kcol = (p.nq + kvh) * HD, vcol = (p.nq + p.nkv + kvh) * HD;
      // An issuer per tile: K tile j + 1 is wanted (for the next S) before V tile j (for this P V), and loads go out in
      // that order; one issuer: K and V of a tile together (their stages also come back together).
      auto load_k = [&](int j) {
        const int st = j % KS;
        if (!mbar_wait(k_empty(st), ((j / KS) & 1u) ^ 1u, abort_flag, p.status)) return false;
        mbar_expect_tx(k_full(st), KB);
#pragma unroll
        for (int x = 0; x < NBOX; ++x) tma_load_2d(sK + st * KB + x * KV_BOX, &map_kv, kcol + x * 64, base + j * BKV, k_full(st));
        return true;
      };
      if (C::TWO_ISSUERS) ok = load_k(0);
      for (int j = 0; j < n_max && ok; ++j) {
        if (!C::TWO_ISSUERS) ok = load_k(j);
        else if (j + 1 < n_max) ok = load_k(j + 1);
        if (!ok) break;
        const int st = j % VS;
        ok = mbar_wait(v_empty(st), ((j / VS) & 1u) ^ 1u, abort_flag, p.status);
        if (!ok) break;
        mbar_expect_tx(v_full(st), KB);
#pragma unroll
        for (int x = 0; x < NBOX; ++x) tma_load_2d(sV + st * KB + x * KV_BOX, &map_kv, vcol + x * 64, base + j * BKV, v_full(st));
      }
      if (!ok) drain_after_abort();
    }
  } else if (warp == 1 || (warp == 2 && C::TWO_ISSUERS)) {
    // Issuer of the tensor-core instructions: one warp per query tile (head_dim 128) or one warp for both (head_dim 64).
    // All 32 lanes run this loop, so that addresses, descriptors and loop state stay warp-uniform; one elected lane issues
    // each instruction.
    const int g_lo = C::TWO_ISSUERS ? warp - 1 : 0, g_hi = C::TWO_ISSUERS ? warp - 1 : 1;
    // S = Q K^T: M = 128 queries, N = BKV keys, both operands K-major over head_dim
    const uint32_t fmt_mask = F16 ? ~((7u << 7) | (7u << 10)) : ~0u;       // operand format fields: 0 = IEEE half
    const uint32_t idesc_s = idesc_bf16(BQ, BKV) & fmt_mask;
    // O += P V: A = P (K-major over keys), B = V as stored [key][dim] = MN-major, N = head_dim
    const uint32_t idesc_pv = (idesc_bf16(BQ, HD) & fmt_mask) | (1u << 16);
    const uint64_t dq0 = desc_kmajor(sQ), dk0 = desc_kmajor(sK), dv0 = desc_mnmajor(sV, KV_BOX);
    const uint32_t dq_lo = (uint32_t)dq0, dk_lo = (uint32_t)dk0, dv_lo = (uint32_t)dv0;
    const uint32_t dk_hi = (uint32_t)(dk0 >> 32), dv_hi = (uint32_t)(dv0 >> 32);      // Q and K share the high word
    auto poll = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_poll(bar, parity)); };
    bool ok = __all_sync(0xffffffffu, mbar_wait(q_full, 0, abort_flag, p.status));
    // Event loop: S of the next key tile and P V of the oldest tile not yet multiplied are issued as soon as their own
    // inputs are there, in whichever order that happens.  ts / tp = next S / P V tile of a query tile; tk / tv = next key
    // tile it does NOT use, whose stage still has to be handed back on its behalf.
    int ts[2] = {0, 0}, tp[2] = {0, 0}, tk[2] = {n_kv[0], n_kv[1]}, tv[2] = {n_kv[0], n_kv[1]};
    int released = 0;                   // one issuer for both tiles: key tiles whose stages have been handed back
    uint32_t idle = 0;
    auto pending = [&](int g) { return tp[g] < n_kv[g] || (C::TWO_ISSUERS && (tk[g] < n_max || tv[g] < n_max)); };
    while (ok && (pending(g_lo) || pending(g_hi))) {
      bool progress = false;
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        if (g < g_lo || g > g_hi) continue;
        const int n = n_kv[g], n_other = n_kv[g ^ 1];
        const uint32_t tS = tmem_base + C::S_COL0 + g * C::S_STRIDE, tP = tmem_base + C::P_COL0 + g * C::P_STRIDE;
        const uint32_t tO = tmem_base + C::O_COL0 + g * C::O_STRIDE;
        auto issue_s = [&]() {
          if (ts[g] < n) {
            const int t = ts[g];
            // the S columns are free once their last user has copied them into registers
            bool ready = t == 0 || poll(s_free(g), (t - 1) & 1u);
            if (C::S_SHARED && ready) {       // uses of the shared buffer alternate: S0(0), S1(0), S0(1), S1(1), ...
              if (g == 1) { if (t < n_other) ready = poll(s_free(0), t & 1u); }
              else if (t > 0 && t - 1 < n_other) ready = poll(s_free(1), (t - 1) & 1u);
            }
            const int ks = t % KS;
            if (ready && poll(k_full(ks), (t / KS) & 1u)) {
              tc_fence_after();
              const uint32_t aq = dq_lo + g * (QB >> 4), bq = dk_lo + ks * (KB >> 4);
              if (elect_one()) mma_ss<false>(tS, aq, dk_hi, bq, dk_hi, idesc_s);
#pragma unroll
              for (int kk = 1; kk < HD / 16; ++kk)
                if (elect_one()) mma_ss<true>(tS, aq + (kk >> 2) * (16384 >> 4) + (kk & 3) * 2, dk_hi, bq + (kk >> 2) * (KV_BOX >> 4) + (kk & 3) * 2, dk_hi, idesc_s);
              if (elect_one()) { tc_commit(s_full(g)); if (C::TWO_ISSUERS) tc_commit(k_empty(ks)); }
              ++ts[g];
              progress = true;
            }
          }
        };
        auto issue_pv = [&]() {
          if (tp[g] < ts[g]) {
            const int t = tp[g], vs = t % VS;
            if (poll(p_ready(g), t & 1u) && poll(v_full(vs), (t / VS) & 1u)) {
              tc_fence_after();
              const uint32_t bv = dv_lo + vs * (KB >> 4);
              if (t > 0) { if (elect_one()) mma_ts<true>(tO, tP, bv, dv_hi, idesc_pv); }
              else { if (elect_one()) mma_ts<false>(tO, tP, bv, dv_hi, idesc_pv); }
#pragma unroll
              for (int kk = 1; kk < BKV / 16; ++kk)      // 16 keys = 8 packed columns of P per step
                if (elect_one()) mma_ts<true>(tO, tP + kk * 8, bv + kk * (2048 >> 4), dv_hi, idesc_pv);
              if (elect_one()) { tc_commit(pv_done(g)); if (C::TWO_ISSUERS) tc_commit(v_empty(vs)); }
              ++tp[g];
              progress = true;
            }
          }
        };
        // one issuer for both tiles: P V first (it is what the tile's next softmax waits for); an issuer per tile: S first
        if (C::TWO_ISSUERS) { issue_s(); issue_pv(); } else { issue_pv(); issue_s(); }
        // (a stage's barrier is only asked about the tile that follows the last one seen on it: parity waits are ambiguous beyond that)
        if (C::TWO_ISSUERS && ts[g] >= n && tk[g] < n_max && poll(k_full(tk[g] % KS), (tk[g] / KS) & 1u)) {
          if (lane == 0) mbar_arrive(k_empty(tk[g] % KS));
          ++tk[g];
          progress = true;
        }
        if (C::TWO_ISSUERS && tp[g] >= n && tv[g] < n_max && poll(v_full(tv[g] % VS), (tv[g] / VS) & 1u)) {
          if (lane == 0) mbar_arrive(v_empty(tv[g] % VS));
          ++tv[g];
          progress = true;
        }
      }
      if (!C::TWO_ISSUERS) {
        // a K / V stage pair goes back to the loader once every query tile that uses its key tile has issued P V on it
        while (released < n_max && (n_kv[0] <= released || tp[0] > released) && (n_kv[1] <= released || tp[1] > released)) {
          if (elect_one()) { tc_commit(k_empty(released % KS)); tc_commit(v_empty(released % VS)); }
          ++released;
        }
      }
      if (progress) {
        idle = 0;
      } else if (++idle > SPIN_LIMIT) {
        if (lane == 0) { *abort_flag = 1; dev_flag(p.status, DEV_TIMEOUT); }
        ok = false;
      } else if ((idle & 63u) == 63u) {
        if (__any_sync(0xffffffffu, *abort_flag != 0)) ok = false;
      }
    }
    if (!ok && lane == 0) drain_after_abort();
    __syncwarp();
  } else if (warp >= 4) {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_HIGH));
    const int g = (warp - 4) >> 2;              // query tile of this warp's group
    const int quarter = warp & 3;               // tensor-memory lane quarter this warp may access
    const int r = quarter * 32 + lane;          // row of the query tile owned by this thread
    const int qs = q0 + g * BQ, q_pos = qs + r;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t tS = tmem_base + lane_off + C::S_COL0 + g * C::S_STRIDE, tO = tmem_base + lane_off + C::O_COL0 + g * C::O_STRIDE;
    const uint32_t tP = tmem_base + lane_off + C::P_COL0 + g * C::P_STRIDE;
    const float c = p.scale_log2e;
    const int n = n_kv[g];
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n; ++j) {
      ok = mbar_wait(s_full(g), j & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float s[BKV];
      tmem_ld128(tS, s);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free(g));
      const int kbase = j * BKV;
      const bool diag = kbase + BKV - 1 > qs;     // some key of this tile lies above some query of the tile
      if (diag) {
#pragma unroll
        for (int i = 0; i < BKV; ++i) if (kbase + i > q_pos) s[i] = -INFINITY;
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};    // four chains of three-input maxima
#pragma unroll
      for (int i = 0; i < BKV; i += 8) {
        mx[0] = fmax3(mx[0], s[i], s[i + 1]); mx[1] = fmax3(mx[1], s[i + 2], s[i + 3]);
        mx[2] = fmax3(mx[2], s[i + 4], s[i + 5]); mx[3] = fmax3(mx[3], s[i + 6], s[i + 7]);
      }
      const float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      // The previous P V product must have read P and finished writing O before P is overwritten or O rescaled.  The
      // exponentials do not depend on it: the wait sits in front of the first P store (and of the rare rescale).
      bool pv_seen = j == 0;
      const bool need = mt > m_ref && (m_ref == -INFINITY || (mt - m_ref) * c > RESCALE_LOG2);
      if (__any_sync(0xffffffffu, need)) {
        if (!pv_seen) {
          ok = mbar_wait(pv_done(g), (j - 1) & 1, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          pv_seen = true;
        }
        const float alpha = (need && m_ref != -INFINITY) ? fast_exp2((m_ref - mt) * c) : 1.f;
        if (j > 0) {
#pragma unroll 1
          for (int cc = 0; cc < HD; cc += 32) {
            float v[32];
            tmem_ld32(tO + cc, v);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] *= alpha;
            tmem_st32(tO + cc, v);
          }
          tmem_st_wait();
        }
        l *= alpha;
        if (need) m_ref = mt;
      }
      const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * c;
      float2 rs2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 c2 = make_float2(c, c), nmc2 = make_float2(-mc, -mc);
#pragma unroll
      for (int hf = 0; hf < BKV / 64; ++hf) {        // 64 keys = 32 packed columns of P per tensor-memory store
        uint32_t pk[32];
#pragma unroll
        for (int g8 = 0; g8 < 8; ++g8) {
          const int k0 = hf * 64 + g8 * 8;
          float2 x[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            x[q] = __ffma2_rn(make_float2(s[k0 + 2 * q], s[k0 + 2 * q + 1]), c2, nmc2);     // two scaled scores per instruction
            if (C::FMA_EXP2 && ((g8 * 4 + q) & 7) == 7) x[q] = exp2_fma(x[q]);
            else { x[q].x = fast_exp2(x[q].x); x[q].y = fast_exp2(x[q].y); }             // exp2(-inf) = 0
            if (F16) {                                                                    // key 2i in the low half of column i
              const __half2 h2 = __floats2half2_rn(x[q].x, x[q].y);
              pk[g8 * 4 + q] = *reinterpret_cast<const uint32_t*>(&h2);
            } else {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(x[q].x, x[q].y);
              pk[g8 * 4 + q] = *reinterpret_cast<const uint32_t*>(&h2);
            }
          }
          rs2[0] = __fadd2_rn(rs2[0], x[0]); rs2[1] = __fadd2_rn(rs2[1], x[1]);
          rs2[0] = __fadd2_rn(rs2[0], x[2]); rs2[1] = __fadd2_rn(rs2[1], x[3]);
        }
        if (hf == 0 && !pv_seen) {
          ok = mbar_wait(pv_done(g), (j - 1) & 1, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          tc_fence_after();
        }
        if (ok) tmem_st32(tP + hf * 32, reinterpret_cast<const float*>(pk));
      }
      if (!ok) break;
      tmem_st_wait();
      l += (rs2[0].x + rs2[0].y) + (rs2[1].x + rs2[1].y);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready(g));
    }
    if (ok && n > 0) {
      ok = mbar_wait(pv_done(g), (n - 1) & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && n > 0) {
      tc_fence_after();
      const float inv = 1.f / l;
      bf16* dst = p.out + (size_t)(base + q_pos) * p.ldo + (size_t)head * HD;
#pragma unroll 1
      for (int cc = 0; cc < HD; cc += 32) {
        float v[32];
        tmem_ld32(tO + cc, v);
        tmem_ld_wait();
        if (q_pos < L) {
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            __nv_bfloat162 a0 = __floats2bfloat162_rn(v[g8 * 8] * inv, v[g8 * 8 + 1] * inv);
            __nv_bfloat162 a1 = __floats2bfloat162_rn(v[g8 * 8 + 2] * inv, v[g8 * 8 + 3] * inv);
            __nv_bfloat162 a2 = __floats2bfloat162_rn(v[g8 * 8 + 4] * inv, v[g8 * 8 + 5] * inv);
            __nv_bfloat162 a3 = __floats2bfloat162_rn(v[g8 * 8 + 6] * inv, v[g8 * 8 + 7] * inv);
            uint4 u;
            u.x = *reinterpret_cast<uint32_t*>(&a0); u.y = *reinterpret_cast<uint32_t*>(&a1);
            u.z = *reinterpret_cast<uint32_t*>(&a2); u.w = *reinterpret_cast<uint32_t*>(&a3);
            *reinterpret_cast<uint4*>(dst + cc + g8 * 8) = u;
            if (p.out_lo) {
              float rem[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) { const float f = v[g8 * 8 + i] * inv; rem[i] = f - __bfloat162float(__float2bfloat16_rn(f)); }
              __nv_bfloat162 b0 = __floats2bfloat162_rn(rem[0], rem[1]), b1 = __floats2bfloat162_rn(rem[2], rem[3]);
              __nv_bfloat162 b2 = __floats2bfloat162_rn(rem[4], rem[5]), b3 = __floats2bfloat162_rn(rem[6], rem[7]);
              uint4 w;
              w.x = *reinterpret_cast<uint32_t*>(&b0); w.y = *reinterpret_cast<uint32_t*>(&b1);
              w.z = *reinterpret_cast<uint32_t*>(&b2); w.w = *reinterpret_cast<uint32_t*>(&b3);
              *reinterpret_cast<uint4*>(p.out_lo + (size_t)(base + q_pos) * p.ldo + (size_t)head * HD + cc + g8 * 8) = w;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// Work list: pairs of query tiles of all sequences, those nearest the end of their sequence
// (most key tiles) first.  One block, thread = sequence.
__global__ void __launch_bounds__(256) attn_schedule_kernel(const int* __restrict__ cu, int batch, int tiles, int2* __restrict__ sched) {
  __shared__ int s_warp[8];
  __shared__ int s_base;
  const int b = threadIdx.x, warp = b >> 5, lane = b & 31;
  const int span = tiles * BQ;            // queries per work item
  const int np = b < batch ? (cu[b + 1] - cu[b] + span - 1) / span : 0;
  int max_np = np;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) max_np = max(max_np, __shfl_xor_sync(0xffffffffu, max_np, o));
  if (lane == 0) s_warp[warp] = max_np;
  if (b == 0) s_base = 0;
  __syncthreads();
  max_np = 0;
  for (int w = 0; w < 8; ++w) max_np = max(max_np, s_warp[w]);
  __syncthreads();
  for (int r = 0; r < max_np; ++r) {
    const bool has = np > r;
    const unsigned bal = __ballot_sync(0xffffffffu, has);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int pos = s_base + __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) pos += s_warp[w];
    if (has) sched[pos] = make_int2(b, (np - 1 - r) * span);
    __syncthreads();
    if (b == 0) { int t = 0; for (int w = 0; w < 8; ++w) t += s_warp[w]; s_base += t; }
    __syncthreads();
  }
}

template <int HD, bool F16>
cudaError_t go(const CUtensorMap& mq, const CUtensorMap& mkv, const Params& p, dim3 grid, cudaStream_t st) {
  static bool raised[TC_MAX_DEVICES] = {};
  cudaError_t e = tc_raise_smem_limit(attn_tc_kernel<HD, F16>, Cfg<HD>::SMEM, raised);
  if (e != cudaSuccess) return e;
  static int regs = 0;                  // a property of the compiled kernel, the same on every device
  if (regs == 0) {
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, attn_tc_kernel<HD, F16>);
    if (e != cudaSuccess) return e;
    regs = fa.numRegs;
  }
  if (regs < REGS_LAUNCH) return cudaErrorLaunchOutOfResources;
  return launch_overlapped(attn_tc_kernel<HD, F16>, grid, dim3(N_THREADS), Cfg<HD>::SMEM, st, mq, mkv, p);
}
}  // namespace

bool attn_tc_supported(int hd, int ld, const void* qkv, int ldo, const void* out) {
  return (hd == 64 || hd == 128) && ld % 8 == 0 && ((uintptr_t)qkv & 15) == 0 && ldo % 8 == 0 && ((uintptr_t)out & 15) == 0;
}

int attn_tc_items(const int* cu_host, int batch, int tiles) {
  int n = 0;
  for (int b = 0; b < batch; ++b) n += (cu_host[b + 1] - cu_host[b] + tiles * BQ - 1) / (tiles * BQ);
  return n;
}

void launch_attn_schedule(const int* cu_dev, int batch, int tiles, int2* sched, cudaStream_t st, int64_t* n_launch) {
  ++*n_launch;
  attn_schedule_kernel<<<1, 256, 0, st>>>(cu_dev, batch, tiles, sched);
}

cudaError_t launch_attn_tc(const bf16* qkv, int ld, int total, int nq, int nkv, int hd, const int* cu_dev, const int2* sched,
                           int n_items, int tiles, bf16* out, int ldo, int* status, cudaStream_t st, int64_t* n_launch,
                           bool half_operands, bf16* out_lo) {
  CUtensorMap mq, mkv;
  const int bkv = 128;
  if (!tc_make_map_bf16(&mq, qkv, total, (long long)(nq + 2 * nkv) * hd, ld, BQ)) return cudaErrorInvalidValue;
  if (!tc_make_map_bf16(&mkv, qkv, total, (long long)(nq + 2 * nkv) * hd, ld, bkv)) return cudaErrorInvalidValue;
  Params p{cu_dev, sched, nq, nkv, out, ldo, (1.f / sqrtf((float)hd)) * 1.4426950408889634f, status, tiles, out_lo};
  dim3 grid(nq, n_items);
  ++*n_launch;
  if (half_operands) return hd == 64 ? go<64, true>(mq, mkv, p, grid, st) : go<128, true>(mq, mkv, p, grid, st);
  return hd == 64 ? go<64, false>(mq, mkv, p, grid, st) : go<128, false>(mq, mkv, p, grid, st);
}
