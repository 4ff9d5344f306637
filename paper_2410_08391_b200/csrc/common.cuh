// Shared device helpers and launch-function declarations for the KV Prediction library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;
// Element of the paged cache in bf16 mode.  The predicted cache is the product of the path, and the base step
// amplifies its rounding about five-fold in the logits, so its 16 bits carry 11 significant bits (IEEE half)
// instead of bfloat16's 8.  Stores saturate at the largest finite half.
typedef __half kv16;

// Codes kernels write into the device status word (first int of the workspace).
enum : int { DEV_OK = 0, DEV_TIMEOUT = 1, DEV_BAD_TOKEN = 2, DEV_BAD_PAGE = 3 };

constexpr int PAGE_TOKENS = 64;
constexpr int MAX_PRED_SEG = 8;   // base layers fed by one auxiliary layer

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f(kv16 v) { return __half2float(v); }
template <class T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ kv16 from_f<kv16>(float v) { return __float2half_rn(fminf(fmaxf(v, -65504.f), 65504.f)); }
// two values as packed IEEE halves (lo in the low 16 bits), saturating at the largest finite half: one instruction
__device__ __forceinline__ uint32_t half2_sat(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// the two cache elements held by a 32-bit word (element 2i in the low half)
__device__ __forceinline__ float kv_lo(uint32_t u) { return __low2float(*reinterpret_cast<const __half2*>(&u)); }
__device__ __forceinline__ float kv_hi(uint32_t u) { return __high2float(*reinterpret_cast<const __half2*>(&u)); }
// cache element type for a run dtype: fp32 pools in fp32 mode, kv16 pools in bf16 mode
template <class T> struct KvOf { typedef T type; };
template <> struct KvOf<bf16> { typedef kv16 type; };

__device__ __forceinline__ void dev_flag(int* status, int code) { atomicCAS(status, DEV_OK, code); }

// Programmatic dependent launch.  A kernel started with launch_overlapped() may begin while the
// kernel before it in the stream is still running (once every CTA of that kernel has called
// pdl_trigger() or exited); it must call pdl_wait() before its first access to global memory,
// which returns when the earlier kernel has finished and its writes are visible.  Both calls do
// nothing in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// RoPE angle pos * inv_freq reduced to [0, 2 pi) in fp64 before the fp32 sincos: at
// position 16 000 an fp32 product would already be off by about 1e-3 rad.
struct InvFreq { double f[64]; };   // theta^(-2c/hd), c < hd/2 <= 64
__device__ __forceinline__ void rope_sincos(int pos, double inv_freq, float* s, float* c) {
  double a = (double)pos * inv_freq;
  const double two_pi = 6.283185307179586476925286766559;
  a -= two_pi * floor(a / two_pi);
  sincosf((float)a, s, c);
}
void fill_inv_freq(InvFreq* f, int hd, float theta);

// Query / key norm: r[h] = 1 / sqrt(mean_c x[h * hd + c]^2 + eps) for h < n_heads (x in global memory,
// read through L2).  One warp per head; every thread of the block must call it; ends with a block barrier.
__device__ __forceinline__ void head_rnorm(const float* x, int n_heads, int hd, float eps, float* r_shared) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int h = warp; h < n_heads; h += nw) {
    float ss = 0.f;
    for (int c = lane; c < hd; c += 32) { const float v = __ldcg(x + (size_t)h * hd + c); ss = fmaf(v, v, ss); }
    ss = warp_sum(ss);
    if (lane == 0) r_shared[h] = rsqrtf(ss / (float)hd + eps);
  }
  __syncthreads();
}

// Where the predictor GEMM scatters its columns: the concatenated outputs of all base
// layers fed by one auxiliary layer; segment s covers columns [col0[s], col0[s+1]).
struct PagedOut {
  int n_seg;
  int col0[MAX_PRED_SEG + 1];
  int n_kv[MAX_PRED_SEG];
  void* pool[MAX_PRED_SEG];
  const float* bias;     // concatenated, may be null
  const int* tok_slot;   // [M] page * PAGE_TOKENS + row, or -1
  int head_dim;
};

// Row placement used when packing weights: plain offset, or gate/up block interleave.
struct RowMap {
  int row_offset;   // G == 0: dst_row = r + row_offset
  int G;            // G > 0: rows interleaved in blocks of G (gate block, then up block)
  int which;        // 0 = gate, 1 = up
  int n_rows_total; // ffn (rows of gate, and of up)
};
__host__ __device__ __forceinline__ int map_row(const RowMap& m, int r) {
  if (m.G == 0) return r + m.row_offset;
  int blk = r / m.G;
  int rem = m.n_rows_total - blk * m.G;
  int gb = rem < m.G ? rem : m.G;
  return 2 * blk * m.G + m.which * gb + (r - blk * m.G);
}

enum GemmEpi : int { EPI_STORE = 0, EPI_RESID = 1, EPI_PAGED = 2, EPI_STORE32 = 3 };

// bf16 mode carries the K/V path in split precision: a value v travels as hi = bf16(v) and
// lo = bf16(v - hi), and a GEMM whose A operand has a lo part accumulates A_hi W^T + A_lo W^T.
// The predicted cache is the product of the path and the base step's logits amplify its
// error, so the operand roundings in front of it are removed where that is cheap.
struct GemmArgs {
  const void* A; int lda;        // [M, K] run dtype
  const void* A2; int lda2;      // optional lo part of A (same shape), or null
  int split_begin;               // output columns >= split_begin use A + A2 (tile granularity)
  const void* W; int ldw;        // [N, K] run dtype
  int M, N, K;
  void* C; int ldc;              // EPI_STORE: run dtype [M, N]; EPI_STORE32: fp32 [M, N]
  float* X; int ldx;             // EPI_RESID: fp32 residual, X += A W^T
  PagedOut paged;                // EPI_PAGED
};

// ---- launchers (defined in the .cu files); all enqueue on `st` and count launches ----
struct LaunchCtx {
  cudaStream_t st;
  int64_t* n_launch;
  int* status;      // device status word
  int dtype;        // 0 f32, 1 bf16
};

void launch_pack_rows(const LaunchCtx&, const void* src, int src_dtype, void* dst, int dst_dtype,
                      int rows, int cols, RowMap map);
void launch_build_index(const LaunchCtx&, const int* cu_host /*[B+1]*/, int batch, int total,
                        int* cu_dev, int* tok_pos, int* tok_slot, int* last_tok_idx,
                        const int* block_table, int max_pages_per_seq, int n_pages, int* seq_lens);
void launch_embed(const LaunchCtx&, const int* tokens, const int* gather_idx, int n_rows,
                  const void* table, int vocab, int d, float* x);
void launch_rmsnorm(const LaunchCtx&, const float* x, const float* gain, float eps, int rows, int d,
                    void* out, int out_dtype, void* out_lo = nullptr, bool out_half = false);
// fp32 projection output [rows, n_heads*hd] -> RoPE on the first n_heads_rot heads -> run dtype
// `out` (row stride ld_out) and, for heads >= lo_head_begin, the bf16 lo part in `out_lo`.
// With q_gain / k_gain (fp32 [head_dim], or null): heads < n_q_heads are RMS-normalised with q_gain and the
// other rotated heads with k_gain (eps) before RoPE.
void launch_rope_split(const LaunchCtx&, const float* in, int ld_in, int rows, int n_heads, int n_heads_rot,
                       int head_dim, const int* tok_pos, float theta, void* out, int ld_out,
                       void* out_lo, int ld_lo, int lo_head_begin, int n_q_heads = 0, const float* q_gain = nullptr,
                       const float* k_gain = nullptr, float eps = 0.f);
void launch_swiglu(const LaunchCtx&, const void* gu, int rows, int ffn, int G, void* act);
void launch_gemm_simt(const LaunchCtx&, const GemmArgs&, int epi);
void launch_attn_prefill_simt(const LaunchCtx&, const void* qkv, int ld, int nq, int nkv, int hd,
                              const int* cu_dev, int batch, int total, void* out, int ldo);

// training-time forward: consistency terms and the predicted cache as a layer's keys and values.
// qkv: one layer's projection buffer [T, ld], own keys at column k_col, values at k_col + nkv * hd; kv_lo (bf16 mode,
// may be null): lo parts [T, ld_lo] of keys then values.  sum_k / sum_v (device) += mean |predicted - own|.
void launch_kv_l1(const LaunchCtx&, const void* qkv, int ld, int k_col, const void* kv_lo, int ld_lo, int T_tokens, int nkv,
                  int hd, const int* tok_slot, const void* kpool, const void* vpool, float* sum_k, float* sum_v,
                  bool qkv_is_half = false /* bf16 mode: keys and values of qkv are IEEE halves, no lo parts */);
void launch_kv_take(const LaunchCtx&, void* qkv, int ld, int k_col, int T_tokens, int nkv, int hd, const int* tok_slot,
                    const void* kpool, const void* vpool, bool qkv_is_half = false);

// base single-token step
enum StepGemvMode : int { GEMV_STORE = 0, GEMV_RESID = 1, GEMV_SWIGLU = 2 };
void launch_step_gemv(const LaunchCtx&, const void* W, int ldw, int N, int K, const float* x, int ldx,
                      int batch, float* y, int ldy, int mode, int G, int ffn, const float* gain = nullptr,
                      float eps = 0.f, float* scratch_h = nullptr);
void launch_step_attn(const LaunchCtx&, const float* q, int ldq, int nq, int nkv, int hd, float theta,
                      const void* kpool, const void* vpool, const int* block_table,
                      int max_pages_per_seq, int n_pages, const int* seq_lens, int extra, int batch,
                      int max_keys, float* part, float* out, const float* q_gain = nullptr, float eps = 0.f,
                      int* split_done = nullptr /* [batch * nkv] ints: lets the attention kernel merge its own key-range splits */);
void launch_step_append(const LaunchCtx&, const float* qkv, int nq, int nkv, int hd, float theta,
                        void* kpool, void* vpool, const int* block_table, int max_pages_per_seq,
                        int n_pages, const int* seq_lens, int batch, const float* k_gain = nullptr, float eps = 0.f);
void launch_argmax(const LaunchCtx&, const float* logits, int batch, int vocab, int* out);
void launch_add_int(const LaunchCtx&, int* v, int n, int delta);
int step_attn_splits(int batch, int nkv, int max_keys);
// warp-level tensor-core variant for the half-precision cache (pages fetched through a swizzling tensor map)
int step_attn_mma_splits(int batch, int nkv, int max_keys, int upper);
bool step_attn_mma_supported(int dtype, int nq, int nkv, int hd, const void* kpool, const void* vpool, int n_pages);
cudaError_t launch_step_attn_mma(const LaunchCtx&, const float* q, int ldq, int nq, int nkv, int hd, float theta, const void* kpool,
                                 const void* vpool, const int* block_table, int max_pages_per_seq, int n_pages, const int* seq_lens,
                                 int extra, int batch, int n_split, int max_keys, float* part, float* out, const float* q_gain,
                                 float eps, int* split_done);
// bandwidth-bound variant for the bf16 cache (pages fetched with bulk asynchronous copies)
int step_attn_ring_splits(int nq, int nkv, int hd, int batch, int max_keys, int upper);
bool step_attn_ring_supported(int dtype, int nq, int nkv, int hd, const void* kpool, const void* vpool);
cudaError_t launch_step_attn_ring(const LaunchCtx&, const float* q, int ldq, int nq, int nkv, int hd, float theta,
                                  const void* kpool, const void* vpool, const int* block_table, int max_pages_per_seq,
                                  int n_pages, const int* seq_lens, int extra, int batch, int n_split, float* part, float* out,
                                  const float* q_gain = nullptr, float eps = 0.f, int* split_done = nullptr);
