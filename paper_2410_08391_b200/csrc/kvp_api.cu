// C ABI of the KV Prediction library: validation, plan, weight packing and the kernel
// schedule of the time-to-first-token path and of the generation step.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "attn_tc.h"
#include "gemm_tc.h"
#include "kvp_internal.h"
#include "kvpred_tc.h"
#include "step_mega.h"
#include "step_tc.h"

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

kvp_status fail(kvp_handle* h, kvp_status code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->err = buf;
  return code;
}

const char* validate_model(const kvp_model_cfg* m) {
  if (!m || !m->layers) return "model config or its layer array is NULL";
  if (m->n_layers <= 0 || m->n_layers > 1024) return "n_layers out of range";
  if (m->d_model <= 0 || m->vocab <= 0) return "d_model and vocab must be positive";
  if (m->qk_norm != 0 && m->qk_norm != 1) return "qk_norm must be 0 or 1";
  if (!(m->rope_theta > 0.f) || !(m->rms_eps >= 0.f)) return "rope_theta must be > 0 and rms_eps >= 0";
  for (int l = 0; l < m->n_layers; ++l) {
    const kvp_layer_cfg& c = m->layers[l];
    if (c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 || c.ffn_dim <= 0) return "layer dimensions must be positive";
    if (c.n_q_heads % c.n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
    if (c.head_dim != m->layers[0].head_dim) return "head_dim must be the same in every layer of a model";
  }
  return nullptr;
}

const char* unsupported_model(const kvp_model_cfg* m) {
  for (int l = 0; l < m->n_layers; ++l) {
    const kvp_layer_cfg& c = m->layers[l];
    if (c.head_dim % 2 || c.head_dim > 128) return "head_dim must be even and <= 128";
    if (c.n_q_heads / c.n_kv_heads > 8) return "more than 8 query heads per kv head";
    if (m->qk_norm && c.n_kv_heads > 64) return "key norm with more than 64 kv heads";
  }
  return nullptr;
}

void plan_model(ModelPlan& p, const kvp_model_cfg* m, int es, bool bf16_mode, size_t& off, bool with_head) {
  p.n_layers = m->n_layers; p.d = m->d_model; p.vocab = m->vocab; p.theta = m->rope_theta; p.eps = m->rms_eps;
  p.qk_norm = m->qk_norm != 0;
  p.max_nqkv = p.max_dq = p.max_dkv = p.max_ffn = p.max_group = p.max_nkv = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  p.embed = take((size_t)m->vocab * m->d_model * es);
  p.L.resize(m->n_layers);
  for (int l = 0; l < m->n_layers; ++l) {
    LayerPlan& L = p.L[l];
    const kvp_layer_cfg& c = m->layers[l];
    L.nq = c.n_q_heads; L.nkv = c.n_kv_heads; L.hd = c.head_dim; L.ffn = c.ffn_dim;
    L.dq = L.nq * L.hd; L.dkv = L.nkv * L.hd; L.nqkv = L.dq + 2 * L.dkv;
    L.G = (bf16_mode && L.ffn % 64 == 0) ? 64 : 0;
    L.wqkv = take((size_t)L.nqkv * p.d * es);
    L.wo = take((size_t)p.d * L.dq * es);
    L.wgu = take((size_t)2 * L.ffn * p.d * es);
    L.wd = take((size_t)p.d * L.ffn * es);
    L.attn_norm = take((size_t)p.d * 4);
    L.ffn_norm = take((size_t)p.d * 4);
    L.q_norm = L.k_norm = 0;
    if (p.qk_norm) { L.q_norm = take((size_t)L.hd * 4); L.k_norm = take((size_t)L.hd * 4); }
    p.max_nqkv = std::max(p.max_nqkv, L.nqkv); p.max_dq = std::max(p.max_dq, L.dq);
    p.max_ffn = std::max(p.max_ffn, L.ffn); p.max_group = std::max(p.max_group, L.nq / L.nkv);
    p.max_nkv = std::max(p.max_nkv, L.nkv); p.max_dkv = std::max(p.max_dkv, L.dkv);
  }
  p.final_norm = p.lm_head = 0;
  if (with_head) {
    p.final_norm = take((size_t)p.d * 4);
    p.lm_head = take((size_t)m->vocab * m->d_model * es);
  }
}

void add_model_slots(kvp_handle* h, const char* prefix, const ModelPlan& p, int n_live_layers, bool with_head, const std::vector<uint8_t>* qkv_half = nullptr) {
  int dt = h->opt.dtype;
  auto name = [&](int l, const char* leaf) { char b[96]; snprintf(b, sizeof b, "%s.L%d.%s", prefix, l, leaf); return std::string(b); };
  h->slots[std::string(prefix) + ".embed"] = PackSlot{p.embed, p.vocab, p.d, dt, RowMap{0, 0, 0, 0}};
  for (int l = 0; l < n_live_layers; ++l) {
    const LayerPlan& L = p.L[l];
    h->slots[name(l, "attn_norm")] = PackSlot{L.attn_norm, 1, p.d, 0, RowMap{0, 0, 0, 0}};
    h->slots[name(l, "ffn_norm")] = PackSlot{L.ffn_norm, 1, p.d, 0, RowMap{0, 0, 0, 0}};
    if (p.qk_norm) {
      h->slots[name(l, "q_norm")] = PackSlot{L.q_norm, 1, L.hd, 0, RowMap{0, 0, 0, 0}};
      h->slots[name(l, "k_norm")] = PackSlot{L.k_norm, 1, L.hd, 0, RowMap{0, 0, 0, 0}};
    }
    const int dq3 = (qkv_half && (*qkv_half)[l]) ? 2 : dt;     // stored as IEEE halves where the projection runs on f16 operands
    h->slots[name(l, "wq")] = PackSlot{L.wqkv, L.dq, p.d, dq3, RowMap{0, 0, 0, 0}};
    h->slots[name(l, "wk")] = PackSlot{L.wqkv, L.dkv, p.d, dq3, RowMap{L.dq, 0, 0, 0}};
    h->slots[name(l, "wv")] = PackSlot{L.wqkv, L.dkv, p.d, dq3, RowMap{L.dq + L.dkv, 0, 0, 0}};
    h->slots[name(l, "wo")] = PackSlot{L.wo, p.d, L.dq, dt, RowMap{0, 0, 0, 0}};
    h->slots[name(l, "w_gate")] = PackSlot{L.wgu, L.ffn, p.d, dt, RowMap{0, L.G, 0, L.ffn}};
    h->slots[name(l, "w_up")] = PackSlot{L.wgu, L.ffn, p.d, dt, RowMap{L.G == 0 ? L.ffn : 0, L.G, 1, L.ffn}};
    h->slots[name(l, "w_down")] = PackSlot{L.wd, p.d, L.ffn, dt, RowMap{0, 0, 0, 0}};
  }
  if (with_head) {
    h->slots[std::string(prefix) + ".final_norm"] = PackSlot{p.final_norm, 1, p.d, 0, RowMap{0, 0, 0, 0}};
    h->slots[std::string(prefix) + ".lm_head"] = PackSlot{p.lm_head, p.vocab, p.d, dt, RowMap{0, 0, 0, 0}};
  }
}

WsLayout ws_layout(const kvp_handle* h, int64_t Bm, int64_t Tm) {
  WsLayout w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const ModelPlan &A = h->aux, &B = h->base;
  size_t es = h->es;
  w.status = take(16384);     // status word, barrier counter, argmax slots; from byte 256: optional phase trace
  w.cu = take((Bm + 1) * 4);
  w.last_idx = take(Bm * 4);
  w.tok_pos = take(Tm * 4);
  w.tok_slot = take(Tm * 4);
  w.rope_tab = take(Tm * (size_t)((A.L[0].hd / 2 + 1) & ~1) * 8);     // entries hold two frequencies: an even number of them
  w.x = take(Tm * A.d * 4);
  w.h = take(Tm * A.d * es);
  w.h_lo = take(Tm * A.d * es);
  w.qkv = take(Tm * A.max_nqkv * es);
  w.qkv32 = take(Tm * A.max_nqkv * 4);
  w.kv_lo = take(Tm * 2 * (size_t)A.max_dkv * es);
  w.attn = take(Tm * A.max_dq * es);
  w.gu = take(Tm * 2 * (size_t)A.max_ffn * es);
  w.act = take(Tm * (size_t)A.max_ffn * es);
  w.xb = take(Bm * B.d * 4);
  w.hb = take(Bm * B.d * 4);
  w.qkvb = take(Bm * B.max_nqkv * 4);
  w.ab = take(Bm * B.max_dq * 4);
  w.actb = take(Bm * (size_t)B.max_ffn * 4);
  w.part = take((size_t)(2 * 148 + Bm * B.max_nkv) * B.max_group * (B.L[0].hd + 2) * 4);
  w.tok_stage = take(Tm * 4);
  w.first_stage = take(Bm * 4);
  // tensor-core step projections: operand rows (hi + lo) of the widest input, fp32 gate/up outputs
  const int64_t Bp = step_tc_rows((int)Bm);
  const int64_t k_max = std::max((int64_t)B.d, std::max((int64_t)B.max_dq, (int64_t)B.max_ffn));
  w.xbt = take(2 * Bp * k_max * 2);
  w.gub = take(Bm * 2 * (size_t)B.max_ffn * 4);
  w.attn_sched = take((size_t)(Tm / 128 + Bm + 1) * 8);
  w.attn_done = take((size_t)Bm * B.max_nkv * 4);
  // fused RMSNorm: per auxiliary layer two vectors of row sums of squares (one memset clears all)
  w.norm_ss = take((size_t)2 * A.n_layers * Tm * 4);
  w.total = off;
  return w;
}

kvp_status check_cuda(kvp_handle* h, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, KVP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return KVP_OK;
}

struct CallShape { std::vector<int> cu; int total; int max_len; };

kvp_status common_checks(kvp_handle* h, const int32_t* lengths, int32_t batch, const kvp_cache* cache, void* ws,
                         int extra_tokens, CallShape* cs) {
  if (!h) return KVP_ERR_INVALID_ARG;
  h->err.clear();
  if (!lengths || !cache || !ws) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  if (batch <= 0 || batch > KVP_MAX_BATCH) return fail(h, KVP_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, KVP_MAX_BATCH);
  if (!cache->k_pools || !cache->v_pools || !cache->block_table || !cache->seq_lens)
    return fail(h, KVP_ERR_INVALID_ARG, "cache has a NULL member");
  if (cache->max_pages_per_seq <= 0 || cache->n_pages <= 0) return fail(h, KVP_ERR_INVALID_ARG, "cache has no pages");
  for (int i = 0; i < h->base.n_layers; ++i)
    if (!cache->k_pools[i] || !cache->v_pools[i]) return fail(h, KVP_ERR_INVALID_ARG, "cache pool of base layer %d is NULL", i);
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return check_cuda(h, "cudaGetDevice");
  if (dev != h->device) return fail(h, KVP_ERR_INVALID_ARG, "current device %d is not the handle's device %d", dev, h->device);
  cs->cu.assign(batch + 1, 0);
  cs->max_len = 0;
  int64_t total = 0, pages = 0;
  for (int b = 0; b < batch; ++b) {
    if (lengths[b] <= 0) return fail(h, KVP_ERR_INVALID_ARG, "lengths[%d] = %d must be >= 1", b, lengths[b]);
    int64_t need = ((int64_t)lengths[b] + extra_tokens + PAGE_TOKENS - 1) / PAGE_TOKENS;
    if (need > cache->max_pages_per_seq)
      return fail(h, KVP_ERR_CACHE_FULL, "sequence %d needs %lld pages, block table has %d per sequence", b, (long long)need, cache->max_pages_per_seq);
    pages += need;
    total += lengths[b];
    if (total > 0x7fffffff / 2) return fail(h, KVP_ERR_INVALID_ARG, "too many tokens");
    cs->cu[b + 1] = (int)total;
    cs->max_len = std::max(cs->max_len, (int)lengths[b]);
  }
  if (pages > cache->n_pages) return fail(h, KVP_ERR_CACHE_FULL, "batch needs %lld pages, pools hold %d", (long long)pages, cache->n_pages);
  cs->total = (int)total;
  if ((uintptr_t)ws % 256) return fail(h, KVP_ERR_WORKSPACE, "workspace is not 256-byte aligned");
  return KVP_OK;
}

bool ends_with(const std::string& s, const char* suf) {
  size_t n = strlen(suf);
  return s.size() >= n && s.compare(s.size() - n, n, suf) == 0;
}

// Tries the tcgen05 GEMM; returns false when the shape is not one it takes (caller falls back).
bool try_tc(kvp_handle* h, const LaunchCtx& ctx, TcGemm& t, int cls, cudaError_t* err) {
  if (h->opt.dtype != KVP_BF16) return false;
  t.n_sm = h->gemm_sms;
  if (!tc_gemm_supported(t)) return false;
  TimedScope ts(h, ctx.st, cls);
  cudaError_t e = launch_gemm_tc(t, ctx.status, ctx.st, ctx.n_launch);
  if (e != cudaSuccess && *err == cudaSuccess) *err = e;
  return true;
}

// Are the step's projections run on the tensor cores?  (Everything the persistent kernel does not take:
// batches of more than 4 rows, and small batches over long caches.)
bool step_uses_tc(const kvp_handle* h, int batch) {
  if (h->opt.dtype != KVP_BF16 || step_tc_rows(batch) > 128) return false;
  const ModelPlan& B = h->base;
  if (B.d % 8) return false;
  for (int i = 0; i < B.n_layers; ++i)
    if (B.L[i].dq % 8 || B.L[i].ffn % 8) return false;
  return true;
}

// y += W x on the tensor cores: operand rows from `src` (RMS-normalised with `gain`, or SwiGLU of a
// gate/up row, or as they are), output cleared first unless it is the residual stream.
void step_proj_tc(kvp_handle* h, const LaunchCtx& ctx, const WsLayout& w, char* ws, int mode, const float* src, int ld_src,
                  int K, int batch, const float* gain, int G, const void* W, int N, float* Y, int ldy, bool clear,
                  cudaError_t* err, const void* next_w = nullptr, size_t next_bytes = 0) {
  bf16* XB = (bf16*)(ws + w.xbt);
  KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_prep(ctx, mode, src, ld_src, K, batch, gain, h->base.eps, G, XB, clear ? Y : nullptr, ldy, N));
  TimedScope ts(h, ctx.st, KVP_CLASS_STEP_GEMV);
  cudaError_t e = launch_step_gemm_tc((const bf16*)W, K, N, K, XB, batch, Y, ldy, h->step_grid_sms, ctx.status, ctx.st, ctx.n_launch, next_w, next_bytes);
  if (e != cudaSuccess && *err == cudaSuccess) *err = e;
}

// one base-model layer of a single-token step (shared by the first step and generation)
void base_layer_step(kvp_handle* h, const LaunchCtx& ctx, int i, const kvp_cache* cache, const WsLayout& w, char* ws,
                     int batch, int max_keys, bool generation, cudaError_t* err) {
  const ModelPlan& B = h->base;
  const LayerPlan& L = B.L[i];
  const char* P = h->packed;
  float* xb = (float*)(ws + w.xb);
  float* hb = (float*)(ws + w.hb);
  float* qkvb = (float*)(ws + w.qkvb);
  float* ab = (float*)(ws + w.ab);
  float* actb = (float*)(ws + w.actb);
  // the first step needs q only (keys and values are the predicted ones); generation needs q, k, v
  int n_out = generation ? L.nqkv : L.dq;
  const bool tc = step_uses_tc(h, batch);
  // every projection names the weights of the one after it (the next layer's queries, or the LM head, after the down projection)
  const size_t es = (size_t)h->es;
  const bool last_layer = i + 1 == B.n_layers;
  const void* w_after = last_layer ? P + B.lm_head : P + B.L[last_layer ? i : i + 1].wqkv;
  const size_t b_after = last_layer ? (size_t)B.vocab * B.d * es : (size_t)(generation ? B.L[i + 1].nqkv : B.L[i + 1].dq) * B.d * es;
  if (tc)
    step_proj_tc(h, ctx, w, ws, PREP_NORM, xb, B.d, B.d, batch, (const float*)(P + L.attn_norm), 0, P + L.wqkv, n_out, qkvb, n_out, true, err,
                 P + L.wo, (size_t)B.d * L.dq * es);
  else
    KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_gemv(ctx, P + L.wqkv, B.d, n_out, B.d, xb, B.d, batch, qkvb, n_out, GEMV_STORE, 0, 0,
                                                    (const float*)(P + L.attn_norm), B.eps, hb));
  const float* qn = B.qk_norm ? (const float*)(P + L.q_norm) : nullptr;
  const float* kn = B.qk_norm ? (const float*)(P + L.k_norm) : nullptr;
  if (generation)
    KVP_TIMED(KVP_CLASS_OTHER, launch_step_append(ctx, qkvb, L.nq, L.nkv, L.hd, B.theta, cache->k_pools[i], cache->v_pools[i], cache->block_table,
                       cache->max_pages_per_seq, cache->n_pages, cache->seq_lens, batch, kn, B.eps));
  KVP_TIMED(KVP_CLASS_STEP_ATTN, launch_step_attn(ctx, qkvb, n_out, L.nq, L.nkv, L.hd, B.theta, cache->k_pools[i], cache->v_pools[i], cache->block_table,
                   cache->max_pages_per_seq, cache->n_pages, cache->seq_lens, generation ? 1 : 0, batch, max_keys,
                   (float*)(ws + w.part), ab, qn, B.eps, (int*)(ws + w.attn_done)));
  if (tc) {
    float* gub = (float*)(ws + w.gub);
    step_proj_tc(h, ctx, w, ws, PREP_PLAIN, ab, L.dq, L.dq, batch, nullptr, 0, P + L.wo, B.d, xb, B.d, false, err, P + L.wgu, (size_t)2 * L.ffn * B.d * es);
    step_proj_tc(h, ctx, w, ws, PREP_NORM, xb, B.d, B.d, batch, (const float*)(P + L.ffn_norm), 0, P + L.wgu, 2 * L.ffn, gub, 2 * L.ffn, true, err,
                 P + L.wd, (size_t)B.d * L.ffn * es);
    step_proj_tc(h, ctx, w, ws, PREP_SWIGLU, gub, 2 * L.ffn, L.ffn, batch, nullptr, L.G, P + L.wd, B.d, xb, B.d, false, err, w_after, b_after);
    return;
  }
  KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_gemv(ctx, P + L.wo, L.dq, B.d, L.dq, ab, L.dq, batch, xb, B.d, GEMV_RESID, 0, 0));
  KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_gemv(ctx, P + L.wgu, B.d, L.ffn, B.d, xb, B.d, batch, actb, L.ffn, GEMV_SWIGLU, L.G, L.ffn,
                                                  (const float*)(P + L.ffn_norm), B.eps, hb));
  KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_gemv(ctx, P + L.wd, L.ffn, B.d, L.ffn, actb, L.ffn, batch, xb, B.d, GEMV_RESID, 0, 0));
}

// Parameters of the persistent step kernel for this call; false = the kernel does not apply.
bool mega_prepare(kvp_handle* h, const LaunchCtx& ctx, const kvp_cache* cache, const WsLayout& w, char* ws, int batch,
                  int max_keys, bool generation, const int* tokens, const int* gather_idx, float* logits,
                  int32_t* token_out, MegaParams* out, int* k_max_out) {
  const ModelPlan& B = h->base;
  int k_max = std::max(B.d, std::max(B.max_dq, B.max_ffn));
  // its attention phase reads cache pages with plain loads: fine for a few thousand keys, several times
  // slower than the ring-fed kernel beyond that
  if (max_keys > 4096) return false;
  if (B.n_layers > MEGA_MAX_LAYERS || !step_mega_supported(batch, B.L[0].hd, k_max, B.max_group, h->es)) return false;
  // bulk copies need 16-byte rows: every projection's row length must be a multiple of 16 bytes
  for (int i = 0; i < B.n_layers; ++i)
    if ((B.d * h->es) % 16 || (B.L[i].dq * h->es) % 16 || (B.L[i].ffn * h->es) % 16) return false;
  const char* P = h->packed;
  MegaParams& p = *out;
  p = MegaParams{};
  p.n_layers = B.n_layers; p.d = B.d; p.vocab = B.vocab; p.hd = B.L[0].hd; p.batch = batch; p.generation = generation ? 1 : 0;
  p.eps = B.eps;
  fill_inv_freq(&p.inv, p.hd, B.theta);
  p.tokens = tokens; p.gather_idx = gather_idx;
  p.embed = P + B.embed; p.final_norm = (const float*)(P + B.final_norm); p.lm_head = P + B.lm_head;
  p.block_table = cache->block_table; p.mpps = cache->max_pages_per_seq; p.n_pages = cache->n_pages; p.seq_lens = cache->seq_lens;
  p.xb = (float*)(ws + w.xb); p.qkvb = (float*)(ws + w.qkvb); p.ab = (float*)(ws + w.ab); p.actb = (float*)(ws + w.actb);
  p.part = (float*)(ws + w.part);
  p.attn_done = (int*)(ws + w.attn_done);
  p.logits = logits; p.token_out = token_out; p.status = ctx.status;
#ifdef KVP_MEGA_TRACE     // build-time diagnostic: per-phase clocks of the persistent step kernel, from byte 256 of the status block
  p.trace = (long long*)((char*)ctx.status + 256);
#else
  p.trace = nullptr;
#endif
  int min_nkv = B.L[0].nkv;
  for (int i = 0; i < B.n_layers; ++i) {
    const LayerPlan& L = B.L[i];
    MegaLayer& m = p.layers[i];
    m.wqkv = P + L.wqkv; m.wo = P + L.wo; m.wgu = P + L.wgu; m.wd = P + L.wd;
    m.attn_norm = (const float*)(P + L.attn_norm); m.ffn_norm = (const float*)(P + L.ffn_norm);
    m.q_norm = B.qk_norm ? (const float*)(P + L.q_norm) : nullptr;
    m.k_norm = B.qk_norm ? (const float*)(P + L.k_norm) : nullptr;
    m.kpool = cache->k_pools[i]; m.vpool = cache->v_pools[i];
    m.nq = L.nq; m.nkv = L.nkv; m.dq = L.dq; m.nqkv = L.nqkv; m.ffn = L.ffn; m.G = L.G;
    min_nkv = std::min(min_nkv, L.nkv);
  }
  p.n_split = step_attn_splits(batch, min_nkv, max_keys);   // sized for the layer with the fewest kv heads
  p.layer_begin = 0; p.layer_end = B.n_layers; p.do_embed = 1; p.do_head = 1; p.counter_idx = 0;
  *k_max_out = k_max;
  return true;
}

// The whole base step (all layers, LM head, argmax) as one persistent kernel; false = not applicable.
// The caller has cleared the first MEGA_STATUS_BYTES of the status block (or at least its counters).
bool base_step_fused(kvp_handle* h, const LaunchCtx& ctx, const kvp_cache* cache, const WsLayout& w, char* ws, int batch,
                     int max_keys, bool generation, const int* tokens, const int* gather_idx, float* logits,
                     int32_t* token_out, cudaError_t* err) {
  MegaParams p;
  int k_max = 0;
  if (!mega_prepare(h, ctx, cache, w, ws, batch, max_keys, generation, tokens, gather_idx, logits, token_out, &p, &k_max)) return false;
  cudaMemsetAsync(p.attn_done, 0, (size_t)batch * h->base.max_nkv * 4, ctx.st);
  TimedScope ts(h, ctx.st, KVP_CLASS_STEP_FUSED);
  cudaError_t e = launch_step_mega(p, h->opt.dtype, k_max, h->n_sm, ctx.st, ctx.n_launch);
  if (e != cudaSuccess && *err == cudaSuccess) *err = e;
  return true;
}

void base_head(kvp_handle* h, const LaunchCtx& ctx, const WsLayout& w, char* ws, int batch, float* logits,
               int32_t* token_out, cudaError_t* err) {
  const ModelPlan& B = h->base;
  const char* P = h->packed;
  float* xb = (float*)(ws + w.xb);
  float* hb = (float*)(ws + w.hb);
  if (step_uses_tc(h, batch))
    step_proj_tc(h, ctx, w, ws, PREP_NORM, xb, B.d, B.d, batch, (const float*)(P + B.final_norm), 0, P + B.lm_head, B.vocab, logits, B.vocab, true, err);
  else
  KVP_TIMED(KVP_CLASS_STEP_GEMV, launch_step_gemv(ctx, P + B.lm_head, B.d, B.vocab, B.d, xb, B.d, batch, logits, B.vocab, GEMV_STORE, 0, 0,
                                                  (const float*)(P + B.final_norm), B.eps, hb));
  if (token_out) KVP_TIMED(KVP_CLASS_OTHER, launch_argmax(ctx, logits, batch, B.vocab, token_out));
}

}  // namespace

// =========================================================================================
extern "C" {

kvp_status kvp_layer_map_canonical(int32_t n_base, int32_t n_aux, int32_t* out) {
  if (!out || n_base <= 0 || n_aux <= 0 || n_aux > n_base) return KVP_ERR_INVALID_ARG;
  int per = n_base / n_aux, more = n_base % n_aux, i = 0;
  for (int j = 0; j < n_aux; ++j)
    for (int c = 0; c < per + (j < more ? 1 : 0); ++c) out[i++] = j;
  return KVP_OK;
}

kvp_status kvp_layer_map_pruned(int32_t n_base, const int32_t* retained, int32_t n_aux, int32_t* out) {
  if (!out || !retained || n_base <= 0 || n_aux <= 0 || retained[0] != 0) return KVP_ERR_INVALID_ARG;
  for (int j = 1; j < n_aux; ++j)
    if (retained[j] <= retained[j - 1] || retained[j] >= n_base) return KVP_ERR_INVALID_ARG;
  int j = 0;
  for (int i = 0; i < n_base; ++i) {
    while (j + 1 < n_aux && retained[j + 1] <= i) ++j;
    out[i] = j;
  }
  return KVP_OK;
}

kvp_status kvp_layer_map_uniform(int32_t n_base, int32_t n_aux, int32_t* out) {
  if (!out || n_base <= 0 || n_aux <= 0) return KVP_ERR_INVALID_ARG;
  for (int i = 0; i < n_base; ++i) out[i] = (int32_t)(((int64_t)i * n_aux) / n_base);
  return KVP_OK;
}

kvp_status kvp_create(const kvp_model_cfg* aux, const kvp_model_cfg* base, const int32_t* layer_map,
                      const kvp_options* opt, kvp_handle** out) {
  if (!out) return KVP_ERR_INVALID_ARG;
  *out = nullptr;
  if (!aux || !base || !layer_map || !opt) return KVP_ERR_INVALID_ARG;
  if (validate_model(aux) || validate_model(base)) return KVP_ERR_SHAPE;
  if (opt->dtype != KVP_F32 && opt->dtype != KVP_BF16) return KVP_ERR_INVALID_ARG;
  if (opt->page_tokens != PAGE_TOKENS || (opt->flags & ~(KVP_OPT_FUSED_KV_PRED | KVP_OPT_SEPARATE_NORM)) != 0) return KVP_ERR_INVALID_ARG;
  if (opt->predictor_bias != 0 && opt->predictor_bias != 1) return KVP_ERR_INVALID_ARG;
  if (aux->vocab != base->vocab) return KVP_ERR_SHAPE;   // one token stream feeds both models
  if (unsupported_model(aux) || unsupported_model(base)) return KVP_ERR_UNSUPPORTED;
  int j_max = 0;
  for (int i = 0; i < base->n_layers; ++i) {
    if (layer_map[i] < 0 || layer_map[i] >= aux->n_layers) return KVP_ERR_INVALID_ARG;
    if (i && layer_map[i] < layer_map[i - 1]) return KVP_ERR_INVALID_ARG;
    j_max = std::max(j_max, layer_map[i]);
  }
  kvp_handle* h = new (std::nothrow) kvp_handle();
  if (!h) return KVP_ERR_INVALID_ARG;
  h->opt = *opt;
  h->es = opt->dtype == KVP_BF16 ? 2 : 4;
  h->map.assign(layer_map, layer_map + base->n_layers);
  h->j_max = j_max;
  h->device = 0;
  if (cudaGetDevice(&h->device) == cudaSuccess) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, h->device) == cudaSuccess && n > 0) h->n_sm = n;
  }
  cudaGetLastError();
  {
    if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess) h->side = nullptr;
    if (h->side && (cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                    cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess)) {
      cudaStreamDestroy(h->side);
      h->side = nullptr;
    }
    cudaGetLastError();
  }
  h->gemm_sms = h->step_grid_sms = h->n_sm;
  if (h->step_tc_sms < 8 || h->step_tc_sms > h->n_sm) h->step_tc_sms = 0;
  if (h->step_sms < 8 || h->step_sms > h->n_sm - 32 || !h->side) h->step_sms = 0;
  if (h->step_sms) {
    if (cudaStreamCreateWithFlags(&h->step_st, cudaStreamNonBlocking) != cudaSuccess) h->step_st = nullptr;
    if (!h->step_st || cudaEventCreateWithFlags(&h->ev_step, cudaEventDisableTiming) != cudaSuccess) h->step_sms = 0;
    cudaGetLastError();
  }
  size_t off = 0;
  bool bf = opt->dtype == KVP_BF16;
  plan_model(h->aux, aux, h->es, bf, off, false);
  plan_model(h->base, base, h->es, bf, off, true);
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  h->groups.resize(j_max + 1);
  for (int j = 0; j <= j_max; ++j) {
    PredGroup& g = h->groups[j];
    g.n_seg = 0; g.col0[0] = 0; g.din = h->aux.L[j].dkv; g.fk = g.fv = g.bk = g.bv = 0;
    for (int i = 0; i < base->n_layers; ++i) {
      if (layer_map[i] != j) continue;
      if (g.n_seg == MAX_PRED_SEG) { delete h; return KVP_ERR_UNSUPPORTED; }
      g.base_layer[g.n_seg] = i;
      g.col0[g.n_seg + 1] = g.col0[g.n_seg] + h->base.L[i].dkv;
      ++g.n_seg;
    }
    int dout = g.col0[g.n_seg];
    // The predictor's input has to carry more than bf16's 8 significant bits (the logits amplify its rounding).
    // Where everything on its way runs on the tensor cores, K_A / V_A travel as IEEE halves and FK / FV are
    // stored as halves (exact for |w| >= 2^-14, absolute error <= 2^-25 below): one MMA pass.  Otherwise K_A / V_A
    // travel as a bf16 value plus its bf16 remainder and the matrices stay in the run dtype: two passes.
    g.half_path = bf && (h->aux.L[j].hd == 64 || h->aux.L[j].hd == 128) && h->aux.d % 8 == 0 && g.din % 8 == 0 &&
                  h->base.L[0].hd % 32 == 0;
    if (dout == 0) continue;
    g.fk = take((size_t)dout * g.din * h->es);
    g.fv = take((size_t)dout * g.din * h->es);
    if (opt->predictor_bias) { g.bk = take((size_t)dout * 4); g.bv = take((size_t)dout * 4); }
  }
  h->packed_bytes = off;
  // The QKV projection of an auxiliary layer takes f16 operands wherever the tensor-core kernel is sure to run it (the
  // kernel that does K/V projection and predictor in one reads bf16 weights, so not with that option).
  h->qkv_half.assign(j_max + 1, 0);
  for (int j = 0; j <= j_max; ++j)
    h->qkv_half[j] = bf && (h->aux.L[j].hd == 64 || h->aux.L[j].hd == 128) && h->aux.d % 8 == 0 && !(opt->flags & KVP_OPT_FUSED_KV_PRED);
  add_model_slots(h, "aux", h->aux, j_max + 1, false, &h->qkv_half);
  add_model_slots(h, "base", h->base, base->n_layers, true);
  for (int j = 0; j <= j_max; ++j) {
    const PredGroup& g = h->groups[j];
    for (int s = 0; s < g.n_seg; ++s) {
      int i = g.base_layer[s], dout = g.col0[s + 1] - g.col0[s];
      char b[64];
      snprintf(b, sizeof b, "pred.L%d.fk", i);
      const int f_dtype = g.half_path ? 2 : opt->dtype;
      h->slots[b] = PackSlot{g.fk + (size_t)g.col0[s] * g.din * h->es, dout, g.din, f_dtype, RowMap{0, 0, 0, 0}};
      snprintf(b, sizeof b, "pred.L%d.fv", i);
      h->slots[b] = PackSlot{g.fv + (size_t)g.col0[s] * g.din * h->es, dout, g.din, f_dtype, RowMap{0, 0, 0, 0}};
      if (opt->predictor_bias) {
        snprintf(b, sizeof b, "pred.L%d.bk", i);
        h->slots[b] = PackSlot{g.bk + (size_t)g.col0[s] * 4, 1, dout, 0, RowMap{0, 0, 0, 0}};
        snprintf(b, sizeof b, "pred.L%d.bv", i);
        h->slots[b] = PackSlot{g.bv + (size_t)g.col0[s] * 4, 1, dout, 0, RowMap{0, 0, 0, 0}};
      }
    }
  }
  char last[32];
  snprintf(last, sizeof last, "aux.L%d.", j_max);
  for (auto& kv : h->slots) {
    const std::string& n = kv.first;
    bool is_kv = ends_with(n, ".wk") || ends_with(n, ".wv");
    bool base_kv = n.rfind("base.L", 0) == 0 && (is_kv || ends_with(n, ".k_norm"));
    // in the last mapped auxiliary layer only the attention norm and the K/V projections are live
    bool aux_last_dead = n.rfind(last, 0) == 0 && !(ends_with(n, ".attn_norm") || ends_with(n, ".k_norm") || is_kv);
    if (aux_last_dead) continue;            // accepted if given, never required
    (base_kv ? h->req_decode_extra : h->req_prefill).push_back(n);
  }
  *out = h;
  return KVP_OK;
}

void kvp_destroy(kvp_handle* h) { delete h; }

const char* kvp_last_error(const kvp_handle* h) { return h ? h->err.c_str() : "NULL handle"; }

int64_t kvp_launch_count(const kvp_handle* h) { return h ? h->n_launch : 0; }

kvp_status kvp_packed_weight_bytes(const kvp_handle* h, size_t* bytes) {
  if (!h || !bytes) return KVP_ERR_INVALID_ARG;
  *bytes = h->packed_bytes;
  return KVP_OK;
}

kvp_status kvp_workspace_bytes(const kvp_handle* h, int32_t max_batch, int64_t max_total_tokens, size_t* bytes) {
  if (!h || !bytes || max_batch <= 0 || max_batch > KVP_MAX_BATCH || max_total_tokens < max_batch) return KVP_ERR_INVALID_ARG;
  *bytes = ws_layout(h, max_batch, max_total_tokens).total;
  return KVP_OK;
}

kvp_status kvp_cache_layout(const kvp_handle* h, int32_t base_layer, size_t* bytes_per_page) {
  if (!h || !bytes_per_page || base_layer < 0 || base_layer >= h->base.n_layers) return KVP_ERR_INVALID_ARG;
  *bytes_per_page = (size_t)h->base.L[base_layer].dkv * PAGE_TOKENS * h->es;
  return KVP_OK;
}

kvp_status kvp_load_weights(kvp_handle* h, const kvp_tensor* tensors, int32_t n, void* packed, size_t packed_bytes,
                            void* stream) {
  if (!h) return KVP_ERR_INVALID_ARG;
  h->err.clear();
  if (!tensors || n < 0 || !packed) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  if (packed_bytes < h->packed_bytes || (uintptr_t)packed % 256)
    return fail(h, KVP_ERR_WORKSPACE, "packed buffer needs %zu bytes, 256-byte aligned", h->packed_bytes);
  // validate everything before launching anything
  for (int t = 0; t < n; ++t) {
    const kvp_tensor& T = tensors[t];
    if (!T.name || !T.data) return fail(h, KVP_ERR_INVALID_ARG, "tensor %d has a NULL name or pointer", t);
    auto it = h->slots.find(T.name);
    if (it == h->slots.end()) {
      // tensors of dead auxiliary layers / the unused auxiliary head are accepted and ignored
      if (strncmp(T.name, "aux.", 4) == 0) continue;
      return fail(h, KVP_ERR_SHAPE, "unknown tensor name '%s'", T.name);
    }
    const PackSlot& s = it->second;
    if (T.dtype != KVP_F32 && T.dtype != KVP_BF16) return fail(h, KVP_ERR_INVALID_ARG, "tensor '%s': bad dtype", T.name);
    bool ok = (s.rows == 1 && T.ndim == 1) ? (T.shape[0] == s.cols)
                                           : (T.ndim == 2 && T.shape[0] == s.rows && T.shape[1] == s.cols);
    if (!ok) return fail(h, KVP_ERR_SHAPE, "tensor '%s': expected [%d, %d]", T.name, s.rows, s.cols);
  }
  if (h->packed && h->packed != packed) { h->loaded.clear(); h->ready_prefill = h->ready_decode = false; }
  h->packed = (char*)packed;
  LaunchCtx ctx{(cudaStream_t)stream, &h->n_launch, nullptr, h->opt.dtype};
  for (int t = 0; t < n; ++t) {
    const kvp_tensor& T = tensors[t];
    auto it = h->slots.find(T.name);
    if (it == h->slots.end()) continue;
    const PackSlot& s = it->second;
    launch_pack_rows(ctx, T.data, T.dtype, h->packed + s.off, s.dst_dtype, s.rows, s.cols, s.map);
    h->loaded.insert(T.name);
  }
  auto all = [&](const std::vector<std::string>& v) {
    for (auto& nme : v) if (!h->loaded.count(nme)) return false;
    return true;
  };
  h->ready_prefill = all(h->req_prefill);
  h->ready_decode = h->ready_prefill && all(h->req_decode_extra);
  return check_cuda(h, "kvp_load_weights");
}

// Enqueues every kernel of the time-to-first-token path on `stream` (validates first).
static kvp_status prefill_direct(kvp_handle* h, const int32_t* tokens, const int32_t* lengths, int32_t batch,
                                 const kvp_cache* cache, void* workspace, size_t workspace_bytes, float* logits_out,
                                 int32_t* first_token, void* stream) {
  CallShape cs;
  kvp_status st = common_checks(h, lengths, batch, cache, workspace, 0, &cs);
  if (st != KVP_OK) return st;
  if (!tokens || !logits_out) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  if (!h->ready_prefill) return fail(h, KVP_ERR_NOT_LOADED, "kvp_load_weights has not supplied every required tensor");
  WsLayout w = ws_layout(h, batch, cs.total);
  if (workspace_bytes < w.total) return fail(h, KVP_ERR_WORKSPACE, "workspace needs %zu bytes, got %zu", w.total, workspace_bytes);
  char* ws = (char*)workspace;
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)(ws + w.status);
  LaunchCtx ctx{s, &h->n_launch, status, h->opt.dtype};
  const ModelPlan& A = h->aux;
  const char* P = h->packed;
  const int T = cs.total, es = h->es;
  cudaMemsetAsync(status, 0, MEGA_STATUS_BYTES, s);

  int* cu_dev = (int*)(ws + w.cu);
  int* tok_pos = (int*)(ws + w.tok_pos);
  int* tok_slot = (int*)(ws + w.tok_slot);
  int* last_idx = (int*)(ws + w.last_idx);
  float* x = (float*)(ws + w.x);
  char* hbuf = ws + w.h;
  char* qkv = ws + w.qkv;
  const bool split = h->opt.dtype == KVP_BF16;   // K/V path in hi + lo bf16 parts
  char* h_lo = split ? ws + w.h_lo : nullptr;
  char* kv_lo = split ? ws + w.kv_lo : nullptr;
  float* qkv32 = (float*)(ws + w.qkv32);
  float2* rope_tab = (float2*)(ws + w.rope_tab);
  cudaError_t tc_err = cudaSuccess;
  char* attn = ws + w.attn;
  char* gu = ws + w.gu;
  char* act = ws + w.act;

  KVP_TIMED(KVP_CLASS_OTHER, launch_build_index(ctx, cs.cu.data(), batch, T, cu_dev, tok_pos, tok_slot, last_idx, cache->block_table,
                     cache->max_pages_per_seq, cache->n_pages, cache->seq_lens));
  // RMSNorm is folded into the GEMMs around it wherever both neighbours run on the tensor cores: the residual GEMM
  // that completes x writes bf16(x * gain) and the rows' sums of squares, the next GEMM scales its accumulator rows
  // by 1 / rms.  fused_in[j][0 / 1]: layer j's QKV / gate-up projection takes its operand that way.
  float* norm_ss = (float*)(ws + w.norm_ss);
  // (the producer needs every output tile to belong to one CTA: enough tiles for the SMs the GEMMs of this call get)
  const int sms_for_gemms = (h->side != nullptr && !h->timing && T <= 4096 && h->step_sms > 0) ? h->n_sm - h->step_sms : h->n_sm;
  const bool can_fuse = (h->opt.flags & KVP_OPT_SEPARATE_NORM) == 0 && tc_gemm_resid_can_fuse(T, A.d, h->n_sm) &&
                        tc_gemm_resid_can_fuse(T, A.d, sms_for_gemms);
  if (can_fuse) cudaMemsetAsync(norm_ss, 0, (size_t)2 * A.n_layers * T * 4, s);
  auto shape_ok = [&](int K, int N) { return can_fuse && h->opt.dtype == KVP_BF16 && K % 8 == 0 && N % 8 == 0 && A.d % 8 == 0; };
  std::vector<char> fused_in(2 * (h->j_max + 1), 0);
  for (int j = 0; j <= h->j_max; ++j) {
    const LayerPlan& L = A.L[j];
    const bool hd_ok = L.hd == 64 || L.hd == 128;
    // QKV of layer j (j >= 1) is fed by layer j-1's down projection; gate/up of layer j by its own O projection
    if (j >= 1 && hd_ok && shape_ok(A.d, L.nqkv) && shape_ok(A.L[j - 1].ffn, A.d)) fused_in[2 * j] = 1;
    if (j < h->j_max && L.ffn % 64 == 0 && shape_ok(A.d, 2 * L.ffn) && shape_ok(L.dq, A.d)) fused_in[2 * j + 1] = 1;
  }
  int2* attn_sched = (int2*)(ws + w.attn_sched);
  // two query tiles per CTA share their K/V tiles; with so few tokens that even the widest layer's pairs
  // would leave SMs idle, one tile per CTA finishes sooner
  int max_nq = 1;
  for (int j = 0; j <= h->j_max; ++j) max_nq = std::max(max_nq, A.L[j].nq);
  const int attn_tiles = attn_tc_items(cs.cu.data(), batch, 2) * max_nq < h->n_sm ? 1 : 2;
  const int attn_items = attn_tc_items(cs.cu.data(), batch, attn_tiles);
  if (h->opt.dtype == KVP_BF16 && (A.L[0].hd == 64 || A.L[0].hd == 128)) {
    KVP_TIMED(KVP_CLASS_OTHER, launch_rope_table(ctx, rope_tab, cs.max_len, A.L[0].hd, A.theta));
    KVP_TIMED(KVP_CLASS_OTHER, launch_attn_schedule(cu_dev, batch, attn_tiles, attn_sched, ctx.st, ctx.n_launch));
  }
  // ---- stage 1 + 2: auxiliary prefill, each layer's K/V pushed through the predictor ----
  // (only worth it while a layer's kernels leave SMs idle: with many tokens every kernel fills the GPU by itself)
  const bool fork = h->side != nullptr && !h->timing && T <= 4096;
  bool pending_join = false;
  // The base step in pieces beside the prefill: piece j = the base layers whose cache (and that of every
  // layer below them) is complete once auxiliary layer j has gone through the predictor.
  MegaParams mp;
  int mega_kmax = 0, piece = 0, base_done = 0, piece_split = 1;
  bool piped = fork && h->step_sms > 0 && h->j_max + 1 <= MEGA_COUNTERS &&
               mega_prepare(h, ctx, cache, w, ws, batch, cs.max_len, false, tokens, last_idx, logits_out, first_token, &mp, &mega_kmax);
  std::vector<int> ready_after(h->j_max + 2, 0);      // ready_after[j] = base layers runnable after auxiliary layer j
  if (piped) {
    int dep = 0, i = 0;
    for (int j = 0; j <= h->j_max; ++j) {
      while (i < h->base.n_layers && std::max(dep, h->map[i]) <= j) { dep = std::max(dep, h->map[i]); ++i; }
      ready_after[j] = i;
    }
    cudaMemsetAsync(mp.attn_done, 0, (size_t)batch * h->base.max_nkv * 4, s);
    h->gemm_sms = h->n_sm - h->step_sms;
    // key-range splits of the pieces: one attention item per CTA of the piece (measured: 2.72 against 2.83 ms at C2
    // with the 16 splits chosen for the whole GPU, which make two rounds on 72 SMs)
    int min_nkv = h->base.L[0].nkv;
    for (int i = 0; i < h->base.n_layers; ++i) min_nkv = std::min(min_nkv, h->base.L[i].nkv);
    piece_split = std::max(1, std::min(mp.n_split, h->step_sms / (batch * min_nkv)));
  }
  // More than 4 sequences: the step is a chain of short per-layer kernels bound by launch latency; the same
  // pieces go to the step stream as plain launches.  Their projections size their grids for step_tc_sms SMs;
  // the prefill's GEMMs keep the whole GPU (measured: restricting them costs more than the step gains).
  const bool piped_tc = !piped && fork && h->step_sms > 0 && h->step_tc_sms > 0 && step_uses_tc(h, batch);
  if (piped_tc) {
    int dep = 0, i = 0;
    for (int j = 0; j <= h->j_max; ++j) {
      while (i < h->base.n_layers && std::max(dep, h->map[i]) <= j) { dep = std::max(dep, h->map[i]); ++i; }
      ready_after[j] = i;
    }
    h->step_grid_sms = h->step_tc_sms;
  }
  KVP_TIMED(KVP_CLASS_OTHER, launch_embed(ctx, tokens, nullptr, T, P + A.embed, A.vocab, A.d, x));
  for (int j = 0; j <= h->j_max; ++j) {
    const LayerPlan& L = A.L[j];
    const bool last = (j == h->j_max);   // only K and V of the last mapped layer are needed
    const bool qkv_fused = fused_in[2 * j] != 0, gu_fused = fused_in[2 * j + 1] != 0;
    const bool next_fused = !last && fused_in[2 * (j + 1)] != 0;
    const bool qkv_half = h->qkv_half[j] != 0;
    if (!qkv_fused)
      KVP_TIMED(KVP_CLASS_OTHER, launch_rmsnorm(ctx, x, (const float*)(P + L.attn_norm), A.eps, T, A.d, hbuf, h->opt.dtype, qkv_half ? nullptr : h_lo, qkv_half));
    // predictor of this layer: K_hat_i = K_A,j FK_i^T, V_hat_i = V_A,j FV_i^T for every base layer i with j_i = j
    const PredGroup& pg = h->groups[j];
    const bool half_path = pg.half_path;
    PagedOut paged[2];
    for (int kv = 0; kv < 2; ++kv) {
      PagedOut& q = paged[kv];
      q.n_seg = pg.n_seg;
      for (int sg = 0; sg <= pg.n_seg; ++sg) q.col0[sg] = pg.col0[sg];
      for (int sg = 0; sg < pg.n_seg; ++sg) {
        int i = pg.base_layer[sg];
        q.n_kv[sg] = h->base.L[i].nkv;
        q.pool[sg] = kv ? cache->v_pools[i] : cache->k_pools[i];
      }
      q.bias = h->opt.predictor_bias ? (const float*)(P + (kv ? pg.bv : pg.bk)) : nullptr;
      q.tok_slot = tok_slot;
      q.head_dim = h->base.L[0].hd;
    }
    // With enough tokens to give every SM a work item, the K/V projection and the predictor are ONE kernel: the
    // predictor is the projection's epilogue and K_A / V_A reach it through shared memory.
    KvPred kp{};
    kp.A = (const bf16*)hbuf; kp.lda = A.d; kp.A_lo = (const bf16*)h_lo; kp.lda_lo = A.d;
    kp.Wkv = (const bf16*)(P + L.wqkv + (size_t)L.dq * A.d * es); kp.ldw = A.d; kp.M = T; kp.K = A.d;
    kp.dkv = L.dkv; kp.hd = L.hd; kp.kv_begin = 0; kp.kv_end = 2;
    if (qkv_fused) { kp.ss_in = norm_ss + (size_t)(2 * j) * T; kp.rms_eps = A.eps; }
    kp.rope_tab = rope_tab; kp.tab_stride = cs.max_len; kp.tok_pos = tok_pos; kp.k_gain = A.qk_norm ? (const float*)(P + L.k_norm) : nullptr; kp.eps = A.eps;
    kp.C = (bf16*)qkv; kp.ldc = L.nqkv; kp.k_col = L.dq;
    kp.FK = P + pg.fk; kp.FV = P + pg.fv; kp.n_tot = pg.col0[pg.n_seg]; kp.paged[0] = paged[0]; kp.paged[1] = paged[1];
    kp.n_sm = h->gemm_sms;
    const bool fused_kv = (h->opt.flags & KVP_OPT_FUSED_KV_PRED) != 0 && half_path && split && pg.n_seg > 0 && 2 * ((T + 127) / 128) >= h->n_sm && kvpred_tc_supported(kp);
    int col_begin = last ? L.dq : 0;
    int n_out = L.nqkv - col_begin;
    const int q_heads = last ? 0 : L.nq;
    if (fused_kv) { col_begin = 0; n_out = L.dq; }      // the GEMM below projects the queries only
    TcGemm tq{};
    tq.A = (const bf16*)hbuf; tq.lda = A.d; tq.A2 = (const bf16*)h_lo; tq.lda2 = A.d; tq.split_begin = L.dq - col_begin;
    tq.W = (const bf16*)(P + L.wqkv + (size_t)col_begin * A.d * es); tq.ldw = A.d; tq.M = T; tq.N = n_out; tq.K = A.d;
    tq.epi = TC_QKV; tq.C = (bf16*)(qkv + (size_t)col_begin * es); tq.ldc = L.nqkv;
    tq.C_lo = (bf16*)kv_lo; tq.ld_lo = 2 * L.dkv; tq.lo_col_begin = q_heads * L.hd;
    tq.rot_cols = (q_heads + L.nkv) * L.hd; tq.hd = L.hd; tq.rope_tab = rope_tab; tq.tab_stride = cs.max_len; tq.tok_pos = tok_pos;
    if (fused_kv) { tq.C_lo = nullptr; tq.rot_cols = q_heads * L.hd; tq.A2 = nullptr; }
    if (qkv_half) { tq.A2 = nullptr; tq.f16_operands = 1; }      // h and W_qkv are halves: one pass over every column
    const float* qn = A.qk_norm ? (const float*)(P + L.q_norm) : nullptr;
    const float* kn = A.qk_norm ? (const float*)(P + L.k_norm) : nullptr;
    tq.q_gain = qn; tq.k_gain = kn; tq.q_cols = q_heads * L.hd; tq.eps = A.eps;
    if (qkv_fused) { tq.ss_in = norm_ss + (size_t)(2 * j) * T; tq.rms_eps = A.eps; }
    tq.lo_is_half = half_path ? 1 : 0;
    if (fused_kv) {
      TimedScope ts(h, ctx.st, KVP_CLASS_KV_PRED);
      cudaError_t e = launch_kvpred_tc(kp, ctx.status, ctx.st, ctx.n_launch);
      if (e != cudaSuccess && tc_err == cudaSuccess) tc_err = e;
    }
    if (fused_kv && last) {
      // only keys and values of the last mapped layer are needed: nothing else to project
    } else if (!try_tc(h, ctx, tq, KVP_CLASS_AUX_GEMM, &tc_err)) {
      if (half_path && h->groups[j].n_seg > 0) return fail(h, KVP_ERR_CUDA, "internal: half-precision predictor input planned for a projection the tensor-core kernel refuses");
      if (qkv_fused) return fail(h, KVP_ERR_CUDA, "internal: fused norm planned for a projection the tensor-core kernel refuses");
      if (qkv_half) return fail(h, KVP_ERR_CUDA, "internal: half-precision operands planned for a projection the tensor-core kernel refuses");
      GemmArgs g{};
      g.A = hbuf; g.lda = A.d; g.M = T; g.K = A.d;
      g.A2 = h_lo; g.lda2 = A.d;
      g.split_begin = L.dq - col_begin;    // the K and V columns take the lo part of h as well
      g.W = P + L.wqkv + (size_t)col_begin * A.d * es; g.ldw = A.d; g.N = n_out;
      g.C = qkv32; g.ldc = g.N;
      KVP_TIMED(KVP_CLASS_AUX_GEMM, launch_gemm_simt(ctx, g, EPI_STORE32));
      KVP_TIMED(KVP_CLASS_OTHER, launch_rope_split(ctx, qkv32, g.N, T, g.N / L.hd, q_heads + L.nkv, L.hd, tok_pos, A.theta,
                                                   qkv + (size_t)col_begin * es, L.nqkv, kv_lo, 2 * L.dkv, q_heads, q_heads, qn, kn, A.eps));
    }
    if (pg.n_seg > 0) {
      LaunchCtx pctx = ctx;
      if (fork) {
        cudaEventRecord(h->ev_fork, s);
        cudaStreamWaitEvent(h->side, h->ev_fork, 0);
        pctx.st = h->side;
      }
      const LaunchCtx& ctx = pctx;      // the predictor's launches go to the side stream
      for (int kv = 0; kv < 2 && !fused_kv; ++kv) {
        GemmArgs p{};
        p.A = qkv + (size_t)(L.dq + kv * L.dkv) * es; p.lda = L.nqkv; p.M = T; p.K = L.dkv;
        if (split) { p.A2 = kv_lo + (size_t)(kv * L.dkv) * es; p.lda2 = 2 * L.dkv; p.split_begin = 0; }
        p.W = P + (kv ? pg.fv : pg.fk); p.ldw = L.dkv; p.N = pg.col0[pg.n_seg];
        p.paged = paged[kv];
        TcGemm tp{};
        tp.A = (const bf16*)p.A; tp.lda = p.lda; tp.A2 = (const bf16*)p.A2; tp.lda2 = p.lda2; tp.split_begin = 0;
        tp.W = (const bf16*)p.W; tp.ldw = p.ldw; tp.M = T; tp.N = p.N; tp.K = p.K; tp.epi = TC_PAGED; tp.paged = p.paged;
        if (half_path) {     // K_A / V_A as halves (written by the projection's epilogue), FK / FV stored as halves: one pass
          tp.A = (const bf16*)(kv_lo + (size_t)(kv * L.dkv) * es); tp.lda = 2 * L.dkv; tp.A2 = nullptr; tp.f16_operands = 1;
        }
        if (!try_tc(h, ctx, tp, KVP_CLASS_PREDICTOR, &tc_err)) {
          if (half_path) tc_err = cudaErrorInvalidValue;    // the matrices are stored as halves: no other kernel reads them
          else KVP_TIMED(KVP_CLASS_PREDICTOR, launch_gemm_simt(ctx, p, EPI_PAGED));
        }
      }
      if (fork) {
        cudaEventRecord(h->ev_join, h->side);
        pending_join = true;
      }
      if (piped && (ready_after[j] > base_done || last)) {
        cudaStreamWaitEvent(h->step_st, h->ev_join, 0);
        MegaParams q = mp;
        q.layer_begin = base_done; q.layer_end = last ? h->base.n_layers : ready_after[j];
        q.do_embed = base_done == 0; q.do_head = last; q.counter_idx = piece++;
        q.n_split = piece_split;
        // the last piece starts when the prefill has nothing left to run: it takes every SM
        cudaError_t e = launch_step_mega(q, h->opt.dtype, mega_kmax, last ? h->n_sm : h->step_sms, h->step_st, ctx.n_launch);
        if (e != cudaSuccess && tc_err == cudaSuccess) tc_err = e;
        base_done = q.layer_end;
      }
      if (piped_tc && (ready_after[j] > base_done || last)) {
        cudaStreamWaitEvent(h->step_st, h->ev_join, 0);
        LaunchCtx sctx = ctx;
        sctx.st = h->step_st;
        const int end = last ? h->base.n_layers : ready_after[j];
        if (last) h->step_grid_sms = h->n_sm;          // the prefill has nothing left to run
        if (base_done == 0)
          launch_embed(sctx, tokens, last_idx, batch, P + h->base.embed, h->base.vocab, h->base.d, (float*)(ws + w.xb));
        for (int i = base_done; i < end; ++i) base_layer_step(h, sctx, i, cache, w, ws, batch, cs.max_len, false, &tc_err);
        if (last) base_head(h, sctx, w, ws, batch, logits_out, first_token, &tc_err);
        base_done = end;
      }
    }
    if (last) break;
    if (split && attn_items <= 65535 && attn_tc_supported(L.hd, L.nqkv, qkv, L.dq, attn)) {
      TimedScope ts(h, ctx.st, KVP_CLASS_AUX_ATTN);
      cudaError_t e = launch_attn_tc((const bf16*)qkv, L.nqkv, T, L.nq, L.nkv, L.hd, cu_dev, attn_sched, attn_items, attn_tiles, (bf16*)attn,
                                     L.dq, ctx.status, ctx.st, ctx.n_launch);
      if (e != cudaSuccess && tc_err == cudaSuccess) tc_err = e;
    } else {
      KVP_TIMED(KVP_CLASS_AUX_ATTN, launch_attn_prefill_simt(ctx, qkv, L.nqkv, L.nq, L.nkv, L.hd, cu_dev, batch, T, attn, L.dq));
    }
    GemmArgs o{};
    o.A = attn; o.lda = L.dq; o.W = P + L.wo; o.ldw = L.dq; o.M = T; o.N = A.d; o.K = L.dq; o.X = x; o.ldx = A.d;
    TcGemm to{};
    to.A = (const bf16*)attn; to.lda = L.dq; to.W = (const bf16*)(P + L.wo); to.ldw = L.dq; to.M = T; to.N = A.d; to.K = L.dq;
    to.epi = TC_RESID; to.X = x; to.ldx = A.d;
    if (gu_fused) {      // the O projection completes x: it also writes the gate/up projection's operand
      to.H = (bf16*)hbuf; to.ldh = A.d; to.gain_next = (const float*)(P + L.ffn_norm);
      to.ss_out = norm_ss + (size_t)(2 * j + 1) * T;
    }
    if (!try_tc(h, ctx, to, KVP_CLASS_AUX_GEMM, &tc_err)) {
      if (gu_fused) return fail(h, KVP_ERR_CUDA, "internal: fused norm planned for a projection the tensor-core kernel refuses");
      KVP_TIMED(KVP_CLASS_AUX_GEMM, launch_gemm_simt(ctx, o, EPI_RESID));
    }
    if (!gu_fused)
      KVP_TIMED(KVP_CLASS_OTHER, launch_rmsnorm(ctx, x, (const float*)(P + L.ffn_norm), A.eps, T, A.d, hbuf, h->opt.dtype));
    GemmArgs f{};
    f.A = hbuf; f.lda = A.d; f.W = P + L.wgu; f.ldw = A.d; f.M = T; f.N = 2 * L.ffn; f.K = A.d; f.C = gu; f.ldc = 2 * L.ffn;
    TcGemm tf{};
    tf.A = (const bf16*)hbuf; tf.lda = A.d; tf.W = (const bf16*)(P + L.wgu); tf.ldw = A.d; tf.M = T; tf.N = 2 * L.ffn; tf.K = A.d;
    tf.epi = TC_SWIGLU; tf.C = (bf16*)act; tf.ldc = L.ffn; tf.ffn = L.G == 64 ? L.ffn : 1;
    if (gu_fused) { tf.ss_in = norm_ss + (size_t)(2 * j + 1) * T; tf.rms_eps = A.eps; }
    if (!try_tc(h, ctx, tf, KVP_CLASS_AUX_GEMM, &tc_err)) {
      if (gu_fused) return fail(h, KVP_ERR_CUDA, "internal: fused norm planned for a projection the tensor-core kernel refuses");
      KVP_TIMED(KVP_CLASS_AUX_GEMM, launch_gemm_simt(ctx, f, EPI_STORE));
      KVP_TIMED(KVP_CLASS_OTHER, launch_swiglu(ctx, gu, T, L.ffn, L.G, act));
    }
    GemmArgs d{};
    d.A = act; d.lda = L.ffn; d.W = P + L.wd; d.ldw = L.ffn; d.M = T; d.N = A.d; d.K = L.ffn; d.X = x; d.ldx = A.d;
    TcGemm td{};
    td.A = (const bf16*)act; td.lda = L.ffn; td.W = (const bf16*)(P + L.wd); td.ldw = L.ffn; td.M = T; td.N = A.d; td.K = L.ffn;
    td.epi = TC_RESID; td.X = x; td.ldx = A.d;
    if (next_fused) {    // the down projection completes x: it also writes the next layer's QKV operand (hi + lo parts)
      const bool next_half = h->qkv_half[j + 1] != 0;     // ... or as halves, where that projection takes f16 operands
      td.H = (bf16*)hbuf; td.H_lo = next_half ? nullptr : (bf16*)h_lo; td.h_is_half = next_half ? 1 : 0;
      td.ldh = A.d; td.gain_next = (const float*)(P + A.L[j + 1].attn_norm);
      td.ss_out = norm_ss + (size_t)(2 * (j + 1)) * T;
    }
    if (!try_tc(h, ctx, td, KVP_CLASS_AUX_GEMM, &tc_err)) {
      if (next_fused) return fail(h, KVP_ERR_CUDA, "internal: fused norm planned for a projection the tensor-core kernel refuses");
      KVP_TIMED(KVP_CLASS_AUX_GEMM, launch_gemm_simt(ctx, d, EPI_RESID));
    }
  }
  if (pending_join) cudaStreamWaitEvent(s, h->ev_join, 0);     // the base step reads what the predictor wrote
  h->gemm_sms = h->step_grid_sms = h->n_sm;
  if (piped || piped_tc) {     // the step is already enqueued in pieces: join its stream
    cudaEventRecord(h->ev_step, h->step_st);
    cudaStreamWaitEvent(s, h->ev_step, 0);
  }
  if (tc_err != cudaSuccess) return fail(h, KVP_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(tc_err));
  // ---- stage 3: one base step per sequence on its last prompt token ----
  if (!piped && !piped_tc && !base_step_fused(h, ctx, cache, w, ws, batch, cs.max_len, false, tokens, last_idx, logits_out, first_token, &tc_err)) {
    KVP_TIMED(KVP_CLASS_OTHER, launch_embed(ctx, tokens, last_idx, batch, P + h->base.embed, h->base.vocab, h->base.d, (float*)(ws + w.xb)));
    for (int i = 0; i < h->base.n_layers; ++i) base_layer_step(h, ctx, i, cache, w, ws, batch, cs.max_len, false, &tc_err);
    base_head(h, ctx, w, ws, batch, logits_out, first_token, &tc_err);
  }
  if (tc_err != cudaSuccess) return fail(h, KVP_ERR_CUDA, "base step launch: %s", cudaGetErrorString(tc_err));
  return check_cuda(h, "kvp_prefill_predict");
}

// The schedule is a few hundred short kernels, so the host's launch cost would exceed the device
// time.  The first call with a given set of arguments records the schedule into a CUDA graph;
// later calls with the same arguments replay it (token values may change, they are read on the
// device).  Everything baked into the kernels' parameters is part of the key.
kvp_status kvp_prefill_predict(kvp_handle* h, const int32_t* tokens, const int32_t* lengths, int32_t batch,
                               const kvp_cache* cache, void* workspace, size_t workspace_bytes, float* logits_out,
                               int32_t* first_token, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  // (the legacy default stream cannot record)
  bool graph_ok = h && h->use_graph && s != nullptr && s != cudaStreamLegacy && !h->timing && lengths && cache && cache->k_pools && cache->v_pools && batch > 0 &&
                  batch <= KVP_MAX_BATCH && cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
  if (!graph_ok) {
    cudaGetLastError();
    return prefill_direct(h, tokens, lengths, batch, cache, workspace, workspace_bytes, logits_out, first_token, stream);
  }
  std::vector<uint64_t> key;
  key.reserve(12 + batch + 2 * h->base.n_layers);
  key.push_back((uint64_t)(uintptr_t)tokens); key.push_back((uint64_t)batch);
  key.push_back((uint64_t)(uintptr_t)workspace); key.push_back((uint64_t)workspace_bytes);
  key.push_back((uint64_t)(uintptr_t)logits_out); key.push_back((uint64_t)(uintptr_t)first_token);
  key.push_back((uint64_t)(uintptr_t)cache->block_table); key.push_back((uint64_t)(uintptr_t)cache->seq_lens);
  key.push_back((uint64_t)cache->max_pages_per_seq); key.push_back((uint64_t)cache->n_pages);
  key.push_back((uint64_t)(uintptr_t)h->packed); key.push_back((uint64_t)(uintptr_t)s);
  for (int b = 0; b < batch; ++b) key.push_back((uint64_t)(uint32_t)lengths[b]);
  for (int i = 0; i < h->base.n_layers; ++i) {
    key.push_back((uint64_t)(uintptr_t)cache->k_pools[i]);
    key.push_back((uint64_t)(uintptr_t)cache->v_pools[i]);
  }
  for (auto& g : h->graphs)
    if (g.key == key) {
      g.last_use = ++h->graph_clock;
      h->err.clear();
      if (cudaGraphLaunch(g.exec, s) != cudaSuccess) return check_cuda(h, "cudaGraphLaunch");
      h->n_launch += g.launches;
      return KVP_OK;
    }
  // record
  int64_t n0 = h->n_launch;
  if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    return prefill_direct(h, tokens, lengths, batch, cache, workspace, workspace_bytes, logits_out, first_token, stream);
  }
  kvp_status st = prefill_direct(h, tokens, lengths, batch, cache, workspace, workspace_bytes, logits_out, first_token, stream);
  cudaGraph_t graph = nullptr;
  cudaError_t ce = cudaStreamEndCapture(s, &graph);
  if (st != KVP_OK) {               // argument error: nothing was launched, drop the empty capture
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
    h->n_launch = n0;
    return st;
  }
  cudaGraphExec_t exec = nullptr;
  if (ce != cudaSuccess || !graph || cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) {
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
    h->n_launch = n0;
    h->use_graph = false;           // this context cannot record: run directly from now on
    return prefill_direct(h, tokens, lengths, batch, cache, workspace, workspace_bytes, logits_out, first_token, stream);
  }
  cudaGraphDestroy(graph);
  int64_t launches = h->n_launch - n0;
  h->n_launch = n0;
  if (h->graphs.size() >= 8) {      // evict the least recently used schedule
    size_t victim = 0;
    for (size_t i = 1; i < h->graphs.size(); ++i) if (h->graphs[i].last_use < h->graphs[victim].last_use) victim = i;
    cudaGraphExecDestroy(h->graphs[victim].exec);
    h->graphs.erase(h->graphs.begin() + victim);
  }
  h->graphs.push_back({key, exec, launches, ++h->graph_clock});
  if (cudaGraphLaunch(exec, s) != cudaSuccess) return check_cuda(h, "cudaGraphLaunch");
  h->n_launch += launches;
  return KVP_OK;
}

kvp_status kvp_prefill_predict_host(kvp_handle* h, const int32_t* tokens_host, const int32_t* lengths, int32_t batch,
                                    const kvp_cache* cache, void* workspace, size_t workspace_bytes, float* logits_dev,
                                    float* logits_host, int32_t* first_token_host, void* stream) {
  CallShape cs;
  kvp_status st = common_checks(h, lengths, batch, cache, workspace, 0, &cs);
  if (st != KVP_OK) return st;
  if (!tokens_host || !logits_dev || !first_token_host) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  WsLayout w = ws_layout(h, batch, cs.total);
  if (workspace_bytes < w.total) return fail(h, KVP_ERR_WORKSPACE, "workspace needs %zu bytes, got %zu", w.total, workspace_bytes);
  char* ws = (char*)workspace;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t* tok_dev = (int32_t*)(ws + w.tok_stage);
  int32_t* first_dev = (int32_t*)(ws + w.first_stage);
  if (cudaMemcpyAsync(tok_dev, tokens_host, (size_t)cs.total * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return check_cuda(h, "token upload");
  st = kvp_prefill_predict(h, tok_dev, lengths, batch, cache, workspace, workspace_bytes, logits_dev, first_dev, stream);
  if (st != KVP_OK) return st;
  if (logits_host)
    cudaMemcpyAsync(logits_host, logits_dev, (size_t)batch * h->base.vocab * 4, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(first_token_host, first_dev, (size_t)batch * 4, cudaMemcpyDeviceToHost, s);
  if (cudaStreamSynchronize(s) != cudaSuccess) return check_cuda(h, "kvp_prefill_predict_host");
  return check_cuda(h, "kvp_prefill_predict_host");
}

kvp_status kvp_decode_step(kvp_handle* h, const int32_t* tokens, const int32_t* lengths_host, int32_t batch,
                           const kvp_cache* cache, void* workspace, size_t workspace_bytes, float* logits_out,
                           int32_t* next_token, void* stream) {
  CallShape cs;
  kvp_status st = common_checks(h, lengths_host, batch, cache, workspace, 1, &cs);
  if (st != KVP_OK) return st;
  if (!tokens || !logits_out) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  if (!h->ready_decode) return fail(h, KVP_ERR_NOT_LOADED, "kvp_load_weights has not supplied every required tensor");
  WsLayout w = ws_layout(h, batch, batch);
  if (workspace_bytes < w.total) return fail(h, KVP_ERR_WORKSPACE, "workspace needs %zu bytes, got %zu", w.total, workspace_bytes);
  char* ws = (char*)workspace;
  LaunchCtx ctx{(cudaStream_t)stream, &h->n_launch, (int*)(ws + w.status), h->opt.dtype};
  cudaError_t mega_err = cudaSuccess;
  cudaMemsetAsync((char*)(ws + w.status) + 128, 0, MEGA_COUNTERS * 4, ctx.st);     // barrier counters of the persistent kernel
  if (base_step_fused(h, ctx, cache, w, ws, batch, cs.max_len + 1, true, tokens, nullptr, logits_out, next_token, &mega_err)) {
    if (mega_err != cudaSuccess) return fail(h, KVP_ERR_CUDA, "base step launch: %s", cudaGetErrorString(mega_err));
    return check_cuda(h, "kvp_decode_step");
  }
  KVP_TIMED(KVP_CLASS_OTHER, launch_embed(ctx, tokens, nullptr, batch, h->packed + h->base.embed, h->base.vocab, h->base.d, (float*)(ws + w.xb)));
  for (int i = 0; i < h->base.n_layers; ++i) base_layer_step(h, ctx, i, cache, w, ws, batch, cs.max_len + 1, true, &mega_err);
  base_head(h, ctx, w, ws, batch, logits_out, next_token, &mega_err);
  KVP_TIMED(KVP_CLASS_OTHER, launch_add_int(ctx, cache->seq_lens, batch, 1));
  if (mega_err != cudaSuccess) return fail(h, KVP_ERR_CUDA, "base step launch: %s", cudaGetErrorString(mega_err));
  return check_cuda(h, "kvp_decode_step");
}

kvp_status kvp_timing_enable(kvp_handle* h, int32_t on) {
  if (!h) return KVP_ERR_INVALID_ARG;
  h->timing = on != 0;
  return KVP_OK;
}

kvp_status kvp_timing_read(kvp_handle* h, double* ms, int64_t* launches) {
  if (!h || !ms || !launches) return KVP_ERR_INVALID_ARG;
  for (int c = 0; c < KVP_N_CLASSES; ++c) { ms[c] = 0.0; launches[c] = 0; }
  for (auto& r : h->recs) {
    float t = 0.f;
    if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) {
      cudaError_t e = cudaGetLastError();
      return fail(h, KVP_ERR_CUDA, "kvp_timing_read: %s", cudaGetErrorString(e));
    }
    ms[r.cls] += t;
    launches[r.cls] += r.launches;
    h->free_events.push_back(r.a);
    h->free_events.push_back(r.b);
  }
  h->recs.clear();
  return KVP_OK;
}

kvp_status kvp_poll_status(kvp_handle* h, void* workspace, void* stream) {
  if (!h || !workspace) return KVP_ERR_INVALID_ARG;
  h->err.clear();
  cudaStream_t s = (cudaStream_t)stream;
  int code = 0;
  if (cudaStreamSynchronize(s) != cudaSuccess || cudaMemcpy(&code, workspace, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemset(workspace, 0, MEGA_STATUS_BYTES) != cudaSuccess) {
    cudaError_t e = cudaGetLastError();
    return fail(h, KVP_ERR_CUDA, "kvp_poll_status: %s", cudaGetErrorString(e));
  }
  switch (code) {
    case DEV_OK: return KVP_OK;
    case DEV_TIMEOUT: return fail(h, KVP_ERR_TIMEOUT, "a device-side wait ran out");
    case DEV_BAD_TOKEN: return fail(h, KVP_ERR_BAD_INDEX, "a token id was outside [0, vocab)");
    case DEV_BAD_PAGE: return fail(h, KVP_ERR_BAD_INDEX, "a block-table entry was outside [0, n_pages)");
    default: return fail(h, KVP_ERR_CUDA, "unknown device status %d", code);
  }
}

}  // extern "C"

// ---- training-time forward (Sec. 4.1 "Training", Sec. 4.3) ------------------------------------------------
namespace {
struct TrainWs {
  size_t status, cu, last_idx, tok_pos, tok_slot, rope_tab, x, h, h_lo, qkv, qkv32, kv_lo, attn, attn_lo, gu, act, act_lo, attn_sched, total;
};
TrainWs train_ws_layout(const kvp_handle* h, int64_t Bm, int64_t Tm) {
  TrainWs w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const ModelPlan& B = h->base;
  const size_t es = h->es;
  w.status = take(16384);
  w.cu = take((Bm + 1) * 4);
  w.last_idx = take(Bm * 4);
  w.tok_pos = take(Tm * 4);
  w.tok_slot = take(Tm * 4);
  w.rope_tab = take(Tm * (size_t)((B.L[0].hd / 2 + 1) & ~1) * 8);
  w.x = take(Tm * B.d * 4);
  w.h = take(Tm * B.d * es);
  w.h_lo = take(Tm * B.d * es);
  w.qkv = take(Tm * B.max_nqkv * es);
  w.qkv32 = take(Tm * B.max_nqkv * 4);
  w.kv_lo = take(Tm * 2 * (size_t)B.max_dkv * es);
  w.attn = take(Tm * B.max_dq * es);
  w.attn_lo = take(Tm * B.max_dq * es);
  w.gu = take(Tm * 2 * (size_t)B.max_ffn * es);
  w.act = take(Tm * (size_t)B.max_ffn * es);
  w.act_lo = take(Tm * (size_t)B.max_ffn * es);
  w.attn_sched = take((size_t)(Tm / 128 + Bm + 1) * 8);
  w.total = off;
  return w;
}
}  // namespace

extern "C" kvp_status kvp_train_workspace_bytes(const kvp_handle* h, int32_t max_batch, int64_t max_total_tokens, size_t* bytes) {
  if (!h || !bytes || max_batch <= 0 || max_batch > KVP_MAX_BATCH || max_total_tokens < max_batch) return KVP_ERR_INVALID_ARG;
  *bytes = train_ws_layout(h, max_batch, max_total_tokens).total;
  return KVP_OK;
}

extern "C" kvp_status kvp_train_forward(kvp_handle* h, const int32_t* tokens, const int32_t* lengths, int32_t batch,
                                        const kvp_cache* cache, void* workspace, size_t workspace_bytes, float* logits_out,
                                        float* l1_k, float* l1_v, void* stream) {
  CallShape cs;
  kvp_status st = common_checks(h, lengths, batch, cache, workspace, 0, &cs);
  if (st != KVP_OK) return st;
  if (!tokens || !l1_k || !l1_v) return fail(h, KVP_ERR_INVALID_ARG, "NULL argument");
  if (!h->ready_decode) return fail(h, KVP_ERR_NOT_LOADED, "kvp_load_weights has not supplied every required tensor");
  const int T = cs.total, es = h->es;
  TrainWs w = train_ws_layout(h, batch, T);
  if (workspace_bytes < w.total) return fail(h, KVP_ERR_WORKSPACE, "workspace needs %zu bytes, got %zu", w.total, workspace_bytes);
  char* ws = (char*)workspace;
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)(ws + w.status);
  LaunchCtx ctx{s, &h->n_launch, status, h->opt.dtype};
  const ModelPlan& B = h->base;
  const char* P = h->packed;
  cudaMemsetAsync(status, 0, MEGA_STATUS_BYTES, s);
  cudaMemsetAsync(l1_k, 0, (size_t)B.n_layers * 4, s);
  cudaMemsetAsync(l1_v, 0, (size_t)B.n_layers * 4, s);
  int* cu_dev = (int*)(ws + w.cu);
  int* tok_pos = (int*)(ws + w.tok_pos);
  int* tok_slot = (int*)(ws + w.tok_slot);
  float* x = (float*)(ws + w.x);
  char* hbuf = ws + w.h;
  char* qkv = ws + w.qkv;
  const bool split = h->opt.dtype == KVP_BF16;
  char* h_lo = split ? ws + w.h_lo : nullptr;
  char* kv_lo = split ? ws + w.kv_lo : nullptr;
  float* qkv32 = (float*)(ws + w.qkv32);
  float2* rope_tab = (float2*)(ws + w.rope_tab);
  char* attn = ws + w.attn;
  char* gu = ws + w.gu;
  char* act = ws + w.act;
  int2* attn_sched = (int2*)(ws + w.attn_sched);
  cudaError_t tc_err = cudaSuccess;
  // This forward feeds activations to four projections per layer at EVERY position and its attention reads the whole
  // predicted cache, so bf16's 8 significant bits at those points would dominate the logits error.  Where the tensor-core
  // kernels take the shapes, every projection operand travels as a bf16 value plus its bf16 remainder (two MMA passes),
  // q / k / v reach the attention as IEEE halves (the cache's own format: predicted entries are copied, not re-rounded).
  bool hp = split && (B.L[0].hd == 64 || B.L[0].hd == 128) && B.d % 8 == 0 && B.vocab % 4 == 0;
  for (int i = 0; i < B.n_layers && hp; ++i) hp = B.L[i].ffn % 64 == 0 && B.L[i].G == 64;
  char* attn_lo = hp ? ws + w.attn_lo : nullptr;
  char* act_lo = hp ? ws + w.act_lo : nullptr;
  // token -> (sequence position, cache slot); seq_lens is rewritten with the same lengths the cache already holds
  launch_build_index(ctx, cs.cu.data(), batch, T, cu_dev, tok_pos, tok_slot, (int*)(ws + w.last_idx), cache->block_table,
                     cache->max_pages_per_seq, cache->n_pages, cache->seq_lens);
  int max_nq = 1;
  for (int i = 0; i < B.n_layers; ++i) max_nq = std::max(max_nq, B.L[i].nq);
  const int attn_tiles = attn_tc_items(cs.cu.data(), batch, 2) * max_nq < h->n_sm ? 1 : 2;
  const int attn_items = attn_tc_items(cs.cu.data(), batch, attn_tiles);
  if (h->opt.dtype == KVP_BF16 && (B.L[0].hd == 64 || B.L[0].hd == 128)) {
    launch_rope_table(ctx, rope_tab, cs.max_len, B.L[0].hd, B.theta);
    launch_attn_schedule(cu_dev, batch, attn_tiles, attn_sched, ctx.st, ctx.n_launch);
  }
  // pass 0: the base model's ordinary forward, for its own cache KV_B (consistency terms against the predicted one);
  // pass 1: the forward whose attention reads the predicted cache, for the logits
  for (int pass = 0; pass < 2; ++pass) {
    if (pass == 1 && !logits_out) break;
    launch_embed(ctx, tokens, nullptr, T, P + B.embed, B.vocab, B.d, x);
    for (int i = 0; i < B.n_layers; ++i) {
      const LayerPlan& L = B.L[i];
      const bool last = pass == 0 && i == B.n_layers - 1;     // only this layer's keys and values are still needed
      launch_rmsnorm(ctx, x, (const float*)(P + L.attn_norm), B.eps, T, B.d, hbuf, h->opt.dtype, h_lo);
      const int col_begin = last ? L.dq : 0;
      const int n_out = L.nqkv - col_begin, q_heads = last ? 0 : L.nq;
      const float* qn = B.qk_norm ? (const float*)(P + L.q_norm) : nullptr;
      const float* kn = B.qk_norm ? (const float*)(P + L.k_norm) : nullptr;
      TcGemm tq{};
      tq.A = (const bf16*)hbuf; tq.lda = B.d; tq.A2 = (const bf16*)h_lo; tq.lda2 = B.d; tq.split_begin = hp ? 0 : L.dq - col_begin;
      tq.W = (const bf16*)(P + L.wqkv + (size_t)col_begin * B.d * es); tq.ldw = B.d; tq.M = T; tq.N = n_out; tq.K = B.d;
      tq.epi = TC_QKV; tq.C = (bf16*)(qkv + (size_t)col_begin * es); tq.ldc = L.nqkv;
      tq.C_lo = (bf16*)kv_lo; tq.ld_lo = 2 * L.dkv; tq.lo_col_begin = q_heads * L.hd;
      tq.rot_cols = (q_heads + L.nkv) * L.hd; tq.hd = L.hd; tq.rope_tab = rope_tab; tq.tab_stride = cs.max_len; tq.tok_pos = tok_pos;
      tq.q_gain = qn; tq.k_gain = kn; tq.q_cols = q_heads * L.hd; tq.eps = B.eps;
      if (hp) { tq.c_is_half = 1; tq.C_lo = nullptr; }
      if (!try_tc(h, ctx, tq, KVP_CLASS_OTHER, &tc_err)) {
        if (hp) return fail(h, KVP_ERR_CUDA, "internal: the tensor-core kernel refused a projection of the training-time forward");
        GemmArgs g{};
        g.A = hbuf; g.lda = B.d; g.M = T; g.K = B.d; g.A2 = h_lo; g.lda2 = B.d; g.split_begin = L.dq - col_begin;
        g.W = P + L.wqkv + (size_t)col_begin * B.d * es; g.ldw = B.d; g.N = n_out; g.C = qkv32; g.ldc = g.N;
        launch_gemm_simt(ctx, g, EPI_STORE32);
        launch_rope_split(ctx, qkv32, g.N, T, g.N / L.hd, q_heads + L.nkv, L.hd, tok_pos, B.theta, qkv + (size_t)col_begin * es,
                          L.nqkv, kv_lo, 2 * L.dkv, q_heads, q_heads, qn, kn, B.eps);
      }
      if (pass == 0) {
        launch_kv_l1(ctx, qkv, L.nqkv, L.dq, kv_lo, 2 * L.dkv, T, L.nkv, L.hd, tok_slot, cache->k_pools[i], cache->v_pools[i],
                     l1_k + i, l1_v + i, hp);
        if (last) break;
      } else {
        launch_kv_take(ctx, qkv, L.nqkv, L.dq, T, L.nkv, L.hd, tok_slot, cache->k_pools[i], cache->v_pools[i], hp);
      }
      if (split && attn_items <= 65535 && attn_tc_supported(L.hd, L.nqkv, qkv, L.dq, attn)) {
        cudaError_t e = launch_attn_tc((const bf16*)qkv, L.nqkv, T, L.nq, L.nkv, L.hd, cu_dev, attn_sched, attn_items, attn_tiles,
                                       (bf16*)attn, L.dq, ctx.status, ctx.st, ctx.n_launch, hp, (bf16*)attn_lo);
        if (e != cudaSuccess && tc_err == cudaSuccess) tc_err = e;
      } else {
        if (hp) return fail(h, KVP_ERR_CUDA, "internal: the tensor-core attention refused the training-time forward");
        launch_attn_prefill_simt(ctx, qkv, L.nqkv, L.nq, L.nkv, L.hd, cu_dev, batch, T, attn, L.dq);
      }
      TcGemm to{};
      to.A = (const bf16*)attn; to.lda = L.dq; to.W = (const bf16*)(P + L.wo); to.ldw = L.dq; to.M = T; to.N = B.d; to.K = L.dq;
      to.epi = TC_RESID; to.X = x; to.ldx = B.d;
      if (hp) { to.A2 = (const bf16*)attn_lo; to.lda2 = L.dq; to.split_begin = 0; }
      if (!try_tc(h, ctx, to, KVP_CLASS_OTHER, &tc_err)) {
        if (hp) return fail(h, KVP_ERR_CUDA, "internal: the tensor-core kernel refused a projection of the training-time forward");
        GemmArgs o{};
        o.A = attn; o.lda = L.dq; o.W = P + L.wo; o.ldw = L.dq; o.M = T; o.N = B.d; o.K = L.dq; o.X = x; o.ldx = B.d;
        launch_gemm_simt(ctx, o, EPI_RESID);
      }
      launch_rmsnorm(ctx, x, (const float*)(P + L.ffn_norm), B.eps, T, B.d, hbuf, h->opt.dtype, hp ? h_lo : nullptr);
      TcGemm tf{};
      tf.A = (const bf16*)hbuf; tf.lda = B.d; tf.W = (const bf16*)(P + L.wgu); tf.ldw = B.d; tf.M = T; tf.N = 2 * L.ffn; tf.K = B.d;
      tf.epi = TC_SWIGLU; tf.C = (bf16*)act; tf.ldc = L.ffn; tf.ffn = L.G == 64 ? L.ffn : 1;
      if (hp) { tf.A2 = (const bf16*)h_lo; tf.lda2 = B.d; tf.split_begin = 0; tf.C_lo = (bf16*)act_lo; tf.ld_lo = L.ffn; }
      if (!try_tc(h, ctx, tf, KVP_CLASS_OTHER, &tc_err)) {
        if (hp) return fail(h, KVP_ERR_CUDA, "internal: the tensor-core kernel refused a projection of the training-time forward");
        GemmArgs f{};
        f.A = hbuf; f.lda = B.d; f.W = P + L.wgu; f.ldw = B.d; f.M = T; f.N = 2 * L.ffn; f.K = B.d; f.C = gu; f.ldc = 2 * L.ffn;
        launch_gemm_simt(ctx, f, EPI_STORE);
        launch_swiglu(ctx, gu, T, L.ffn, L.G, act);
      }
      TcGemm td{};
      td.A = (const bf16*)act; td.lda = L.ffn; td.W = (const bf16*)(P + L.wd); td.ldw = L.ffn; td.M = T; td.N = B.d; td.K = L.ffn;
      td.epi = TC_RESID; td.X = x; td.ldx = B.d;
      if (hp) { td.A2 = (const bf16*)act_lo; td.lda2 = L.ffn; td.split_begin = 0; }
      if (!try_tc(h, ctx, td, KVP_CLASS_OTHER, &tc_err)) {
        if (hp) return fail(h, KVP_ERR_CUDA, "internal: the tensor-core kernel refused a projection of the training-time forward");
        GemmArgs d{};
        d.A = act; d.lda = L.ffn; d.W = P + L.wd; d.ldw = L.ffn; d.M = T; d.N = B.d; d.K = L.ffn; d.X = x; d.ldx = B.d;
        launch_gemm_simt(ctx, d, EPI_RESID);
      }
    }
  }
  if (logits_out) {      // logits of every position: final norm, LM head (accumulated onto zeros by the residual epilogue)
    launch_rmsnorm(ctx, x, (const float*)(P + B.final_norm), B.eps, T, B.d, hbuf, h->opt.dtype, hp ? h_lo : nullptr);
    cudaMemsetAsync(logits_out, 0, (size_t)T * B.vocab * 4, s);
    TcGemm tl{};
    tl.A = (const bf16*)hbuf; tl.lda = B.d; tl.W = (const bf16*)(P + B.lm_head); tl.ldw = B.d; tl.M = T; tl.N = B.vocab; tl.K = B.d;
    tl.epi = TC_RESID; tl.X = logits_out; tl.ldx = B.vocab;
    if (hp) { tl.A2 = (const bf16*)h_lo; tl.lda2 = B.d; tl.split_begin = 0; }
    if (!try_tc(h, ctx, tl, KVP_CLASS_OTHER, &tc_err)) {
      GemmArgs g{};
      g.A = hbuf; g.lda = B.d; g.W = P + B.lm_head; g.ldw = B.d; g.M = T; g.N = B.vocab; g.K = B.d; g.X = logits_out; g.ldx = B.vocab;
      launch_gemm_simt(ctx, g, EPI_RESID);
    }
  }
  if (tc_err != cudaSuccess) return fail(h, KVP_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(tc_err));
  return check_cuda(h, "kvp_train_forward");
}
