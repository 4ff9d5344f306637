// Host-side plan of the KV Prediction library: shapes, packed-weight offsets, workspace layout.
#pragma once
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <unordered_set>
#include <vector>

#include "../../include/kvp.h"
#include "common.cuh"

struct LayerPlan {
  int nq, nkv, hd, ffn;
  int dq, dkv, nqkv;   // nq*hd, nkv*hd, (nq + 2 nkv)*hd
  int G;               // gate/up row interleave of the packed w_gate/w_up (0 = [gate; up])
  size_t wqkv, wo, wgu, wd, attn_norm, ffn_norm;   // byte offsets into the packed buffer
  size_t q_norm, k_norm;                           // query / key norm gains (fp32 [hd]); only with qk_norm
};

struct ModelPlan {
  int n_layers, d, vocab;
  float theta, eps;
  bool qk_norm;
  std::vector<LayerPlan> L;
  size_t embed, final_norm, lm_head;
  int max_nqkv, max_dq, max_dkv, max_ffn, max_group, max_nkv;
};

// All base layers predicted from one auxiliary layer: their FK (and FV) matrices are stored
// one under the other so that one GEMM produces every predicted K (or V) of that group.
struct PredGroup {
  int n_seg;
  int base_layer[MAX_PRED_SEG];
  int col0[MAX_PRED_SEG + 1];
  int din;
  size_t fk, fv, bk, bv;
  bool half_path;     // FK / FV stored as IEEE halves; K_A / V_A reach the predictor as halves in one pass
};

struct PackSlot {
  size_t off;      // destination byte offset of row 0 / element 0
  int rows, cols;  // expected source shape (rows = 1 for vectors)
  int dst_dtype;   // 0 f32, 1 bf16, 2 IEEE half
  RowMap map;
};

struct WsLayout {
  size_t status, cu, last_idx, tok_pos, tok_slot, rope_tab, x, h, h_lo, qkv, qkv32, kv_lo, attn, gu, act;
  size_t xb, hb, qkvb, ab, actb, part, tok_stage, first_stage, xbt, gub, attn_sched, attn_done, norm_ss, total;
};

struct kvp_handle {
  ModelPlan aux, base;
  std::vector<int> map;
  int j_max;
  kvp_options opt;
  int es;                               // element size of the run dtype
  std::vector<PredGroup> groups;        // one per auxiliary layer 0..j_max
  // Auxiliary layers whose QKV projection takes its operands as IEEE halves: the normalised input is written once as
  // halves (11 significant bits) instead of a bf16 value plus remainder, W_q / W_k / W_v are stored as halves, and the
  // K / V columns need no second pass.
  std::vector<uint8_t> qkv_half;
  std::unordered_map<std::string, PackSlot> slots;
  std::vector<std::string> req_prefill, req_decode_extra;
  std::unordered_set<std::string> loaded;
  bool ready_prefill = false, ready_decode = false;
  size_t packed_bytes = 0;
  char* packed = nullptr;
  int device = 0;
  int n_sm = 148;
  int64_t n_launch = 0;
  std::string err;
  // captured kernel schedules of kvp_prefill_predict, keyed by every argument that is baked in
  struct GraphEntry { std::vector<uint64_t> key; cudaGraphExec_t exec; int64_t launches; uint64_t last_use; };
  std::vector<GraphEntry> graphs;
  bool use_graph = true;
  uint64_t graph_clock = 0;
  // The predictor GEMMs of an auxiliary layer depend only on that layer's K/V projection, so they
  // run on a stream of the handle's own beside the layer's attention and FFN (fork / join by events).
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // The base step at small batch is one persistent kernel bound by HBM latency, the auxiliary prefill a chain
  // of tensor-core kernels: base layer i only needs the predicted cache of layers <= i, so the step runs in
  // pieces (one per auxiliary layer that completes some base layers' cache) on a stream of its own, on
  // `step_sms` SMs, while the prefill's kernels size their grids for the others.  0 = the step runs after the prefill.
  cudaStream_t step_st = nullptr;
  cudaEvent_t ev_step = nullptr;
  int step_sms = 72;
  int gemm_sms = 148;                   // SMs the tensor-core GEMMs of the current call size their grids for
  int step_tc_sms = 96;                 // grid of the step's projections when its per-layer kernels (batch > 4) run beside the prefill
  int step_grid_sms = 148;              // SMs the step's tensor-core projections size their grids for
  // instrumentation
  struct TimingRec { int cls; int64_t launches; cudaEvent_t a, b; };
  bool timing = false;
  std::vector<TimingRec> recs;
  std::vector<cudaEvent_t> free_events;
  ~kvp_handle() {
    for (auto& r : recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (auto e : free_events) cudaEventDestroy(e);
    for (auto& g : graphs) cudaGraphExecDestroy(g.exec);
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ev_join) cudaEventDestroy(ev_join);
    if (side) cudaStreamDestroy(side);
    if (ev_step) cudaEventDestroy(ev_step);
    if (step_st) cudaStreamDestroy(step_st);
  }
};

// Brackets the launches issued by `body` with events when instrumentation is on.
struct TimedScope {
  kvp_handle* h; cudaStream_t st; int cls; int64_t n0; cudaEvent_t a = nullptr, b = nullptr;
  static cudaEvent_t get(kvp_handle* h) {
    if (!h->free_events.empty()) { cudaEvent_t e = h->free_events.back(); h->free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  TimedScope(kvp_handle* h_, cudaStream_t s, int c) : h(h_), st(s), cls(c), n0(h_->n_launch) {
    if (h->timing) { a = get(h); b = get(h); cudaEventRecord(a, st); }
  }
  ~TimedScope() {
    if (a) { cudaEventRecord(b, st); h->recs.push_back({cls, h->n_launch - n0, a, b}); }
  }
};
#define KVP_TIMED(cls, stmt) do { TimedScope _ts(h, ctx.st, cls); stmt; } while (0)
