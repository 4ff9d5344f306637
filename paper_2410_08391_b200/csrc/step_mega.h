// Host interface of the persistent single-token step kernel.
#pragma once
#include "common.cuh"

constexpr int MEGA_MAX_LAYERS = 64;
constexpr int MEGA_COUNTERS = 32;      // grid-barrier counter words in the status block (one per launch of a step)
constexpr int MEGA_STATUS_BYTES = 256; // what a caller clears before a step: status word, argmax slots, counters

struct MegaLayer {
  const void *wqkv, *wo, *wgu, *wd;      // packed weights of the layer (run dtype)
  const float *attn_norm, *ffn_norm;
  const float *q_norm, *k_norm;          // query / key norm gains [hd], or null
  void *kpool, *vpool;                   // cache pools of the layer
  int nq, nkv, dq, nqkv, ffn, G;
};

struct MegaParams {
  int n_layers, d, vocab, hd, batch, generation, n_split;
  float eps;
  InvFreq inv;
  const int* tokens; const int* gather_idx;      // token of row b = tokens[gather_idx ? gather_idx[b] : b]
  const void* embed; const float* final_norm; const void* lm_head;
  const int* block_table; int mpps, n_pages;
  int* seq_lens;
  float *xb, *qkvb, *ab, *actb, *part;           // workspace: residual, projections, attention out, FFN act, partials
  int* attn_done;                                // [batch * max n_kv] splits finished per (sequence, kv head); zero on entry, left zero
  float* logits; int* token_out;
  // One launch may cover only base layers [layer_begin, layer_end): the residual stream stays in xb between
  // launches.  do_embed: start from the token embeddings; do_head: end with the LM head and the token.
  int layer_begin, layer_end, do_embed, do_head;
  int counter_idx;                               // which grid-barrier counter word this launch uses (zero on entry)
  int stage_bytes, slot_bytes;                   // shared-memory plan (set by the launcher)
  long long* trace;                              // optional: clock64 of CTA 0 around every barrier (debugging aid)
  int* status;                                   // [0] status word, +64 bytes: argmax slots, +128 bytes: MEGA_COUNTERS barrier counters
  MegaLayer layers[MEGA_MAX_LAYERS];
};

bool step_mega_supported(int batch, int hd, int k_max, int max_group, int es);
cudaError_t launch_step_mega(MegaParams p, int dtype, int k_max, int n_sm, cudaStream_t st, int64_t* n_launch);
