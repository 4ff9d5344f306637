/*
 * kvp.h - C ABI of the KV Prediction time-to-first-token library (CUDA, sm_100a).
 *
 * The library runs the inference algorithm of KV Prediction (arXiv 2410.08391,
 * Fig. 2(b) "KV Prediction Inference", Sec. 4.1 "Inference"):
 *
 *     a, KV_A  <- A(I)                auxiliary model over the whole prompt
 *     KV_B_hat <- P(KV_A)             per-base-layer linear maps (Sec. 4.2)
 *     b        <- B(I[-1], KV_B_hat)  one base-model step on the predicted cache
 *     loop:  b, p <- B(I[-1], KV_B_hat);  KV_B_hat <- KV_B_hat + p
 *
 * General conventions
 *   - Every call returns a kvp_status (0 = KVP_OK, negative = error).  Nothing
 *     throws or aborts.  State lives in the handle; the only process-wide state is a
 *     set of per-device flags (which kernels have had their shared-memory limit
 *     raised on which device) and the built-in scratch array of kvp_decode_step_static.
 *     kvp_last_error() returns a message owned by the handle, valid until the next
 *     call on that handle.
 *   - "dev" pointers are CUDA device pointers on the device that was current when
 *     kvp_create() ran; "host" pointers are ordinary host memory.
 *   - The caller owns ALL device memory (weights, packed weights, workspace, cache
 *     pools, block table, outputs).  The handle borrows the packed-weight pointer
 *     until kvp_destroy(); it owns host metadata, the CUDA graphs it records, and two
 *     internal streams with their events (created by kvp_create on the current device).
 *   - Calls that take a stream only enqueue work on it and return without
 *     synchronising (except the *_host variant, which synchronises the stream);
 *     arguments are validated on the host before anything is launched.
 *   - Device-side waits are bounded; a kernel that gives up, or that meets an
 *     out-of-range token id or page index, records a code in a status word inside
 *     the workspace and skips the access.  kvp_poll_status() reads it.  The status
 *     word is cleared by kvp_prefill_predict() at its start and by kvp_poll_status();
 *     poll once on a fresh workspace before using it for kvp_decode_step() alone.
 *   - Matrices are [out_features, in_features], row-major, dense.
 *   - Reproducibility: some projections add partial sums with fp32 atomic adds, so two runs
 *     on the same inputs agree up to fp32 reassociation (about 1e-6 relative in the fp32
 *     quantities, occasionally one unit in the last place of a stored 16-bit cache element), not bit for bit.
 */
#ifndef KVP_H_
#define KVP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t kvp_status;
enum {
  KVP_OK = 0,
  KVP_ERR_INVALID_ARG = -1, /* NULL pointer, bad enum, batch <= 0, length <= 0 ...          */
  KVP_ERR_SHAPE = -2,       /* tensor shape or model dimensions inconsistent                 */
  KVP_ERR_UNSUPPORTED = -3, /* valid but not implemented (e.g. odd head_dim)                 */
  KVP_ERR_NOT_LOADED = -4,  /* compute call before kvp_load_weights() supplied every tensor  */
  KVP_ERR_CACHE_FULL = -5,  /* prompt needs more pages than block table / pools provide      */
  KVP_ERR_CUDA = -6,        /* a CUDA runtime or driver call failed                          */
  KVP_ERR_TIMEOUT = -7,     /* a bounded device-side wait ran out                            */
  KVP_ERR_WORKSPACE = -8,   /* workspace or packed-weight buffer too small or misaligned     */
  KVP_ERR_BAD_INDEX = -9    /* device met a token id or page index out of range              */
};

enum { KVP_F32 = 0, KVP_BF16 = 1 };

#define KVP_MAX_BATCH 256

/* One transformer layer.  OpenELM-style models vary these per layer (Sec. 4.2
 * "OpenELM KV Prediction Specification": the KV cache width differs per layer). */
typedef struct {
  int32_t n_q_heads;  /* multiple of n_kv_heads                       */
  int32_t n_kv_heads; /* >= 1                                         */
  int32_t head_dim;   /* even; same for every layer of one model      */
  int32_t ffn_dim;    /* SwiGLU hidden width                          */
} kvp_layer_cfg;

/* A pre-norm decoder: RMSNorm -> GQA attention with RoPE (rotate-half pairing)
 * -> residual; RMSNorm -> SwiGLU FFN -> residual; final RMSNorm -> LM head. */
typedef struct {
  int32_t n_layers;
  int32_t d_model;
  int32_t vocab;
  float rope_theta;
  float rms_eps;
  int32_t qk_norm;             /* 1: queries and keys are RMS-normalised per head (over head_dim, eps = rms_eps,
                                  gains "L{l}.q_norm" / "L{l}.k_norm" [head_dim]) before RoPE: OpenELM's key norm
                                  (Sec. 7 "Analysis").  The cache then holds normalised, rotated keys. 0: off. */
  const kvp_layer_cfg* layers; /* host, [n_layers]; copied by kvp_create */
} kvp_model_cfg;

typedef struct {
  int32_t dtype;          /* KVP_F32 | KVP_BF16: storage type of weights and activations (tensor-core operands).
                             Accumulation, norms, softmax and the base step's activations are fp32.  The cache
                             holds fp32 elements in KVP_F32 mode and IEEE half elements in KVP_BF16 mode.    */
  int32_t page_tokens;    /* tokens per cache page; must be 64                                       */
  int32_t predictor_bias; /* 1: the predictor has bias vectors pred.L{i}.bk / bv                     */
  int32_t flags;          /* 0, or a sum of KVP_OPT_* (kernel variants; results are the same within rounding) */
} kvp_options;

/* Schedule variants (results are the same within rounding; the design notes give the measurements):
 *   KVP_OPT_FUSED_KV_PRED  the K/V projection of an auxiliary layer and the KV predictor as ONE kernel (the predictor
 *                          is the projection's epilogue; K_A / V_A reach it through shared memory), used for calls
 *                          with at least one 128-token block per SM.  Off by default: it measured slower than the
 *                          projection GEMM followed by a predictor GEMM.
 *   KVP_OPT_SEPARATE_NORM  RMSNorm as a kernel of its own in front of every projection.  By default, wherever every
 *                          output tile of the residual GEMMs belongs to one CTA (calls of some thousand tokens and
 *                          more), RMSNorm is folded into the GEMMs around it: the residual GEMM that completes x also
 *                          writes x * gain as the next GEMM's 16-bit operand and the rows' sums of squares, the next GEMM
 *                          scales its rows by 1 / rms. */
enum { KVP_OPT_FUSED_KV_PRED = 1, KVP_OPT_SEPARATE_NORM = 2 };

/* A named tensor handed to kvp_load_weights().  Names:
 *   "aux.embed" [vocab, d_A]
 *   "aux.L{j}.attn_norm" [d_A]   "aux.L{j}.ffn_norm" [d_A]
 *   "aux.L{j}.wq" [nq*hd, d_A]   "aux.L{j}.wk" / "wv" [nkv*hd, d_A]   "aux.L{j}.wo" [d_A, nq*hd]
 *   "aux.L{j}.w_gate" / "w_up" [ffn, d_A]   "aux.L{j}.w_down" [d_A, ffn]
 *   with qk_norm: "aux.L{j}.q_norm" [hd] and "aux.L{j}.k_norm" [hd]
 *   the same under "base.", plus "base.final_norm" [d_B] and "base.lm_head" [vocab, d_B]
 *   "pred.L{i}.fk" / "fv" [d_kvB_i, d_kvA_{j_i}]  and, with predictor_bias, "pred.L{i}.bk" / "bv" [d_kvB_i]
 * Auxiliary layers above max_i j_i, "aux.final_norm" and "aux.lm_head" are never read
 * (the auxiliary logits are unused at inference, Sec. 4.3) and may be omitted. */
typedef struct {
  const char* name;
  const void* data;  /* dev, dense row-major                      */
  int32_t dtype;     /* KVP_F32 | KVP_BF16 (converted on load)    */
  int32_t ndim;      /* 1 or 2                                    */
  int64_t shape[2];
} kvp_tensor;

/* The paged base-model KV cache, the user-visible product of prefill (Sec. 4.1:
 * the predicted cache is what the base model's attention then consumes).
 * Base layer i has one K pool and one V pool of n_pages pages; a page is
 * [n_kv_heads_i][page_tokens][head_dim] elements: fp32 in KVP_F32 mode; in KVP_BF16 mode 16-bit IEEE half
 * (fp16: 11 significant bits, stores saturate at +-65504), not bfloat16: the cache is the product of the path
 * and the base model's step amplifies its rounding several times in the logits.  Entry t of
 * sequence b lives in page block_table[b * max_pages_per_seq + t / page_tokens]
 * at row t % page_tokens, in every layer's pools.  Keys are stored after RoPE.
 * Rows at or beyond a sequence's length are unspecified. */
typedef struct {
  void* const* k_pools;        /* host array [n_base_layers] of dev pointers            */
  void* const* v_pools;        /* host array [n_base_layers] of dev pointers            */
  const int32_t* block_table;  /* dev, [>= batch][max_pages_per_seq], filled by caller  */
  int32_t* seq_lens;           /* dev, [>= batch]; written by prefill, +1 per decode    */
  int32_t max_pages_per_seq;
  int32_t n_pages;             /* pages in every pool                                   */
} kvp_cache;

typedef struct kvp_handle kvp_handle;

/* Validates both models and the layer map j_i (Sec. 4.2: j_i in [0, n_A), here also
 * required non-decreasing; both models share one vocabulary) and builds the kernel
 * plan.  aux/base/layer_map/opt: host.  *out receives the handle. */
kvp_status kvp_create(const kvp_model_cfg* aux, const kvp_model_cfg* base,
                      const int32_t* layer_map /* host [base->n_layers] */,
                      const kvp_options* opt, kvp_handle** out);

void kvp_destroy(kvp_handle* h);

/* NUL-terminated description of the last error on this handle ("" if none). */
const char* kvp_last_error(const kvp_handle* h);

/* Layer-map helpers (Sec. 4.2 and Table 1): write j_0..j_{n_base-1} to out (host).
 * canonical: consecutive base layers share an aux layer, the first n_base mod n_aux aux
 *            layers feed one more base layer than the rest (the KVP-C rows of Table 1);
 * pruned:    aux = base with only `retained` layers kept (ascending, retained[0] == 0);
 *            j_i = index of the largest retained layer <= i (the KVP-LP rows);
 * uniform:   j_i = floor(i * n_aux / n_base). */
kvp_status kvp_layer_map_canonical(int32_t n_base, int32_t n_aux, int32_t* out);
kvp_status kvp_layer_map_pruned(int32_t n_base, const int32_t* retained, int32_t n_aux, int32_t* out);
kvp_status kvp_layer_map_uniform(int32_t n_base, int32_t n_aux, int32_t* out);

/* Bytes of the packed-weight buffer kvp_load_weights() fills (256-byte aligned dev memory). */
kvp_status kvp_packed_weight_bytes(const kvp_handle* h, size_t* bytes);

/* Bytes of workspace for calls with batch <= max_batch and sum of lengths <= max_total_tokens. */
kvp_status kvp_workspace_bytes(const kvp_handle* h, int32_t max_batch, int64_t max_total_tokens,
                               size_t* bytes);

/* Bytes of one page of base layer `base_layer` (K or V; both are equal). */
kvp_status kvp_cache_layout(const kvp_handle* h, int32_t base_layer, size_t* bytes_per_page);

/* Converts and re-lays-out the n given tensors into `packed` (dev) with kernels enqueued on
 * `stream`.  May be called several times with disjoint subsets; compute calls need every
 * required tensor.  Once the enqueued work has finished the source tensors may be freed;
 * `packed` must stay alive until kvp_destroy().  Shape or name mismatch -> KVP_ERR_SHAPE. */
kvp_status kvp_load_weights(kvp_handle* h, const kvp_tensor* tensors, int32_t n,
                            void* packed, size_t packed_bytes, void* stream);

/* The time-to-first-token path (Fig. 2(b), first three statements): auxiliary prefill over
 * all prompts, KV prediction into the paged cache, one base step per sequence on its last
 * prompt token at position L_b - 1 attending to predicted entries 0..L_b-1 (nothing is
 * appended; the base K/V projections are unused).
 *   tokens        dev  int32 [sum(lengths)]  prompts packed back to back
 *   lengths       host int32 [batch]         each >= 1
 *   cache              pools and block table as described above; seq_lens[b] <- L_b
 *   workspace     dev, 256-byte aligned, >= kvp_workspace_bytes(batch, sum(lengths))
 *   logits_out    dev  fp32 [batch, vocab]
 *   first_token   dev  int32 [batch], argmax of logits (lowest index on ties); may be NULL
 * The first call with a given set of arguments (pointers, lengths, stream) records the kernel
 * schedule into a CUDA graph owned by the handle; later calls with the same arguments replay it
 * (the token values themselves may change between calls).  If `stream` is already being
 * captured by the caller, the kernels are enqueued into the caller's capture instead.
 * For short prompts part of the work is enqueued on the handle's internal streams, forked from
 * and joined back into `stream` with events: the predictor of an auxiliary layer beside that
 * layer's attention and FFN, and (batch <= 4) the base model's step in pieces, each as soon as the
 * predicted cache of its layers is complete (Fig. 2(b): B needs only the predicted cache).  From
 * the caller's point of view everything is ordered on `stream` as usual. */
kvp_status kvp_prefill_predict(kvp_handle* h, const int32_t* tokens, const int32_t* lengths,
                               int32_t batch, const kvp_cache* cache, void* workspace,
                               size_t workspace_bytes, float* logits_out, int32_t* first_token,
                               void* stream);

/* Same path with HOST tokens and HOST outputs: copies the tokens to the device, runs
 * kvp_prefill_predict, copies logits (if logits_host != NULL) and first tokens back and
 * synchronises `stream`.  The token staging area lives at the end of the workspace
 * (accounted for by kvp_workspace_bytes); logits_dev is a dev scratch [batch, vocab]. */
kvp_status kvp_prefill_predict_host(kvp_handle* h, const int32_t* tokens_host,
                                    const int32_t* lengths, int32_t batch, const kvp_cache* cache,
                                    void* workspace, size_t workspace_bytes, float* logits_dev,
                                    float* logits_host, int32_t* first_token_host, void* stream);

/* One generation step (Fig. 2(b), loop body): for every sequence the base model computes
 * q, k, v of `tokens[b]` with its own projections at position seq_lens[b], appends k
 * (after RoPE) and v to the cache, attends over seq_lens[b] + 1 entries and emits logits;
 * seq_lens[b] += 1.  lengths_host[b] must equal the current seq_lens[b] (host copy used
 * for validation and scheduling).  KVP_ERR_CACHE_FULL if a sequence has no room left.
 * The call may be recorded into a CUDA graph by the caller (stream capture) and replayed for the
 * following steps: the kernels read positions from seq_lens and the token from `tokens` on the
 * device; lengths_host only sizes the key-range splits and checks capacity at recording time, so
 * the caller has to make sure that the block table has pages for every replayed step (the choice
 * of kernels and splits stays the one made for the recorded length). */
kvp_status kvp_decode_step(kvp_handle* h, const int32_t* tokens /* dev [batch] */,
                           const int32_t* lengths_host, int32_t batch, const kvp_cache* cache,
                           void* workspace, size_t workspace_bytes, float* logits_out,
                           int32_t* next_token, void* stream);

/* (The paper has no counterpart to this call: it exists for the library's users.)
 * kvp_decode_step for callers that must not allocate device memory and therefore have no
 * workspace to pass: code running while a CUDA memory pool is frozen, inside a latency-critical
 * serving loop where cudaMalloc would synchronise the whole device, or in a plug-in whose host
 * application owns the allocator.  Same inputs, outputs and semantics as kvp_decode_step, but
 * the step's scratch is a fixed array of KVP_STATIC_SCRATCH_BYTES inside the library image
 * (every GPU that loads the library holds it until the process exits).  The call itself
 * performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   - A step whose kvp_workspace_bytes(h, batch, batch) exceeds KVP_STATIC_SCRATCH_BYTES is
 *     rejected with KVP_ERR_WORKSPACE and a message naming both sizes.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before any stream capture begins.  Arguments are checked
 *     before the array or the stream is touched.
 *   - All calls on a device share the one array, which keeps the previous call's contents.
 *     The call clears the status word itself; everything else is overwritten before it is
 *     read.  Two calls that overlap on the GPU (different streams or handles) race on the
 *     array: keep them on one stream or order them with events.
 *   - status_out (dev int32, may be NULL) receives the device status word of this step:
 *     0 = ok, 1 = a wait ran out, 2 = bad token id, 3 = bad page index. */
#define KVP_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
kvp_status kvp_decode_step_static(kvp_handle* h, const int32_t* tokens /* dev [batch] */,
                                  const int32_t* lengths_host, int32_t batch, const kvp_cache* cache,
                                  float* logits_out, int32_t* next_token, int32_t* status_out,
                                  void* stream);

/* Training-time forward, no backward (Sec. 4.1 "Training", Fig. 2(a); consistency loss of Sec. 4.3).
 * To be called after kvp_prefill_predict for the same tokens / lengths / cache: the cache then holds
 * the predicted K_hat_i, V_hat_i of the whole prompt.  Two passes of the base model over ALL prompt tokens:
 *   (1) its ordinary forward, whose own keys (after RoPE) and values are the target cache KV_B:
 *       l1_k[i] = mean over tokens and columns of |K_hat_i - K_B,i|, l1_v[i] likewise (dev fp32 [n_base_layers]);
 *       the paper's L_C is their sum (lambda_C = 1) or mean (lambda_C = 1 / n_B) over i, K and V together;
 *   (2) the forward in which every layer's attention reads the predicted cache instead of the layer's own
 *       keys and values (query t sees predicted entries 0..t: "masked cross-attention"):
 *       logits_out = dev fp32 [sum(lengths), vocab], row t = logits after token t (the input of the paper's
 *       base loss L_B); may be NULL, then pass (2) is skipped.
 * The predicted cache is read in its own element type (IEEE halves in KVP_BF16 mode, fp32 in KVP_F32 mode).  The cache and seq_lens are not
 * changed.  workspace: dev, 256-byte aligned, >= kvp_train_workspace_bytes(batch, sum(lengths)) (its own
 * layout: base-model widths for every token).  Launches kernel by kernel on `stream`, no synchronisation.
 * Needs every base tensor including wk / wv.  Errors as kvp_prefill_predict. */
kvp_status kvp_train_workspace_bytes(const kvp_handle* h, int32_t max_batch, int64_t max_total_tokens, size_t* bytes);
kvp_status kvp_train_forward(kvp_handle* h, const int32_t* tokens /* dev [sum(lengths)] */, const int32_t* lengths /* host */,
                             int32_t batch, const kvp_cache* cache, void* workspace, size_t workspace_bytes,
                             float* logits_out, float* l1_k, float* l1_v, void* stream);

/* Synchronises `stream`, reads the device status word of `workspace`, clears it and returns
 * KVP_OK, KVP_ERR_TIMEOUT, KVP_ERR_BAD_INDEX or KVP_ERR_CUDA. */
kvp_status kvp_poll_status(kvp_handle* h, void* workspace, void* stream);

/* Self-test of the error path behind KVP_ERR_TIMEOUT (the paper has no counterpart).  Enqueues a one-block
 * kernel that waits, with the same bounded wait every kernel of the library uses but a limit of a few thousand
 * polls, on a barrier that nothing completes.  The wait runs out, the kernel returns normally and records its code
 * in the status word of `workspace` (dev, >= 16 bytes, as passed to the compute calls); kvp_poll_status then
 * returns KVP_ERR_TIMEOUT and clears the word, and the handle and the context stay usable. */
kvp_status kvp_selftest_wait_timeout(kvp_handle* h, void* workspace, void* stream);

/* Number of kernels the handle launched since creation (for launch accounting). */
int64_t kvp_launch_count(const kvp_handle* h);

/* Instrumentation (not part of the method): per-kernel-class device timing.  While enabled,
 * every kernel launch of the compute calls is bracketed by CUDA events on the call's stream.
 * kvp_timing_read() waits for the recorded events, adds their durations per class into
 * ms[KVP_N_CLASSES] (host) and the launch counts into launches[KVP_N_CLASSES] (host), and
 * forgets them.  Classes: the KVP_CLASS_* constants.  Events are owned by the handle. */
enum {
  KVP_CLASS_AUX_GEMM = 0,   /* auxiliary QKV / O / gate-up / down projections            */
  KVP_CLASS_AUX_ATTN = 1,   /* auxiliary causal attention                                 */
  KVP_CLASS_PREDICTOR = 2,  /* predictor GEMM writing the paged base cache                */
  KVP_CLASS_STEP_GEMV = 3,  /* base step: weight-streaming projections and LM head        */
  KVP_CLASS_STEP_ATTN = 4,  /* base step: attention over the paged cache                  */
  KVP_CLASS_OTHER = 5,      /* norms, RoPE, SwiGLU, gathers, index, argmax                */
  KVP_CLASS_STEP_FUSED = 6, /* base step as one persistent kernel (batch <= 4)            */
  KVP_CLASS_KV_PRED = 7,    /* auxiliary K/V projection with the predictor as its epilogue */
  KVP_N_CLASSES = 8
};
kvp_status kvp_timing_enable(kvp_handle* h, int32_t on);
kvp_status kvp_timing_read(kvp_handle* h, double* ms, int64_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* KVP_H_ */
