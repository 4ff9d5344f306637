// Generation step for callers that cannot provide a workspace: the step's scratch (activations of
// the current token, split-attention partials, status word) lives in a fixed device array that
// is part of the library image.
#include <stdio.h>

#include "kvp_internal.h"

// One array per GPU that loads the library, held from module load until the process exits.
static __device__ __align__(256) unsigned char g_step_scratch[KVP_STATIC_SCRATCH_BYTES];

namespace {
constexpr int MAX_DEVICES = 64;
// Device address of g_step_scratch per device ordinal.  In host code the name `g_step_scratch`
// is only a handle for the runtime's symbol lookup, never a pointer a kernel may be given.
void* g_scratch_addr[MAX_DEVICES] = {};
}  // namespace

extern "C" kvp_status kvp_decode_step_static(kvp_handle* h, const int32_t* tokens, const int32_t* lengths_host,
                                             int32_t batch, const kvp_cache* cache, float* logits_out,
                                             int32_t* next_token, int32_t* status_out, void* stream) {
  if (!h) return KVP_ERR_INVALID_ARG;
  h->err.clear();
  if (batch <= 0 || batch > KVP_MAX_BATCH) {
    h->err = "batch outside [1, KVP_MAX_BATCH]";
    return KVP_ERR_INVALID_ARG;
  }
  size_t need = 0;
  kvp_status st = kvp_workspace_bytes(h, batch, batch, &need);
  if (st != KVP_OK) return st;
  if (need > (size_t)KVP_STATIC_SCRATCH_BYTES) {
    char buf[256];
    snprintf(buf, sizeof buf,
             "kvp_decode_step_static: a step of batch %d needs %zu bytes of scratch, the built-in array holds %d; "
             "use kvp_decode_step with a caller-provided workspace",
             batch, need, KVP_STATIC_SCRATCH_BYTES);
    h->err = buf;
    return KVP_ERR_WORKSPACE;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    cudaGetLastError();
    h->err = "kvp_decode_step_static: no usable current device";
    return KVP_ERR_CUDA;
  }
  // nothing touches the array or the stream before the arguments have been checked
  if (dev != h->device) {
    h->err = "kvp_decode_step_static: the current device is not the handle's device";
    return KVP_ERR_INVALID_ARG;
  }
  if (!tokens || !lengths_host || !cache || !logits_out || !cache->k_pools || !cache->v_pools || !cache->block_table ||
      !cache->seq_lens) {
    h->err = "kvp_decode_step_static: NULL argument";
    return KVP_ERR_INVALID_ARG;
  }
  if (!h->ready_decode) {
    h->err = "kvp_load_weights has not supplied every required tensor";
    return KVP_ERR_NOT_LOADED;
  }
  // Set-up, once per device, with that device current.  Two threads making their first call on a device at the
  // same moment both look the address up and store the same value.
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_step_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      h->err = std::string("kvp_decode_step_static: cudaGetSymbolAddress failed: ") + cudaGetErrorString(e);
      return KVP_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  void* ws = g_scratch_addr[dev];
  cudaStream_t s = (cudaStream_t)stream;
  // The array keeps whatever the previous call left.  Only the status word has to start at zero;
  // every other region is written by this step before it is read.
  if (cudaMemsetAsync(ws, 0, 16, s) != cudaSuccess) {
    h->err = std::string("kvp_decode_step_static: ") + cudaGetErrorString(cudaGetLastError());
    return KVP_ERR_CUDA;
  }
  st = kvp_decode_step(h, tokens, lengths_host, batch, cache, ws, (size_t)KVP_STATIC_SCRATCH_BYTES, logits_out,
                       next_token, stream);
  if (st != KVP_OK) return st;
  if (status_out && cudaMemcpyAsync(status_out, ws, 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess) {
    h->err = std::string("kvp_decode_step_static: ") + cudaGetErrorString(cudaGetLastError());
    return KVP_ERR_CUDA;
  }
  return KVP_OK;
}
