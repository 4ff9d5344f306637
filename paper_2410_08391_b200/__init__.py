"""KV Prediction time-to-first-token path on one B200 (sm_100a): thin Python binding over the
C-ABI library `libkvp.so`.  Every step of the path runs in the library's CUDA kernels; this
package only marshals arguments.  Importing it does not load the library; `binding.lib()`
does, and raises if the library has not been built."""
from . import binding  # noqa: F401
from .binding import (KVP_OPT_FUSED_KV_PRED, KVP_OPT_SEPARATE_NORM, KvpError, Session, kvp_cache_layout, kvp_create, kvp_decode_step, kvp_decode_step_static, kvp_destroy,  # noqa: F401
                      kvp_last_error, kvp_launch_count, kvp_layer_map_canonical, kvp_layer_map_pruned,
                      kvp_layer_map_uniform, kvp_load_weights, kvp_packed_weight_bytes, kvp_poll_status,
                      kvp_prefill_predict, kvp_prefill_predict_host, kvp_selftest_wait_timeout, kvp_timing_enable, kvp_timing_read,
                      kvp_train_forward, kvp_train_workspace_bytes, kvp_workspace_bytes, lib)
