"""ctypes binding of include/kvp.h.  The functions carry the C names and only marshal
arguments; `Session` adds the device-memory plumbing (torch allocates, the library computes).
There is no CPU fallback: if libkvp.so is missing or no CUDA device is present, calls raise."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvp.so")

KVP_OK = 0
KVP_F32, KVP_BF16 = 0, 1
STATUS_NAMES = {0: "KVP_OK", -1: "KVP_ERR_INVALID_ARG", -2: "KVP_ERR_SHAPE", -3: "KVP_ERR_UNSUPPORTED",
                -4: "KVP_ERR_NOT_LOADED", -5: "KVP_ERR_CACHE_FULL", -6: "KVP_ERR_CUDA", -7: "KVP_ERR_TIMEOUT",
                -8: "KVP_ERR_WORKSPACE", -9: "KVP_ERR_BAD_INDEX"}


class KvpError(RuntimeError):
    def __init__(self, status: int, msg: str = ""):
        self.status = status
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")


class LayerCfgC(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn_dim", C.c_int32)]


class ModelCfgC(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("vocab", C.c_int32), ("rope_theta", C.c_float),
                ("rms_eps", C.c_float), ("qk_norm", C.c_int32), ("layers", C.POINTER(LayerCfgC))]


class OptionsC(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("page_tokens", C.c_int32), ("predictor_bias", C.c_int32), ("flags", C.c_int32)]


class TensorC(C.Structure):
    _fields_ = [("name", C.c_char_p), ("data", C.c_void_p), ("dtype", C.c_int32), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 2)]


class CacheC(C.Structure):
    _fields_ = [("k_pools", C.POINTER(C.c_void_p)), ("v_pools", C.POINTER(C.c_void_p)), ("block_table", C.c_void_p),
                ("seq_lens", C.c_void_p), ("max_pages_per_seq", C.c_int32), ("n_pages", C.c_int32)]


EXPORTS = ["kvp_create", "kvp_destroy", "kvp_last_error", "kvp_layer_map_canonical", "kvp_layer_map_pruned",
           "kvp_layer_map_uniform", "kvp_packed_weight_bytes", "kvp_workspace_bytes", "kvp_cache_layout",
           "kvp_load_weights", "kvp_prefill_predict", "kvp_prefill_predict_host", "kvp_decode_step",
           "kvp_poll_status", "kvp_launch_count", "kvp_timing_enable", "kvp_timing_read",
           "kvp_decode_step_static", "kvp_train_workspace_bytes", "kvp_train_forward", "kvp_selftest_wait_timeout"]

CLASS_NAMES = ["aux_gemm", "aux_attn", "predictor", "step_gemv", "step_attn", "other", "step_fused", "kv_pred"]

_lib = None


def lib() -> C.CDLL:
    """Loads libkvp.so (once).  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2410_08391_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.kvp_create.argtypes = [C.POINTER(ModelCfgC), C.POINTER(ModelCfgC), C.POINTER(i32), C.POINTER(OptionsC), C.POINTER(vp)]
        L.kvp_destroy.argtypes = [vp]
        L.kvp_destroy.restype = None
        L.kvp_last_error.argtypes = [vp]
        L.kvp_last_error.restype = C.c_char_p
        L.kvp_layer_map_canonical.argtypes = [i32, i32, C.POINTER(i32)]
        L.kvp_layer_map_pruned.argtypes = [i32, C.POINTER(i32), i32, C.POINTER(i32)]
        L.kvp_layer_map_uniform.argtypes = [i32, i32, C.POINTER(i32)]
        L.kvp_packed_weight_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.kvp_workspace_bytes.argtypes = [vp, i32, i64, C.POINTER(C.c_size_t)]
        L.kvp_cache_layout.argtypes = [vp, i32, C.POINTER(C.c_size_t)]
        L.kvp_load_weights.argtypes = [vp, C.POINTER(TensorC), i32, vp, C.c_size_t, vp]
        L.kvp_prefill_predict.argtypes = [vp, vp, C.POINTER(i32), i32, C.POINTER(CacheC), vp, C.c_size_t, vp, vp, vp]
        L.kvp_prefill_predict_host.argtypes = [vp, vp, C.POINTER(i32), i32, C.POINTER(CacheC), vp, C.c_size_t, vp, vp, vp, vp]
        L.kvp_decode_step.argtypes = [vp, vp, C.POINTER(i32), i32, C.POINTER(CacheC), vp, C.c_size_t, vp, vp, vp]
        L.kvp_decode_step_static.argtypes = [vp, vp, C.POINTER(i32), i32, C.POINTER(CacheC), vp, vp, vp, vp]
        L.kvp_train_workspace_bytes.argtypes = [vp, i32, i64, C.POINTER(C.c_size_t)]
        L.kvp_train_forward.argtypes = [vp, vp, C.POINTER(i32), i32, C.POINTER(CacheC), vp, C.c_size_t, vp, vp, vp, vp]
        L.kvp_poll_status.argtypes = [vp, vp, vp]
        L.kvp_selftest_wait_timeout.argtypes = [vp, vp, vp]
        L.kvp_launch_count.argtypes = [vp]
        L.kvp_launch_count.restype = i64
        L.kvp_timing_enable.argtypes = [vp, i32]
        L.kvp_timing_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
        for n in EXPORTS:
            if n not in ("kvp_destroy", "kvp_last_error", "kvp_launch_count"):
                getattr(L, n).restype = i32
        _lib = L
    return _lib


def _check(st: int, h=None):
    if st != KVP_OK:
        msg = lib().kvp_last_error(h).decode() if h else ""
        raise KvpError(st, msg)


def _i32arr(v: Sequence[int]):
    return (C.c_int32 * len(v))(*[int(x) for x in v])


def _model_c(m):
    layers = (LayerCfgC * m.n_layers)(*[LayerCfgC(l.n_q_heads, l.n_kv_heads, l.head_dim, l.ffn_dim) for l in m.layers])
    return ModelCfgC(m.n_layers, m.d_model, m.vocab, m.rope_theta, m.rms_eps, 1 if getattr(m, "qk_norm", False) else 0, layers), layers


# ---- functions with the C names -------------------------------------------------------------
def kvp_layer_map_canonical(n_base: int, n_aux: int) -> List[int]:
    out = (C.c_int32 * max(n_base, 1))()
    _check(lib().kvp_layer_map_canonical(n_base, n_aux, out))
    return list(out)[:n_base]


def kvp_layer_map_pruned(n_base: int, retained: Sequence[int]) -> List[int]:
    out = (C.c_int32 * max(n_base, 1))()
    _check(lib().kvp_layer_map_pruned(n_base, _i32arr(retained), len(retained), out))
    return list(out)[:n_base]


def kvp_layer_map_uniform(n_base: int, n_aux: int) -> List[int]:
    out = (C.c_int32 * max(n_base, 1))()
    _check(lib().kvp_layer_map_uniform(n_base, n_aux, out))
    return list(out)[:n_base]


KVP_OPT_FUSED_KV_PRED, KVP_OPT_SEPARATE_NORM = 1, 2


def kvp_create(aux, base, layer_map: Sequence[int], dtype: str = "bf16", predictor_bias: bool = False,
               page_tokens: int = 64, flags: int = 0) -> int:
    a, _ka = _model_c(aux)
    b, _kb = _model_c(base)
    opt = OptionsC(KVP_BF16 if dtype == "bf16" else KVP_F32, page_tokens, int(predictor_bias), int(flags))
    h = C.c_void_p()
    _check(lib().kvp_create(C.byref(a), C.byref(b), _i32arr(layer_map), C.byref(opt), C.byref(h)))
    return h.value


def kvp_destroy(h) -> None:
    lib().kvp_destroy(h)


def kvp_last_error(h) -> str:
    return lib().kvp_last_error(h).decode()


def kvp_launch_count(h) -> int:
    return int(lib().kvp_launch_count(h))


def kvp_timing_enable(h, on: bool) -> None:
    _check(lib().kvp_timing_enable(h, int(on)), h)


def kvp_timing_read(h):
    """Returns {class name: (milliseconds, launches)} accumulated since the last read."""
    ms = (C.c_double * len(CLASS_NAMES))()
    n = (C.c_int64 * len(CLASS_NAMES))()
    _check(lib().kvp_timing_read(h, ms, n), h)
    return {c: (ms[i], int(n[i])) for i, c in enumerate(CLASS_NAMES)}


def kvp_packed_weight_bytes(h) -> int:
    n = C.c_size_t()
    _check(lib().kvp_packed_weight_bytes(h, C.byref(n)), h)
    return n.value


def kvp_workspace_bytes(h, max_batch: int, max_total_tokens: int) -> int:
    n = C.c_size_t()
    _check(lib().kvp_workspace_bytes(h, max_batch, max_total_tokens, C.byref(n)), h)
    return n.value


def kvp_cache_layout(h, base_layer: int) -> int:
    n = C.c_size_t()
    _check(lib().kvp_cache_layout(h, base_layer, C.byref(n)), h)
    return n.value


def kvp_load_weights(h, tensors: Dict[str, "object"], packed, stream: int) -> None:
    """tensors: name -> torch CUDA tensor (float32 or bfloat16, contiguous)."""
    import torch
    arr = (TensorC * len(tensors))()
    keep = []
    for i, (name, t) in enumerate(tensors.items()):
        assert t.is_cuda and t.is_contiguous()
        nb = name.encode()
        keep.append(nb)
        shp = (C.c_int64 * 2)(*(list(t.shape) + [0])[:2])
        arr[i] = TensorC(nb, t.data_ptr(), KVP_BF16 if t.dtype == torch.bfloat16 else KVP_F32, t.dim(), shp)
    _check(lib().kvp_load_weights(h, arr, len(tensors), packed.data_ptr(), packed.numel() * packed.element_size(), stream), h)


def _cache_c(cache: "Cache") -> CacheC:
    return CacheC(cache._kp, cache._vp, cache.block_table.data_ptr(), cache.seq_lens.data_ptr(),
                  cache.max_pages_per_seq, cache.n_pages)


def kvp_prefill_predict(h, tokens, lengths: Sequence[int], cache: "Cache", workspace, logits_out, first_token,
                        stream: int) -> None:
    cc = _cache_c(cache)
    _check(lib().kvp_prefill_predict(h, tokens.data_ptr(), _i32arr(lengths), len(lengths), C.byref(cc),
                                     workspace.data_ptr(), workspace.numel(), logits_out.data_ptr(),
                                     first_token.data_ptr() if first_token is not None else None, stream), h)


def kvp_prefill_predict_host(h, tokens_host, lengths: Sequence[int], cache: "Cache", workspace, logits_dev,
                             logits_host, first_token_host, stream: int) -> None:
    """tokens_host / logits_host / first_token_host: CPU tensors (pinned for real overlap)."""
    cc = _cache_c(cache)
    _check(lib().kvp_prefill_predict_host(h, tokens_host.data_ptr(), _i32arr(lengths), len(lengths), C.byref(cc),
                                          workspace.data_ptr(), workspace.numel(), logits_dev.data_ptr(),
                                          logits_host.data_ptr() if logits_host is not None else None,
                                          first_token_host.data_ptr(), stream), h)


def kvp_decode_step(h, tokens, lengths_host: Sequence[int], cache: "Cache", workspace, logits_out, next_token,
                    stream: int) -> None:
    cc = _cache_c(cache)
    _check(lib().kvp_decode_step(h, tokens.data_ptr(), _i32arr(lengths_host), len(lengths_host), C.byref(cc),
                                 workspace.data_ptr(), workspace.numel(), logits_out.data_ptr(),
                                 next_token.data_ptr() if next_token is not None else None, stream), h)


def kvp_decode_step_static(h, tokens, lengths_host: Sequence[int], cache: "Cache", logits_out, next_token, status_out,
                           stream: int) -> None:
    """kvp_decode_step without a workspace argument: the scratch is the library's built-in array."""
    cc = _cache_c(cache)
    _check(lib().kvp_decode_step_static(h, tokens.data_ptr(), _i32arr(lengths_host), len(lengths_host), C.byref(cc),
                                        logits_out.data_ptr(), next_token.data_ptr() if next_token is not None else None,
                                        status_out.data_ptr() if status_out is not None else None, stream), h)


def kvp_train_workspace_bytes(h, max_batch: int, max_total_tokens: int) -> int:
    n = C.c_size_t()
    _check(lib().kvp_train_workspace_bytes(h, max_batch, max_total_tokens, C.byref(n)), h)
    return n.value


def kvp_train_forward(h, tokens, lengths: Sequence[int], cache: "Cache", workspace, logits_out, l1_k, l1_v, stream: int) -> None:
    cc = _cache_c(cache)
    _check(lib().kvp_train_forward(h, tokens.data_ptr(), _i32arr(lengths), len(lengths), C.byref(cc), workspace.data_ptr(),
                                   workspace.numel(), logits_out.data_ptr() if logits_out is not None else None,
                                   l1_k.data_ptr(), l1_v.data_ptr(), stream), h)


def kvp_selftest_wait_timeout(h, workspace, stream: int) -> None:
    _check(lib().kvp_selftest_wait_timeout(h, workspace.data_ptr(), stream), h)


def kvp_poll_status(h, workspace, stream: int) -> None:
    _check(lib().kvp_poll_status(h, workspace.data_ptr(), stream), h)


# ---- device-memory plumbing -----------------------------------------------------------------
class Cache:
    """Paged base-model KV cache in torch-allocated device memory."""

    def __init__(self, h, pair, max_batch: int, max_len: int, device, n_pages: Optional[int] = None,
                 shuffle_pages: bool = True, seed: int = 0):
        import torch
        self.pair = pair
        # 16-bit cache elements are IEEE halves (see kvp.h: more significant bits than bfloat16 for the path's product)
        tdt = torch.float16 if pair.dtype == "bf16" else torch.float32
        self.max_pages_per_seq = (max_len + 63) // 64
        self.n_pages = n_pages if n_pages is not None else max_batch * self.max_pages_per_seq
        nl = pair.base.n_layers
        self.k = [torch.zeros((self.n_pages, lc.n_kv_heads, 64, lc.head_dim), dtype=tdt, device=device) for lc in pair.base.layers]
        self.v = [torch.zeros((self.n_pages, lc.n_kv_heads, 64, lc.head_dim), dtype=tdt, device=device) for lc in pair.base.layers]
        for i in range(nl):
            assert self.k[i][0].numel() * self.k[i].element_size() == kvp_cache_layout(h, i)
        self._kp = (C.c_void_p * nl)(*[t.data_ptr() for t in self.k])
        self._vp = (C.c_void_p * nl)(*[t.data_ptr() for t in self.v])
        # pages handed out in a scrambled order so that nothing relies on contiguity
        ids = np.arange(self.n_pages, dtype=np.int32)
        if shuffle_pages:
            np.random.default_rng(seed).shuffle(ids)
        bt = np.full((max_batch, self.max_pages_per_seq), -1, np.int32)
        n = min(self.n_pages, max_batch * self.max_pages_per_seq)
        bt.reshape(-1)[:n] = ids[:n]
        self.block_table_host = bt
        self.block_table = torch.from_numpy(bt).to(device)
        self.seq_lens = torch.zeros(max_batch, dtype=torch.int32, device=device)

    def gather(self, layer: int, b: int, length: int):
        """(K, V) of sequence b in base layer `layer` as float32 numpy [length, n_kv * hd]."""
        import torch
        pages = torch.from_numpy(self.block_table_host[b, :(length + 63) // 64].astype(np.int64)).to(self.k[layer].device)
        out = []
        for pool in (self.k[layer], self.v[layer]):
            t = pool[pages]                                 # [np, nkv, 64, hd]
            t = t.permute(0, 2, 1, 3).reshape(-1, t.shape[1] * t.shape[3])[:length]
            out.append(t.float().cpu().numpy())
        return out[0], out[1]


class Session:
    """Creates a handle for `pair`, uploads and packs weights, allocates workspace and cache."""

    def __init__(self, pair, weights: Dict[str, np.ndarray], max_batch: int, max_total_tokens: int, max_len: int,
                 device="cuda:0", extra_len: int = 0, flags: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the KV Prediction library has no CPU path")
        self.torch = torch
        self.pair = pair
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.h = kvp_create(pair.aux, pair.base, pair.layer_map, pair.dtype, pair.predictor_bias, flags=flags)
        # The library replays a recorded CUDA graph per call, which the legacy default stream cannot record:
        # when that is the current stream the session works on a stream of its own and orders it against the
        # current stream around every call, so a caller still sees everything in the current stream's order.
        cur = torch.cuda.current_stream(self.device)
        self.torch_stream = torch.cuda.Stream(self.device) if cur.cuda_stream == 0 else cur
        self.stream = self.torch_stream.cuda_stream
        self.packed = torch.empty(kvp_packed_weight_bytes(self.h) + 256, dtype=torch.uint8, device=self.device)
        self.load(weights)
        self.max_batch, self.max_total = max_batch, max_total_tokens
        self.workspace = torch.empty(kvp_workspace_bytes(self.h, max_batch, max_total_tokens), dtype=torch.uint8, device=self.device)
        self.cache = Cache(self.h, pair, max_batch, max_len + extra_len, self.device)
        self.logits = torch.empty((max_batch, pair.base.vocab), dtype=torch.float32, device=self.device)
        self.first = torch.empty(max_batch, dtype=torch.int32, device=self.device)

    def load(self, weights: Dict[str, np.ndarray], chunk_bytes: int = 1 << 30):
        """Uploads in chunks (source tensors are freed after packing)."""
        torch = self.torch
        bf = self.pair.dtype == "bf16"
        batch, size = {}, 0
        for name, w in weights.items():
            t = torch.from_numpy(np.ascontiguousarray(w))
            t = t.to(self.device)
            if bf:
                t = t.to(torch.bfloat16)    # exact: the values are already bf16-representable
            batch[name] = t
            size += t.numel() * t.element_size()
            if size >= chunk_bytes:
                kvp_load_weights(self.h, batch, self.packed, self.stream)
                torch.cuda.synchronize()
                batch, size = {}, 0
        if batch:
            kvp_load_weights(self.h, batch, self.packed, self.stream)
            torch.cuda.synchronize()

    def enter(self):
        """Orders the session's stream after the current torch stream; returns the latter for leave()."""
        cur = self.torch.cuda.current_stream(self.device)
        if cur.cuda_stream != self.stream:
            self.torch_stream.wait_stream(cur)
        return cur

    def leave(self, cur):
        if cur.cuda_stream != self.stream:
            cur.wait_stream(self.torch_stream)

    def prefill_predict(self, tokens_dev, lengths: Sequence[int]):
        b = len(lengths)
        cur = self.enter()
        try:
            kvp_prefill_predict(self.h, tokens_dev, lengths, self.cache, self.workspace, self.logits, self.first, self.stream)
        finally:
            self.leave(cur)
        return self.logits[:b], self.first[:b]

    def decode_step(self, tokens_dev, lengths: Sequence[int]):
        b = len(lengths)
        cur = self.enter()
        try:
            kvp_decode_step(self.h, tokens_dev, lengths, self.cache, self.workspace, self.logits, self.first, self.stream)
        finally:
            self.leave(cur)
        return self.logits[:b], self.first[:b]

    def train_forward(self, tokens_dev, lengths: Sequence[int], want_logits: bool = True):
        """After prefill_predict on the same prompt: (logits [T, vocab] or None, l1_k [n_B], l1_v [n_B]) on the device."""
        torch = self.torch
        total = int(sum(lengths))
        need = kvp_train_workspace_bytes(self.h, len(lengths), total)
        if getattr(self, "train_ws", None) is None or self.train_ws.numel() < need:
            self.train_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        logits = torch.empty((total, self.pair.base.vocab), dtype=torch.float32, device=self.device) if want_logits else None
        l1_k = torch.empty(self.pair.base.n_layers, dtype=torch.float32, device=self.device)
        l1_v = torch.empty_like(l1_k)
        cur = self.enter()
        try:
            kvp_train_forward(self.h, tokens_dev, lengths, self.cache, self.train_ws, logits, l1_k, l1_v, self.stream)
        finally:
            self.leave(cur)
        return logits, l1_k, l1_v

    def poll(self):
        kvp_poll_status(self.h, self.workspace, self.stream)

    def close(self):
        if self.h:
            self.torch.cuda.synchronize()
            kvp_destroy(self.h)
            self.h = None
