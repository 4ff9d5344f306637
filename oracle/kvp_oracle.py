"""CPU oracle for the KV Prediction time-to-first-token path (arXiv 2410.08391).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy statement of what
the path computes, written from the paper so that a reader can check it by eye.
Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import it; the product path never does, and this file imports nothing of the
CUDA path.

The method is an approximation scheme (the predicted cache only approximates
the base model's own cache, Sec. 4), so the oracle is the algorithm taken step
by step in the order of the inference algorithm of Fig. 2(b):

    a, KV_A  <- A(I)              auxiliary prefill          (aux_prefill)
    KV_B_hat <- P(KV_A)           linear KV predictor        (predict_kv)
    b        <- B(I[-1], KV_B_hat) one base step on the predicted cache
                                                            (base_first_step)
    loop: b, p <- B(I[-1], KV_B_hat); KV_B_hat <- KV_B_hat + p   (decode_step)

No blocking, fusion or re-ordering is applied beyond evaluating attention a
block of query rows at a time (each row's softmax is still the full, one-pass
definition) to bound memory.  Matrix products use numpy's `@` as a library step.

Readings of points the paper leaves open (the paper only says "OpenELM"):
  * pre-norm decoder blocks, RMSNorm(x; g) = g * x / sqrt(mean(x^2) + eps),
    SwiGLU FFN  down(silu(gate(h)) * up(h)),  final RMSNorm before the LM head;
  * RoPE in the rotate-half pairing (c, c + hd/2), angle pos * theta^(-2c/hd);
  * the KV cache holds what attention consumes: keys after RoPE.  The predictor
    therefore maps aux post-RoPE keys to base post-RoPE keys (Sec. 4.1 "used as
    the keys and values in the attention operations");
  * separate linear maps FK_i, FV_i per base layer over the whole flattened
    kv width (Sec. 4.2: F_i : R^{d_KV_A,j_i} -> R^{d_KV_B,i}), optional bias;
  * the first base step attends to predicted entries 0..L-1 and appends
    nothing; appending starts with the first generated token (Fig. 2(b)).

Pins (tests/test_oracle_pins.py): brute-force attention on tiny inputs,
prefill == token-by-token decoding, identity predictor with aux == base,
textbook reductions, RoPE invariants, batch independence, and the layer-map
rows printed in Table 1.  Parity unpinned: the pre/post-RoPE choice for cached
keys, the bias option, dense-across-heads separate K/V maps, eps and the RoPE
pairing: no printed value or invariant separates the alternatives.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# layer maps  (Sec. 4.2, Table 1; Appendix A, Table 4)
# ----------------------------------------------------------------------------
def layer_map_canonical(n_base: int, n_aux: int) -> List[int]:
    """KVP-C map j_i.  Consecutive base layers share an aux layer; when n_aux does
    not divide n_base the first (n_base mod n_aux) aux layers feed one more base
    layer than the others ("we perform rounding", Sec. 4.2; reproduces every KVP-C
    row of Table 1)."""
    q, r = divmod(n_base, n_aux)
    out: List[int] = []
    for j in range(n_aux):
        out += [j] * (q + 1 if j < r else q)
    return out


def layer_map_pruned(n_base: int, retained: Sequence[int]) -> List[int]:
    """KVP-LP map: the aux model keeps base layers `retained` (Appendix A); base
    layer i is predicted from the aux layer that came from the nearest retained
    base layer at or below i (reproduces every KVP-LP row of Table 1)."""
    out = []
    for i in range(n_base):
        j = max(k for k, r in enumerate(retained) if r <= i)
        out.append(j)
    return out


def layer_map_uniform(n_base: int, n_aux: int) -> List[int]:
    """j_i = floor(i * n_aux / n_base)."""
    return [(i * n_aux) // n_base for i in range(n_base)]


# ----------------------------------------------------------------------------
# transformer ingredients
# ----------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    x = x.astype(F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return g.astype(F64) * x / np.sqrt(ms + eps)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """x: [L, n_heads, hd]; pos: [L] integer positions.  Rotate-half pairing."""
    L, H, hd = x.shape
    half = hd // 2
    c = np.arange(half, dtype=F64)
    inv = theta ** (-2.0 * c / hd)                       # [half]
    ang = pos.astype(F64)[:, None] * inv[None, :]        # [L, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, q_pos: np.ndarray,
              row_block: int = 1024) -> np.ndarray:
    """Grouped-query attention.  q: [Lq, nq, hd]; k, v: [Lk, nkv, hd]; q_pos[t] is
    the cache position of query t, which sees keys s <= q_pos[t].  Query head u
    uses kv head floor(u / (nq / nkv)).  Returns [Lq, nq, hd]."""
    Lq, nq, hd = q.shape
    Lk, nkv, _ = k.shape
    group = nq // nkv
    out = np.empty((Lq, nq, hd), F64)
    s_idx = np.arange(Lk)
    for u in range(nq):
        ku, vu = k[:, u // group, :], v[:, u // group, :]
        for r0 in range(0, Lq, row_block):
            r1 = min(Lq, r0 + row_block)
            s = (q[r0:r1, u, :] @ ku.T) / np.sqrt(hd)
            s = np.where(s_idx[None, :] <= q_pos[r0:r1, None], s, -np.inf)
            out[r0:r1, u, :] = softmax_rows(s) @ vu
    return out


def ffn(h: np.ndarray, wg: np.ndarray, wu: np.ndarray, wd: np.ndarray) -> np.ndarray:
    return (silu(h @ wg.T.astype(F64)) * (h @ wu.T.astype(F64))) @ wd.T.astype(F64)


def _w(W: Dict[str, np.ndarray], name: str) -> np.ndarray:
    return W[name].astype(F64)


def qk_norm(cfg, W, b: str, q, k):
    """OpenELM normalises queries and keys (Sec. 7 "key norm"): an RMSNorm over head_dim of every
    head, one gain vector per layer for q and one for k, applied before RoPE.  Off unless the
    model asks for it; q may be None (a caller that only needs keys)."""
    if not getattr(cfg, "qk_norm", False):
        return q, k
    if q is not None:
        q = rmsnorm(q, W[b + "q_norm"], cfg.rms_eps)
    if k is not None:
        k = rmsnorm(k, W[b + "k_norm"], cfg.rms_eps)
    return q, k


# ----------------------------------------------------------------------------
# a decoder over a whole prompt (used for A, and for B in the invariants)
# ----------------------------------------------------------------------------
def decoder_prefill(cfg, W, prefix: str, tokens: np.ndarray, *, pos0: int = 0,
                    want_logits: bool = False, n_layers: Optional[int] = None, kv_given=None):
    """Run decoder `prefix` ("aux" or "base") over one prompt.

    Returns (kv, x, logits): kv[l] = (k, v) with k [L, nkv_l*hd] after RoPE and
    v [L, nkv_l*hd]; x the final residual stream [L, d]; logits [L, vocab] or None.
    `pos0` shifts every position (only the RoPE shift-invariance pin uses it).
    `kv_given[l] = (K, V)`: attention reads these keys and values (entry s visible to query t >= s)
    instead of the layer's own projections: the training-time forward of Sec. 4.1 ("masked
    cross-attention with the predicted KV cache"); kv still returns the layer's own k, v.
    """
    L = len(tokens)
    pos = np.arange(L) + pos0
    x = _w(W, f"{prefix}.embed")[tokens]
    kv = []
    nl = cfg.n_layers if n_layers is None else n_layers
    for l in range(nl):
        lc = cfg.layers[l]
        b = f"{prefix}.L{l}."
        h = rmsnorm(x, W[b + "attn_norm"], cfg.rms_eps)
        q = (h @ _w(W, b + "wq").T).reshape(L, lc.n_q_heads, lc.head_dim)
        k = (h @ _w(W, b + "wk").T).reshape(L, lc.n_kv_heads, lc.head_dim)
        v = (h @ _w(W, b + "wv").T).reshape(L, lc.n_kv_heads, lc.head_dim)
        q, k = qk_norm(cfg, W, b, q, k)
        q = rope(q, pos, cfg.rope_theta)
        k = rope(k, pos, cfg.rope_theta)
        kv.append((k.reshape(L, -1), v.reshape(L, -1)))
        if kv_given is not None:
            k = np.asarray(kv_given[l][0], dtype=F64).reshape(L, lc.n_kv_heads, lc.head_dim)
            v = np.asarray(kv_given[l][1], dtype=F64).reshape(L, lc.n_kv_heads, lc.head_dim)
        a = attention(q, k, v, np.arange(L))
        x = x + a.reshape(L, -1) @ _w(W, b + "wo").T
        h2 = rmsnorm(x, W[b + "ffn_norm"], cfg.rms_eps)
        x = x + ffn(h2, W[b + "w_gate"], W[b + "w_up"], W[b + "w_down"])
    logits = None
    if want_logits:
        logits = rmsnorm(x, W[f"{prefix}.final_norm"], cfg.rms_eps) @ _w(W, f"{prefix}.lm_head").T
    return kv, x, logits


def aux_prefill(pair, W, tokens: np.ndarray):
    """a, KV_A <- A(I).  The aux logits are never used at inference (Sec. 4.3), and
    layers above the last one the map reads do not influence any output, so only
    layers 0..max(j_i) are evaluated; KV_A[j] = (K post-RoPE, V), each [L, d_kvA_j]."""
    n = max(pair.layer_map) + 1
    kv, _, _ = decoder_prefill(pair.aux, W, "aux", tokens, n_layers=n)
    return kv


# ----------------------------------------------------------------------------
# predictor  (Sec. 4.2)
# ----------------------------------------------------------------------------
def predict_kv(pair, W, kv_aux):
    """KV_B_hat_i = F_i(KV_A_{j_i}) for every base layer i; token-wise linear maps.
    Returns a list over base layers of (K_hat [L, d_kvB_i], V_hat [L, d_kvB_i])."""
    out = []
    for i, j in enumerate(pair.layer_map):
        ka, va = kv_aux[j]
        kh = ka @ _w(W, f"pred.L{i}.fk").T
        vh = va @ _w(W, f"pred.L{i}.fv").T
        if pair.predictor_bias:
            kh = kh + _w(W, f"pred.L{i}.bk")
            vh = vh + _w(W, f"pred.L{i}.bv")
        out.append((kh, vh))
    return out


# ----------------------------------------------------------------------------
# base model single-token steps
# ----------------------------------------------------------------------------
def _base_block_tail(cfg, W, i, x, a):
    b = f"base.L{i}."
    x = x + a.reshape(1, -1) @ _w(W, b + "wo").T
    h2 = rmsnorm(x, W[b + "ffn_norm"], cfg.rms_eps)
    return x + ffn(h2, W[b + "w_gate"], W[b + "w_up"], W[b + "w_down"])


def base_first_step(pair, W, token: int, kv_hat):
    """b <- B(I[-1], KV_B_hat): the base model processes the last prompt token at
    position L-1; in every layer the query comes from the base's own projection
    while keys and values are the L predicted entries (the base K/V projections
    are not used and nothing is appended).  Returns logits [vocab]."""
    cfg = pair.base
    L = kv_hat[0][0].shape[0]
    pos = np.array([L - 1])
    x = _w(W, "base.embed")[[token]]
    for i, lc in enumerate(cfg.layers):
        b = f"base.L{i}."
        h = rmsnorm(x, W[b + "attn_norm"], cfg.rms_eps)
        q = (h @ _w(W, b + "wq").T).reshape(1, lc.n_q_heads, lc.head_dim)
        q, _ = qk_norm(cfg, W, b, q, None)
        q = rope(q, pos, cfg.rope_theta)
        kh, vh = kv_hat[i]
        a = attention(q, kh.reshape(L, lc.n_kv_heads, lc.head_dim),
                      vh.reshape(L, lc.n_kv_heads, lc.head_dim), pos)
        x = _base_block_tail(cfg, W, i, x, a)
    return (rmsnorm(x, W["base.final_norm"], cfg.rms_eps) @ _w(W, "base.lm_head").T)[0]


def decode_step(pair, W, token: int, cache):
    """b, p <- B(I[-1], KV_B_hat); KV_B_hat <- KV_B_hat + p  (generation loop).
    `cache` is a list over base layers of (K [len, d_kv], V [len, d_kv]); the new
    token sits at position len, its own k (post-RoPE) and v are appended, and it
    attends over len+1 entries.  Returns (logits [vocab], new cache)."""
    cfg = pair.base
    p = cache[0][0].shape[0]
    pos = np.array([p])
    x = _w(W, "base.embed")[[token]]
    new_cache = []
    for i, lc in enumerate(cfg.layers):
        b = f"base.L{i}."
        h = rmsnorm(x, W[b + "attn_norm"], cfg.rms_eps)
        q = (h @ _w(W, b + "wq").T).reshape(1, lc.n_q_heads, lc.head_dim)
        k = (h @ _w(W, b + "wk").T).reshape(1, lc.n_kv_heads, lc.head_dim)
        q, k = qk_norm(cfg, W, b, q, k)
        q = rope(q, pos, cfg.rope_theta)
        k = rope(k, pos, cfg.rope_theta)
        v = h @ _w(W, b + "wv").T
        K = np.concatenate([cache[i][0], k.reshape(1, -1)], axis=0)
        V = np.concatenate([cache[i][1], v.reshape(1, -1)], axis=0)
        new_cache.append((K, V))
        a = attention(q, K.reshape(p + 1, lc.n_kv_heads, lc.head_dim),
                      V.reshape(p + 1, lc.n_kv_heads, lc.head_dim), pos)
        x = _base_block_tail(cfg, W, i, x, a)
    logits = (rmsnorm(x, W["base.final_norm"], cfg.rms_eps) @ _w(W, "base.lm_head").T)[0]
    return logits, new_cache


# ----------------------------------------------------------------------------
# training-time forward and consistency terms  (Sec. 4.1 "Training", Sec. 4.3)
# ----------------------------------------------------------------------------
def train_forward(pair, W, tokens: np.ndarray):
    """One prompt through the training-time graph, forward only (Fig. 2(a)):
    KV_A <- A(I);  KV_hat <- P(KV_A);  b <- B(I) with KV_hat as the keys and values of every layer's
    attention (query t sees predicted entries 0..t);  KV_B <- the base model's cache from its ordinary
    forward over I.  Returns (logits_b [L, vocab], abs_k, abs_v, n_k) with abs_k[i] = sum over tokens and
    columns of |K_hat_i - K_B,i|, abs_v[i] likewise, n_k[i] = L * d_kvB_i: the consistency loss of Sec. 4.3
    is the mean abs_k[i] / n_k[i] (and the same for V), summed or averaged over layers."""
    kv_hat = predict_kv(pair, W, aux_prefill(pair, W, tokens))
    kv_b, _, _ = decoder_prefill(pair.base, W, "base", tokens)
    _, _, logits = decoder_prefill(pair.base, W, "base", tokens, want_logits=True, kv_given=kv_hat)
    abs_k = [float(np.abs(kh - kb).sum()) for (kh, _), (kb, _) in zip(kv_hat, kv_b)]
    abs_v = [float(np.abs(vh - vb).sum()) for (_, vh), (_, vb) in zip(kv_hat, kv_b)]
    n = [int(kb.size) for kb, _ in kv_b]
    return logits, abs_k, abs_v, n


def argmax_lowest(logits: np.ndarray) -> int:
    """Greedy token; the lowest index wins ties."""
    return int(np.argmax(logits))


def top2_gap(logits: np.ndarray) -> float:
    s = np.partition(logits, -2)[-2:]
    return float(s[1] - s[0])


# ----------------------------------------------------------------------------
# the whole TTFT path for a batch (sequences are independent)
# ----------------------------------------------------------------------------
def prefill_predict(pair, W, prompts, seqs: Optional[Sequence[int]] = None):
    """For each selected sequence: (kv_hat list over base layers, logits, first token)."""
    out = {}
    for b in (range(prompts.batch) if seqs is None else seqs):
        toks = prompts.seq(b)
        kv_hat = predict_kv(pair, W, aux_prefill(pair, W, toks))
        logits = base_first_step(pair, W, int(toks[-1]), kv_hat)
        out[b] = (kv_hat, logits, argmax_lowest(logits))
    return out
