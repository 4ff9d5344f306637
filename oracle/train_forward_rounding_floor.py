"""Test infrastructure, CPU only: how far do the training-time forward's logits move when nothing but the
storage formats of a bf16 run are applied to the oracle's exact arithmetic?

    python oracle/train_forward_rounding_floor.py c2 192      # workload, tokens of sequence 0

The forward of the base model on the predicted cache (Sec. 4.1 "Training") is evaluated twice in fp64: exactly,
and with every tensor that a bf16 run stores in bf16 rounded once where it is stored: the predicted cache, the
normalised activations that enter the projections, the rotated queries, the attention output and the FFN
activation (the residual stream stays exact: it is fp32 on the GPU).  All sums stay exact.  The relative Frobenius
distance of the two logit matrices is the part of the GPU-vs-oracle error that the storage precision alone
explains; unlike the inference path's single step (fp32 activations), this forward feeds bf16 activations to four
projections per layer at every position.
"""
import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import workloads as wl  # noqa: E402
from oracle import kvp_oracle as orc  # noqa: E402


def r16(x):
    return wl.round_to_bf16(np.asarray(x, dtype=np.float32)).astype(np.float64)


def forward(pair, W, tokens, kv_hat, rnd):
    cfg = pair.base
    L = len(tokens)
    pos = np.arange(L)
    x = orc._w(W, "base.embed")[tokens]
    for i, lc in enumerate(cfg.layers):
        b = f"base.L{i}."
        h = rnd(orc.rmsnorm(x, W[b + "attn_norm"], cfg.rms_eps))
        q = (h @ orc._w(W, b + "wq").T).reshape(L, lc.n_q_heads, lc.head_dim)
        q, _ = orc.qk_norm(cfg, W, b, q, None)
        q = rnd(orc.rope(q, pos, cfg.rope_theta))
        k = rnd(kv_hat[i][0]).reshape(L, lc.n_kv_heads, lc.head_dim)
        v = rnd(kv_hat[i][1]).reshape(L, lc.n_kv_heads, lc.head_dim)
        a = rnd(orc.attention(q, k, v, pos))
        x = x + a.reshape(L, -1) @ orc._w(W, b + "wo").T
        h2 = rnd(orc.rmsnorm(x, W[b + "ffn_norm"], cfg.rms_eps))
        act = rnd(orc.silu(h2 @ orc._w(W, b + "w_gate").T) * (h2 @ orc._w(W, b + "w_up").T))
        x = x + act @ orc._w(W, b + "w_down").T
    return rnd(orc.rmsnorm(x, W["base.final_norm"], cfg.rms_eps)) @ orc._w(W, "base.lm_head").T


def floor(name: str, n: int):
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=0)
    toks = wl.prompts(name, seed=0).seq(0)[:n]
    kv = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    ref = forward(pair, W, toks, kv, lambda t: np.asarray(t, dtype=np.float64))
    got = forward(pair, W, toks, kv, r16)
    rows = np.linalg.norm(got - ref, axis=1) / np.linalg.norm(ref, axis=1)
    return float(np.linalg.norm(got - ref) / np.linalg.norm(ref)), float(rows.max())


if __name__ == "__main__":
    name, n = sys.argv[1], int(sys.argv[2])
    t = time.time()
    whole, worst = floor(name, n)
    print(f"{name}, first {n} tokens: logits move by {whole:.3e} (worst row {worst:.3e}) from bf16 storage alone ({time.time() - t:.0f} s)")
