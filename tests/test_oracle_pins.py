"""Pins for the CPU oracle: each checks oracle/kvp_oracle.py against something the
paper or the mathematics fixes, never against the oracle itself or the CUDA path."""
import math

import os

import numpy as np
import pytest

import workloads as wl
from oracle import kvp_oracle as orc
from conftest import read_layer_map_golden


# --------------------------------------------------------------------------
# Table 1 / Table 4: printed layer maps
# --------------------------------------------------------------------------
@pytest.mark.parametrize("row", read_layer_map_golden(), ids=lambda r: r["name"])
def test_layer_maps_match_table_1(row):
    if row["kind"] == "C":
        got = orc.layer_map_canonical(row["n_base"], row["n_aux"])
    else:
        assert len(row["retained"]) == row["n_aux"]
        got = orc.layer_map_pruned(row["n_base"], row["retained"])
    assert got == row["map"]


def test_uniform_map_is_floor_rule():
    assert orc.layer_map_uniform(4, 2) == [0, 0, 1, 1]
    m = orc.layer_map_uniform(28, 16)
    assert m[0] == 0 and m[-1] == 15 and all(b - a in (0, 1) for a, b in zip(m, m[1:]))


# --------------------------------------------------------------------------
# closed forms for the ingredients
# --------------------------------------------------------------------------
def test_rmsnorm_closed_form():
    y = orc.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)
    r = math.sqrt(12.5)
    np.testing.assert_allclose(y, [[3 / r, 8 / r]], rtol=1e-15)
    # eps enters under the square root, next to the mean square
    y = orc.rmsnorm(np.array([[0.0, 0.0, 2.0]]), np.ones(3), 1.0)
    np.testing.assert_allclose(y[0, 2], 2 / math.sqrt(4 / 3 + 1.0), rtol=1e-15)


def test_silu_values():
    np.testing.assert_allclose(orc.silu(np.array([0.0, 1.0, -1.0, 30.0])),
                               [0.0, 1 / (1 + math.exp(-1)), -1 / (1 + math.e), 30.0], rtol=1e-12)


def test_rope_is_plane_rotation():
    # hd = 2: one pair, frequency theta^0 = 1 -> rotation by `pos` radians
    x = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    y = orc.rope(x, np.array([0.5, 2.0]), 10000.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(0.5), math.sin(0.5)], rtol=1e-15)
    np.testing.assert_allclose(y[1, 0], [-math.sin(2.0), math.cos(2.0)], rtol=1e-15)
    # hd = 4: pair (0,2) turns at rate 1, pair (1,3) at rate theta^(-2/4)
    x = np.array([[[1.0, 1.0, 0.0, 0.0]]])
    y = orc.rope(x, np.array([3.0]), 100.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(3), math.cos(0.3), math.sin(3), math.sin(0.3)], rtol=1e-13)


def test_rope_preserves_norm_and_position_zero_is_identity():
    g = np.random.default_rng(1)
    x = g.standard_normal((7, 3, 16))
    y = orc.rope(x, np.arange(7), 10000.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    np.testing.assert_allclose(y[0], x[0], rtol=0, atol=0)


def test_attention_zero_query_gives_causal_prefix_mean():
    g = np.random.default_rng(2)
    L, nq, nkv, hd = 9, 4, 2, 8
    k = g.standard_normal((L, nkv, hd))
    v = g.standard_normal((L, nkv, hd))
    out = orc.attention(np.zeros((L, nq, hd)), k, v, np.arange(L))
    for t in range(L):
        for u in range(nq):
            np.testing.assert_allclose(out[t, u], v[:t + 1, u // 2].mean(axis=0), rtol=1e-13)


def test_attention_constant_values_pass_through():
    g = np.random.default_rng(3)
    L, nq, nkv, hd = 6, 2, 1, 4
    c = g.standard_normal(hd)
    out = orc.attention(g.standard_normal((L, nq, hd)), g.standard_normal((L, nkv, hd)),
                        np.broadcast_to(c, (L, nkv, hd)), np.arange(L))
    np.testing.assert_allclose(out, np.broadcast_to(c, (L, nq, hd)), rtol=1e-13)


def _brute_attention(q, k, v, q_pos):
    """Scalar loops straight from softmax(q k^T / sqrt(hd)) v with a causal mask."""
    Lq, nq, hd = q.shape
    Lk, nkv, _ = k.shape
    out = np.zeros((Lq, nq, hd))
    for t in range(Lq):
        for u in range(nq):
            g = u // (nq // nkv)
            sc = []
            for s in range(Lk):
                if s <= q_pos[t]:
                    sc.append(sum(q[t, u, c] * k[s, g, c] for c in range(hd)) / math.sqrt(hd))
            m = max(sc)
            w = [math.exp(z - m) for z in sc]
            z = sum(w)
            for c in range(hd):
                out[t, u, c] = sum(w[s] * v[s, g, c] for s in range(len(sc))) / z
    return out


@pytest.mark.parametrize("L,nq,nkv,hd", [(1, 1, 1, 2), (5, 4, 2, 4), (8, 6, 2, 4), (7, 3, 3, 2)])
def test_attention_matches_brute_force(L, nq, nkv, hd):
    g = np.random.default_rng(10 + L)
    q, k, v = (3 * g.standard_normal((L, n, hd)) for n in (nq, nkv, nkv))
    np.testing.assert_allclose(orc.attention(q, k, v, np.arange(L)),
                               _brute_attention(q, k, v, np.arange(L)), rtol=1e-12, atol=1e-14)
    # row blocking must not change anything
    np.testing.assert_allclose(orc.attention(q, k, v, np.arange(L), row_block=3),
                               orc.attention(q, k, v, np.arange(L)), rtol=1e-14, atol=1e-15)
    # a single late query over a longer cache (the base step's shape)
    np.testing.assert_allclose(orc.attention(q[-1:], k, v, np.array([L - 1])),
                               _brute_attention(q[-1:], k, v, [L - 1]), rtol=1e-12, atol=1e-14)


# --------------------------------------------------------------------------
# brute force of the whole path on a tiny pair, scalar loops only
# --------------------------------------------------------------------------
def _matvec(W, x):          # y[n] = sum_k W[n][k] x[k]   (matrices are [out, in])
    return [sum(W[n][k] * x[k] for k in range(len(x))) for n in range(len(W))]


def _norm(x, g, eps):
    ms = sum(a * a for a in x) / len(x)
    return [g[i] * x[i] / math.sqrt(ms + eps) for i in range(len(x))]


def _rope_vec(x, n_heads, hd, pos, theta):
    y = list(x)
    for h in range(n_heads):
        for c in range(hd // 2):
            a = pos * theta ** (-2.0 * c / hd)
            i0, i1 = h * hd + c, h * hd + c + hd // 2
            y[i0] = x[i0] * math.cos(a) - x[i1] * math.sin(a)
            y[i1] = x[i1] * math.cos(a) + x[i0] * math.sin(a)
    return y


def _attend(q, Ks, Vs, nq, nkv, hd):
    out = []
    for u in range(nq):
        g = u // (nq // nkv)
        sc = [sum(q[u * hd + c] * K[g * hd + c] for c in range(hd)) / math.sqrt(hd) for K in Ks]
        m = max(sc)
        w = [math.exp(s - m) for s in sc]
        z = sum(w)
        out += [sum(w[s] * Vs[s][g * hd + c] for s in range(len(Ks))) / z for c in range(hd)]
    return out


def _ffn_vec(W, b, h):
    g, u = _matvec(W[b + "w_gate"], h), _matvec(W[b + "w_up"], h)
    return _matvec(W[b + "w_down"], [g[i] / (1 + math.exp(-g[i])) * u[i] for i in range(len(g))])


def _brute_path(pair, W, toks):
    W = {k: v.astype(np.float64).tolist() for k, v in W.items()}
    A, B = pair.aux, pair.base
    L = len(toks)
    xs = [list(W["aux.embed"][t]) for t in toks]
    KA = []
    for j, lc in enumerate(A.layers):
        b = f"aux.L{j}."
        hs = [_norm(x, W[b + "attn_norm"], A.rms_eps) for x in xs]
        qs = [_rope_vec(_matvec(W[b + "wq"], h), lc.n_q_heads, lc.head_dim, t, A.rope_theta) for t, h in enumerate(hs)]
        ks = [_rope_vec(_matvec(W[b + "wk"], h), lc.n_kv_heads, lc.head_dim, t, A.rope_theta) for t, h in enumerate(hs)]
        vs = [_matvec(W[b + "wv"], h) for h in hs]
        KA.append((ks, vs))
        for t in range(L):
            a = _attend(qs[t], ks[:t + 1], vs[:t + 1], lc.n_q_heads, lc.n_kv_heads, lc.head_dim)
            o = _matvec(W[b + "wo"], a)
            xs[t] = [xs[t][i] + o[i] for i in range(A.d_model)]
            f = _ffn_vec(W, b, _norm(xs[t], W[b + "ffn_norm"], A.rms_eps))
            xs[t] = [xs[t][i] + f[i] for i in range(A.d_model)]
    KH = []
    for i, j in enumerate(pair.layer_map):
        kh = [_matvec(W[f"pred.L{i}.fk"], k) for k in KA[j][0]]
        vh = [_matvec(W[f"pred.L{i}.fv"], v) for v in KA[j][1]]
        if pair.predictor_bias:
            kh = [[a + c for a, c in zip(r, W[f"pred.L{i}.bk"])] for r in kh]
            vh = [[a + c for a, c in zip(r, W[f"pred.L{i}.bv"])] for r in vh]
        KH.append((kh, vh))
    x = list(W["base.embed"][toks[-1]])
    for i, lc in enumerate(B.layers):
        b = f"base.L{i}."
        q = _rope_vec(_matvec(W[b + "wq"], _norm(x, W[b + "attn_norm"], B.rms_eps)),
                      lc.n_q_heads, lc.head_dim, L - 1, B.rope_theta)
        a = _attend(q, KH[i][0], KH[i][1], lc.n_q_heads, lc.n_kv_heads, lc.head_dim)
        o = _matvec(W[b + "wo"], a)
        x = [x[k] + o[k] for k in range(B.d_model)]
        f = _ffn_vec(W, b, _norm(x, W[b + "ffn_norm"], B.rms_eps))
        x = [x[k] + f[k] for k in range(B.d_model)]
    logits = _matvec(W["base.lm_head"], _norm(x, W["base.final_norm"], B.rms_eps))
    return KH, logits


def _tiny_pair(bias=False):
    aux = wl.ModelCfg(d_model=8, vocab=11, layers=(wl.LayerCfg(2, 2, 4, 6), wl.LayerCfg(2, 1, 4, 10)))
    base = wl.ModelCfg(d_model=12, vocab=11, layers=(wl.LayerCfg(4, 2, 2, 14), wl.LayerCfg(2, 2, 2, 6),
                                                     wl.LayerCfg(6, 3, 2, 9)))
    return wl.PairCfg("tiny", aux, base, (0, 1, 1), dtype="f32", predictor_bias=bias)


@pytest.mark.parametrize("bias", [False, True])
def test_whole_path_matches_scalar_brute_force(bias):
    pair = _tiny_pair(bias)
    W = wl.make_weights(pair, seed=5, regime="fanin")
    toks = np.array([3, 7, 0, 10, 7], np.int32)
    kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    logits = orc.base_first_step(pair, W, int(toks[-1]), kv_hat)
    KH, ref_logits = _brute_path(pair, W, toks.tolist())
    for i in range(pair.base.n_layers):
        np.testing.assert_allclose(kv_hat[i][0], np.array(KH[i][0]), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(kv_hat[i][1], np.array(KH[i][1]), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(logits, np.array(ref_logits), rtol=1e-10, atol=1e-12)


# --------------------------------------------------------------------------
# invariants of the method
# --------------------------------------------------------------------------
def _identity_setup(seed=0, regime="fanin", L=12, qk_norm=False):
    model = wl.ModelCfg(d_model=32, vocab=50, qk_norm=qk_norm,
                        layers=(wl.LayerCfg(4, 2, 8, 40), wl.LayerCfg(2, 1, 8, 24),
                                wl.LayerCfg(4, 4, 8, 56)))
    pair = wl.identity_pair(model)
    W = wl.make_weights(pair, seed=seed, regime=regime)
    for k in list(W):
        if k.startswith("base.") and "final_norm" not in k and "lm_head" not in k:
            W["aux." + k[5:]] = W[k]
    for i, lc in enumerate(model.layers):
        W[f"pred.L{i}.fk"] = np.eye(lc.d_kv, dtype=np.float32)
        W[f"pred.L{i}.fv"] = np.eye(lc.d_kv, dtype=np.float32)
    toks = wl.uniform_tokens(L, model.vocab, seed)
    return pair, W, toks


@pytest.mark.parametrize("qk_norm", [False, True])
def test_identity_predictor_reproduces_base_cache_and_logits(qk_norm):
    """aux == base, j_i = i, F = I: the predicted cache is the base model's own prompt cache,
    and the first step (query at position L-1 over L entries, nothing appended) gives the
    base model's ordinary prefill logits at the last position."""
    pair, W, toks = _identity_setup(qk_norm=qk_norm)
    kv_base, _, logits_full = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True)
    kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    for (k, v), (kh, vh) in zip(kv_base, kv_hat):
        np.testing.assert_allclose(kh, k, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(vh, v, rtol=1e-13, atol=1e-14)
    logits = orc.base_first_step(pair, W, int(toks[-1]), kv_hat)
    np.testing.assert_allclose(logits, logits_full[-1], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("qk_norm", [False, True])
def test_prefill_equals_token_by_token_decoding(qk_norm):
    pair, W, toks = _identity_setup(seed=1, qk_norm=qk_norm)
    kv_full, _, logits_full = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True)
    cache = [(np.zeros((0, lc.d_kv)), np.zeros((0, lc.d_kv))) for lc in pair.base.layers]
    for t, tok in enumerate(toks):
        logits, cache = orc.decode_step(pair, W, int(tok), cache)
        np.testing.assert_allclose(logits, logits_full[t], rtol=1e-9, atol=1e-11)
    for (k, v), (kc, vc) in zip(kv_full, cache):
        np.testing.assert_allclose(kc, k, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(vc, v, rtol=1e-11, atol=1e-13)


def test_decode_step_after_prediction_appends_base_own_entry():
    """Identity setup: after the first token, one decode step must append exactly the row the
    base model's prefill of the (L+1)-token prompt holds at position L."""
    pair, W, toks = _identity_setup(seed=2, L=9)
    kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    nxt = 17
    logits, cache = orc.decode_step(pair, W, nxt, kv_hat)
    kv_full, _, logits_full = orc.decoder_prefill(pair.base, W, "base", np.append(toks, nxt), want_logits=True)
    for (k, v), (kc, vc) in zip(kv_full, cache):
        assert kc.shape[0] == len(toks) + 1
        np.testing.assert_allclose(kc, k, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(vc, v, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(logits, logits_full[-1], rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("qk_norm", [False, True])
def test_shifting_all_positions_changes_nothing(qk_norm):
    """With query / key norm this also fixes the order: gains that differ between the two members
    of a rotated pair keep the scores a function of relative position only if they are applied
    before the rotation."""
    pair, W, toks = _identity_setup(seed=3, qk_norm=qk_norm)
    _, x0, l0 = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True)
    _, x1, l1 = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True, pos0=37)
    np.testing.assert_allclose(l1, l0, rtol=1e-8, atol=1e-10)


# --------------------------------------------------------------------------
# training-time forward (Sec. 4.1 "Training", Sec. 4.3 consistency loss)
# --------------------------------------------------------------------------
def test_train_forward_with_identity_predictor_is_the_base_models_own_forward():
    """aux == base, F = I: the predicted cache is the base model's own, so the forward with the predicted
    cache gives the base model's ordinary logits at EVERY position and the consistency terms vanish."""
    pair, W, toks = _identity_setup(seed=6)
    logits, abs_k, abs_v, n = orc.train_forward(pair, W, toks)
    _, _, ref = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True)
    np.testing.assert_allclose(logits, ref, rtol=1e-9, atol=1e-11)
    assert max(abs_k) < 1e-9 and max(abs_v) < 1e-9
    assert n == [len(toks) * lc.d_kv for lc in pair.base.layers]


def test_train_forward_last_position_is_the_inference_first_step():
    """The training-time forward at the last position sees predicted entries 0..L-1 and the query of the last
    token: exactly the first step of inference (Fig. 2(b)), so its last row of logits equals that step's."""
    pair = wl.pair("c1")
    W = wl.make_weights(pair, seed=3, regime="fanin")
    toks = wl.uniform_tokens(11, pair.base.vocab, 3)
    logits, _, _, _ = orc.train_forward(pair, W, toks)
    kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    step = orc.base_first_step(pair, W, int(toks[-1]), kv_hat)
    np.testing.assert_allclose(logits[-1], step, rtol=1e-9, atol=1e-11)
    # and every earlier row is the first step of the truncated prompt (the predicted cache is causal in the prompt)
    for t in (0, 4):
        kv_t = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks[:t + 1]))
        np.testing.assert_allclose(logits[t], orc.base_first_step(pair, W, int(toks[t]), kv_t), rtol=1e-8, atol=1e-10)


def test_consistency_terms_are_plain_l1_sums():
    """Zero predictor: K_hat = V_hat = 0, so the terms are the L1 norms of the base model's own cache, computed
    here by scalar loops over one layer."""
    pair = wl.pair("c1")
    W = wl.make_weights(pair, seed=4, regime="fanin")
    for n in list(W):
        if n.startswith("pred."):
            W[n] = np.zeros_like(W[n])
    toks = wl.uniform_tokens(6, pair.base.vocab, 4)
    _, abs_k, abs_v, _ = orc.train_forward(pair, W, toks)
    kv_b, _, _ = orc.decoder_prefill(pair.base, W, "base", toks)
    for i in (0, pair.base.n_layers - 1):
        sk = sum(abs(float(x)) for row in kv_b[i][0] for x in row)
        sv = sum(abs(float(x)) for row in kv_b[i][1] for x in row)
        assert abs(abs_k[i] - sk) <= 1e-9 * sk and abs(abs_v[i] - sv) <= 1e-9 * sv


def test_qk_norm_makes_every_cached_key_head_unit_rms():
    """Sec. 7 ("key norm"): with gains of one, every head of every cached key is an RMS-normalised
    vector, and RoPE (a rotation) keeps its length: |k_head|^2 = head_dim / (1 + eps / ms)."""
    pair, W, toks = _identity_setup(seed=4, qk_norm=True)
    for n in list(W):
        if n.endswith("q_norm") or n.endswith("k_norm"):
            W[n] = np.ones_like(W[n])
    kv, _, _ = orc.decoder_prefill(pair.base, W, "base", toks)
    for (k, _), lc in zip(kv, pair.base.layers):
        heads = k.reshape(len(toks), lc.n_kv_heads, lc.head_dim)
        ms = (heads ** 2).mean(-1)
        assert np.all(ms < 1.0) and np.all(ms > 1.0 - 1e-3), (ms.min(), ms.max())


def test_qk_norm_removes_the_scale_of_the_query_and_key_projections():
    """Scaling W_q and W_k of a layer by positive constants cannot change anything once queries
    and keys are RMS-normalised per head (up to the eps inside the root); without the norm the
    same scaling must change the logits."""
    for qk_norm in (True, False):
        pair, W, toks = _identity_setup(seed=5, qk_norm=qk_norm)
        _, _, l0 = orc.decoder_prefill(pair.base, W, "base", toks, want_logits=True)
        W2 = dict(W)
        for l in range(pair.base.n_layers):
            W2[f"base.L{l}.wq"] = W[f"base.L{l}.wq"] * np.float32(4.0)
            W2[f"base.L{l}.wk"] = W[f"base.L{l}.wk"] * np.float32(0.5)
        _, _, l1 = orc.decoder_prefill(pair.base, W2, "base", toks, want_logits=True)
        diff = np.abs(l1 - l0).max() / np.abs(l0).max()
        if qk_norm:
            assert diff < 1e-4, diff
        else:
            assert diff > 1e-3, diff


def test_predictor_is_one_matrix_product_per_layer():
    pair = wl.pair("c1")
    W = wl.make_weights(pair, seed=0)
    g = np.random.default_rng(0)
    kv_aux = [(g.standard_normal((5, lc.d_kv)), g.standard_normal((5, lc.d_kv))) for lc in pair.aux.layers]
    out = orc.predict_kv(pair, W, kv_aux)
    for i, j in enumerate(pair.layer_map):
        fk, fv = W[f"pred.L{i}.fk"].astype(float), W[f"pred.L{i}.fv"].astype(float)
        for t in range(5):
            for n in (0, 17, 63):
                assert abs(out[i][0][t, n] - sum(fk[n, c] * kv_aux[j][0][t, c] for c in range(64))) < 1e-12
                assert abs(out[i][1][t, n] - sum(fv[n, c] * kv_aux[j][1][t, c] for c in range(64))) < 1e-12


def test_zero_predictor_removes_attention_branch():
    """FK = FV = 0: predicted values are zero, so every attention output is zero and the
    logits equal those of the base model with its attention branch deleted, a function of
    the last token only."""
    pair = _tiny_pair()
    W = wl.make_weights(pair, seed=9, regime="fanin")
    for i in range(pair.base.n_layers):
        W[f"pred.L{i}.fk"] = np.zeros_like(W[f"pred.L{i}.fk"])
        W[f"pred.L{i}.fv"] = np.zeros_like(W[f"pred.L{i}.fv"])
    toks = np.array([1, 2, 3, 4], np.int32)
    kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    logits = orc.base_first_step(pair, W, 4, kv_hat)
    Wl = {k: v.astype(np.float64).tolist() for k, v in W.items()}
    x = list(Wl["base.embed"][4])
    for i in range(pair.base.n_layers):
        b = f"base.L{i}."
        f = _ffn_vec(Wl, b, _norm(x, Wl[b + "ffn_norm"], pair.base.rms_eps))
        x = [x[k] + f[k] for k in range(len(x))]
    ref = _matvec(Wl["base.lm_head"], _norm(x, Wl["base.final_norm"], pair.base.rms_eps))
    np.testing.assert_allclose(logits, ref, rtol=1e-10, atol=1e-12)


def test_argmax_takes_lowest_index_on_ties():
    assert orc.argmax_lowest(np.array([0.0, 2.0, 2.0, 1.0])) == 1
    assert abs(orc.top2_gap(np.array([0.0, 2.0, 1.5])) - 0.5) < 1e-15


def test_config_1_runs_in_seconds_and_is_finite():
    pair = wl.pair("c1")
    W = wl.make_weights(pair, seed=0)
    pr = wl.prompts("c1")
    res = orc.prefill_predict(pair, W, pr)
    kv_hat, logits, tok = res[0]
    assert len(kv_hat) == 4 and kv_hat[0][0].shape == (64, 64) and logits.shape == (512,)
    assert np.isfinite(logits).all() and 0 <= tok < 512


def test_layer_pruned_workload_pairs_use_the_maps_of_table_1():
    """The KVP-LP pairs of the workload module carry the printed j_i rows (Table 1) and as many auxiliary
    layers as Table 4 (Appendix A) retains."""
    rows = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "layer_maps.txt")):
        if line.startswith("LP | OE1.1B"):
            f = [x.strip() for x in line.split("|")]
            rows[f[1]] = (int(f[3]), tuple(int(x) for x in f[5].split()))
    for name, key in (("lp75", "OE1.1B-KVP-LP-0.75"), ("lp50", "OE1.1B-KVP-LP-0.50"), ("lp25", "OE1.1B-KVP-LP-0.25")):
        p = wl.pair(name)
        assert p.aux.n_layers == rows[key][0] and p.layer_map == rows[key][1]
        assert p.aux.d_model == p.base.d_model and p.aux.layers[0] == p.base.layers[0]
