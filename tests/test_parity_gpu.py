"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs, element by element.  Sizes span several tiles and ragged tails."""
import numpy as np
import pytest

import workloads as wl
from oracle import kvp_oracle as orc
from parity_util import (GAP, TOL, ArgmaxTally, assert_first_tokens, check_cache_layer, compare_prefill, compare_with_golden, load_golden,
                         make_session, rel_fro, run_prefill)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


CASES = [
    ("c1", None, "n002"),
    ("c1", None, "fanin"),
    ("c1_bf16", None, "n002"),
    ("t_small", [150, 37, 1, 64, 65], "n002"),
    ("t_small", [150, 37, 1, 64, 65], "fanin"),
    ("t_small_f32", [150, 37, 1, 64, 65], "fanin"),
    ("t_small_f32", [129], "n002"),
    ("t_hd128", [130, 70, 2], "fanin"),
    ("t_hd128", [200], "n002"),
    ("t_scaled", [100, 33, 257], "fanin"),
    ("t_scaled", [100, 33, 257], "n002"),
    ("t_bias", [40, 90], "fanin"),
    ("t_hd32", [150, 37, 1, 64, 65], "fanin"),      # predictor columns leave as 64-byte pieces (segment boundaries at 96)
    # layer-pruned auxiliary model (KVP-LP): same width as the base, square predictor matrices
    ("t_lp", [100, 59, 59, 7], "fanin"),
    ("t_lp", [130], "n002"),
    # more than 4 sequences: the step's projections run on the tensor cores (operand rows padded to 16, 24)
    ("t_hd128", [40, 9, 130, 17, 64, 65, 3, 90, 128], "fanin"),
    ("t_scaled", [20, 33, 5, 64, 65, 1, 40, 41, 42, 43, 44, 45, 46, 47, 48, 49, 50], "fanin"),
    # a cache of more than 4096 entries with a small batch: the step leaves the persistent kernel for the
    # tensor-core projections + ring-fed attention over 66 pages in several key-range splits
    ("t_small", [4200, 70], "fanin"),
    ("t_hd128", [4100], "n002"),
    # more sequences than the tensor-core step path takes (128): the CUDA-core projections serve the step;
    # many one- and two-token prompts
    ("t_small", [1, 2, 3, 5, 8, 13, 21, 34, 55, 89] * 13, "fanin"),
    # a layer map that skips an auxiliary layer: no predictor and no piece of the base step after that layer
    ("t_small_gap", [150, 37, 1, 64], "fanin"),
    ("t_small_gap", [40, 9, 130, 17, 64, 65], "n002"),
    # query / key norm (Sec. 7, "key norm"): bf16 with both head sizes (fused into the QKV epilogue and the
    # persistent step), fp32 (CUDA-core kernels), more than 4 sequences (tensor-core step projections +
    # ring attention), a long cache (paged step attention in splits) and the 130-sequence CUDA-core step
    ("t_small_qkn", [150, 37, 1, 64, 65], "fanin"),
    ("t_small_qkn", [129, 40], "n002"),
    ("t_small_qkn_f32", [129, 40, 1], "fanin"),
    ("t_hd128_qkn", [130, 70, 2], "fanin"),
    ("t_hd128_qkn", [40, 9, 130, 17, 64, 65, 3, 90, 128], "fanin"),
    ("t_small_qkn", [4200, 70], "fanin"),
    ("t_small_qkn", [1, 2, 3, 5, 8, 13, 21, 34, 55, 89] * 13, "fanin"),
    # many tokens: several waves of tiles per SM in every kernel of the prefill
    ("t_small", [1900] * 9 + [1901], "fanin"),
    # other group sizes of the step attention over the bf16 cache (1, 2 and 8 query heads per kv head), with more
    # than 4 sequences and with a small batch over a long cache
    ("t_mha", [40, 9, 130, 17, 64, 65], "fanin"),
    ("t_g2", [40, 9, 130, 17, 64, 65], "fanin"),
    ("t_g8", [40, 9, 130, 17, 64, 65], "fanin"),
    ("t_mha", [4130, 3], "fanin"),
    ("t_g2", [4130], "n002"),
    ("t_g8", [4130, 64], "fanin"),
]


@pytest.mark.parametrize("name,lens,regime", CASES, ids=lambda v: str(v).replace(" ", ""))
def test_prefill_predict_matches_oracle(name, lens, regime):
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=1, regime=regime)
    pr = wl.prompts(name, seed=1) if lens is None else wl.custom_prompts(pair.base.vocab, lens, seed=1)
    s = make_session(pair, W, pr)
    try:
        ek, ev, el, tally = compare_prefill(s, pair, W, pr)
        print(f"{name} {regime}: K {ek:.2e} V {ev:.2e} logits {el:.2e} argmax compared {tally.compared}/{pr.batch}")
        assert_first_tokens(tally, TOL[pair.dtype], f"{name} {regime}")
    finally:
        s.close()


@pytest.mark.parametrize("flags", [1, 2, 3])
@pytest.mark.parametrize("name,lens,regime", [("t_small", [1900] * 9 + [1901], "fanin"), ("t_hd128", [1300] * 9 + [1207], "n002"),
                                              ("t_small_qkn", [1900] * 10, "fanin"), ("t_bias", [1900] * 10, "fanin"),
                                              ("t_scaled", [1500] * 13, "fanin")],
                         ids=lambda v: str(v).replace(" ", "")[:40])
def test_kernel_variants_match_oracle(name, lens, regime, flags):
    """The schedule variants (kvp_options.flags: K/V projection + predictor as one kernel; RMSNorm as its own kernel
    instead of folded into the GEMMs around it) on calls large enough for the choice to matter (flags = 0, the default, is
    what every other many-token case runs): same results within the same tolerances."""
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=1, regime=regime)
    pr = wl.custom_prompts(pair.base.vocab, lens, seed=1)
    s = make_session(pair, W, pr, flags=flags)
    try:
        ek, ev, el, tally = compare_prefill(s, pair, W, pr, seqs=[0, len(lens) - 1])
        print(f"{name} flags {flags}: K {ek:.2e} V {ev:.2e} logits {el:.2e}")
        assert not tally.mismatches, tally.report()
    finally:
        s.close()


@pytest.mark.parametrize("name,regime,lens", [("t_small", "fanin", [70, 63, 5]), ("t_small_f32", "fanin", [70, 63, 5]),
                                              ("c1", "n002", [64]), ("t_small", "n002", [70, 63, 5, 64, 1, 30]),
                                              ("t_small_qkn", "fanin", [70, 63, 5]),
                                              ("t_small_qkn_f32", "fanin", [70, 5]),
                                              ("t_hd128_qkn", "fanin", [70, 63, 5, 64, 1, 30]),
                                              ("t_mha", "fanin", [70, 63, 5, 64, 1, 30]),
                                              ("t_g2", "fanin", [70, 63, 5, 64, 1, 30]),
                                              ("t_g8", "fanin", [70, 63, 5, 64, 1, 30])],
                         ids=lambda v: str(v).replace(" ", ""))
def test_decode_steps_match_oracle(name, regime, lens):
    import torch
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=2, regime=regime)
    pr = wl.custom_prompts(pair.base.vocab, lens, seed=2)
    steps = 3
    s = make_session(pair, W, pr, extra_len=steps)
    tol = TOL[pair.dtype]
    try:
        toks = torch.from_numpy(pr.tokens).to(s.device)
        s.prefill_predict(toks, lens)
        s.poll()
        ref = orc.prefill_predict(pair, W, pr)
        caches = {b: ref[b][0] for b in range(pr.batch)}
        cur = list(lens)
        g = np.random.default_rng(7)
        for step in range(steps):
            nxt = g.integers(0, pair.base.vocab, size=pr.batch).astype(np.int32)   # same forced token on both sides
            logits, tok = s.decode_step(torch.from_numpy(nxt).to(s.device), cur)
            s.poll()
            logits = logits.cpu().numpy()
            cur = [c + 1 for c in cur]
            assert s.cache.seq_lens[:pr.batch].cpu().tolist() == cur
            for b in range(pr.batch):
                ref_logits, caches[b] = orc.decode_step(pair, W, int(nxt[b]), caches[b])
                assert rel_fro(logits[b], ref_logits) <= tol
                if orc.top2_gap(ref_logits) > GAP:
                    assert int(tok[b]) == orc.argmax_lowest(ref_logits)
                for i in range(pair.base.n_layers):
                    k, v = s.cache.gather(i, b, cur[b])
                    assert rel_fro(k[-1], caches[b][i][0][-1]) <= tol
                    assert rel_fro(v[-1], caches[b][i][1][-1]) <= tol
                    assert rel_fro(k, caches[b][i][0]) <= tol
    finally:
        s.close()


@pytest.mark.parametrize("lens", [[70, 63, 5], [64, 1, 30, 9, 127, 128]], ids=lambda v: str(v).replace(" ", ""))
def test_recorded_decode_step_replays_for_later_positions(lens):
    """One kvp_decode_step recorded into a CUDA graph and replayed: positions come from seq_lens on the device and
    the token from a device buffer, so every replay is the next step of the generation loop (Fig. 2(b))."""
    import torch
    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=5, regime="fanin")
    pr = wl.custom_prompts(pair.base.vocab, lens, seed=5)
    steps = 3
    s = make_session(pair, W, pr, extra_len=steps + 1)
    tol = TOL[pair.dtype]
    try:
        s.prefill_predict(torch.from_numpy(pr.tokens).to(s.device), lens)
        s.poll()
        ref = orc.prefill_predict(pair, W, pr)
        caches = {b: ref[b][0] for b in range(pr.batch)}
        g = np.random.default_rng(9)
        forced = g.integers(0, pair.base.vocab, size=(steps + 1, pr.batch)).astype(np.int32)
        tok = torch.from_numpy(forced[0]).to(s.device)
        s.decode_step(tok, lens)                      # a warm-up step outside the recording (it is step 0)
        s.poll()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s.torch_stream):
            s.decode_step(tok, [c + 1 for c in lens])
        torch.cuda.synchronize()
        for b in range(pr.batch):
            _, caches[b] = orc.decode_step(pair, W, int(forced[0][b]), caches[b])
        cur = [c + 1 for c in lens]
        for step in range(1, steps + 1):
            tok.copy_(torch.from_numpy(forced[step]).to(s.device))
            torch.cuda.synchronize()
            with torch.cuda.stream(s.torch_stream):
                graph.replay()
            torch.cuda.synchronize()
            s.poll()
            logits = s.logits[:pr.batch].cpu().numpy()
            cur = [c + 1 for c in cur]
            assert s.cache.seq_lens[:pr.batch].cpu().tolist() == cur
            for b in range(pr.batch):
                ref_logits, caches[b] = orc.decode_step(pair, W, int(forced[step][b]), caches[b])
                assert rel_fro(logits[b], ref_logits) <= tol
                for i in range(pair.base.n_layers):
                    k, v = s.cache.gather(i, b, cur[b])
                    assert rel_fro(k, caches[b][i][0]) <= tol and rel_fro(v, caches[b][i][1]) <= tol
    finally:
        s.close()


TRAIN_CASES = [
    ("c1", None, "fanin"),                       # fp32, CUDA-core kernels
    ("t_small_f32", [129, 40, 1], "fanin"),
    ("t_small", [150, 37, 1, 64, 65], "fanin"),  # bf16, tensor-core GEMMs and attention, ragged
    ("t_small", [300], "n002"),
    ("t_hd128", [130, 70, 2], "fanin"),
    ("t_scaled", [100, 33, 257], "fanin"),       # heterogeneous layers
    ("t_small_qkn", [129, 40], "fanin"),         # query / key norm
]


@pytest.mark.parametrize("name,lens,regime", TRAIN_CASES, ids=lambda v: str(v).replace(" ", ""))
def test_train_forward_matches_oracle(name, lens, regime):
    """Training-time forward (Sec. 4.1): logits of every position from the base model on the predicted cache, and
    the consistency terms mean |KV_hat - KV_B| per base layer (Sec. 4.3), against the oracle."""
    import torch
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=6, regime=regime)
    pr = wl.prompts(name, seed=6) if lens is None else wl.custom_prompts(pair.base.vocab, lens, seed=6)
    lens = [int(x) for x in pr.lengths]
    s = make_session(pair, W, pr)
    tol = TOL[pair.dtype]
    try:
        toks = torch.from_numpy(pr.tokens).to(s.device)
        s.prefill_predict(toks, lens)
        logits, l1_k, l1_v = s.train_forward(toks, lens)
        s.poll()
        logits, l1_k, l1_v = logits.cpu().numpy(), l1_k.cpu().numpy(), l1_v.cpu().numpy()
        assert s.cache.seq_lens[:pr.batch].cpu().tolist() == lens
        nb = pair.base.n_layers
        abs_k, abs_v, cnt = np.zeros(nb), np.zeros(nb), np.zeros(nb)
        t0 = 0
        for b in range(pr.batch):
            ref_logits, ak, av, n = orc.train_forward(pair, W, pr.seq(b))
            abs_k += ak; abs_v += av; cnt += n
            got = logits[t0:t0 + lens[b]]
            assert rel_fro(got, ref_logits) <= tol, f"seq {b}: logits {rel_fro(got, ref_logits):.3e}"
            # the last row is the inference path's first step (also checked there); every row must hold on its own
            worst = max(rel_fro(got[t], ref_logits[t]) for t in range(lens[b]))
            assert worst <= tol, f"seq {b}: worst row {worst:.3e}"
            t0 += lens[b]
        # the predicted cache is rounded to the run dtype before it is compared: one bf16 rounding of O(1) entries
        slack = 4e-3 if pair.dtype == "bf16" else 1e-5
        for i in range(nb):
            for got, ref in ((l1_k[i], abs_k[i] / cnt[i]), (l1_v[i], abs_v[i] / cnt[i])):
                assert abs(got - ref) <= slack * max(ref, 1e-3) + 1e-6, f"layer {i}: {got} vs {ref}"
    finally:
        s.close()


def test_sequence_alone_equals_sequence_in_batch():
    import torch
    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=3, regime="fanin")
    pr = wl.custom_prompts(pair.base.vocab, [90, 200, 17], seed=3)
    s = make_session(pair, W, pr)
    try:
        lens = [int(x) for x in pr.lengths]
        logits, first = s.prefill_predict(torch.from_numpy(pr.tokens).to(s.device), lens)
        logits = logits.cpu().numpy().copy()
        kv = [s.cache.gather(i, 1, lens[1]) for i in range(pair.base.n_layers)]
        alone = wl.Prompts(pr.seq(1).copy(), np.array([lens[1]], np.int32))
        l1, _ = s.prefill_predict(torch.from_numpy(alone.tokens).to(s.device), [lens[1]])
        s.poll()
        for i in range(pair.base.n_layers):
            k, v = s.cache.gather(i, 0, lens[1])
            # rows are independent, but the residual GEMMs add their k-range partial sums with fp32
            # atomics whose split and order depend on the launch shape: equal up to that reassociation
            assert rel_fro(k, kv[i][0]) <= 3e-3
            assert rel_fro(v, kv[i][1]) <= 3e-3
        assert rel_fro(l1.cpu().numpy()[0], logits[1].astype(np.float64)) <= 3e-3
    finally:
        s.close()


def test_host_entry_point_matches_device_entry_point():
    import torch
    import paper_2410_08391_b200 as kvp
    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=4)
    pr = wl.custom_prompts(pair.base.vocab, [77, 130], seed=4)
    s = make_session(pair, W, pr)
    try:
        lens = [int(x) for x in pr.lengths]
        logits, first = s.prefill_predict(torch.from_numpy(pr.tokens).to(s.device), lens)
        a, fa = logits.cpu().numpy().copy(), first.cpu().numpy().copy()
        th = torch.from_numpy(pr.tokens).pin_memory()
        lh = torch.empty((2, pair.base.vocab), dtype=torch.float32).pin_memory()
        fh = torch.empty(2, dtype=torch.int32).pin_memory()
        kvp.kvp_prefill_predict_host(s.h, th, lens, s.cache, s.workspace, s.logits, lh, fh, s.stream)
        # two runs differ by the order of the residual GEMMs' fp32 atomic adds, nothing else
        for b in range(2):
            assert rel_fro(lh.numpy()[b], a[b].astype(np.float64)) <= 3e-3
            top2 = np.sort(a[b])[-2:]
            if top2[1] - top2[0] > 1e-3:
                assert fh.numpy()[b] == fa[b]
    finally:
        s.close()


def test_error_paths_report_status_and_keep_the_context_usable():
    import torch
    import paper_2410_08391_b200 as kvp
    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=5)
    pr = wl.custom_prompts(pair.base.vocab, [50, 20], seed=5)
    s = make_session(pair, W, pr)
    try:
        lens = [50, 20]
        toks = torch.from_numpy(pr.tokens).to(s.device)
        with pytest.raises(kvp.KvpError) as e:                     # prompt longer than the block table allows
            s.prefill_predict(toks, [65, 5])
        assert e.value.status == -5
        with pytest.raises(kvp.KvpError) as e:
            s.prefill_predict(toks, [50, 0])
        assert e.value.status == -1
        small = torch.empty(1024, dtype=torch.uint8, device=s.device)
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_prefill_predict(s.h, toks, lens, s.cache, small, s.logits, s.first, s.stream)
        assert e.value.status == -8
        bad = toks.clone()
        bad[3] = pair.base.vocab + 5                               # token id out of range: flagged, not dereferenced
        s.prefill_predict(bad, lens)
        with pytest.raises(kvp.KvpError) as e:
            s.poll()
        assert e.value.status == -9
        keep = s.cache.block_table.clone()
        s.cache.block_table[1, 0] = s.cache.n_pages + 3            # page index out of range: flagged, write skipped
        s.prefill_predict(toks, lens)
        with pytest.raises(kvp.KvpError) as e:
            s.poll()
        assert e.value.status == -9
        s.cache.block_table.copy_(keep)
        s.prefill_predict(toks, lens)                              # and the handle still works afterwards
        s.poll()
        # training-time forward: same argument checks; without a logits buffer only the consistency terms are computed
        l1 = torch.empty(pair.base.n_layers, dtype=torch.float32, device=s.device)
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_train_forward(s.h, toks, lens, s.cache, small, None, l1, l1.clone(), s.stream)
        assert e.value.status == -8
        _, k_only, v_only = s.train_forward(toks, lens, want_logits=False)
        _, k_both, v_both = s.train_forward(toks, lens, want_logits=True)
        s.poll()
        assert torch.allclose(k_only, k_both, rtol=1e-3) and torch.allclose(v_only, v_both, rtol=1e-3)   # fp32 atomic sums: order varies
        assert bool((k_only > 0).all()) and bool((v_only > 0).all())
        h2 = kvp.kvp_create(pair.aux, pair.base, pair.layer_map, pair.dtype)
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_prefill_predict(h2, toks, lens, s.cache, s.workspace, s.logits, s.first, s.stream)
        assert e.value.status == -4
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_train_forward(h2, toks, lens, s.cache, s.workspace, None, l1, l1.clone(), s.stream)
        assert e.value.status in (-4, -8)
        kvp.kvp_destroy(h2)
    finally:
        s.close()


def test_bounded_wait_runs_out_and_is_reported_as_timeout():
    """A device-side wait that nothing completes gives up after its limit: the kernel returns, the status word carries the
    code, kvp_poll_status reports KVP_ERR_TIMEOUT, and the same handle then runs the whole path correctly."""
    import torch
    import paper_2410_08391_b200 as kvp
    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=8, regime="fanin")
    pr = wl.custom_prompts(pair.base.vocab, [70, 33], seed=8)
    s = make_session(pair, W, pr)
    try:
        s.poll()
        kvp.kvp_selftest_wait_timeout(s.h, s.workspace, s.stream)
        with pytest.raises(kvp.KvpError) as e:
            s.poll()
        assert e.value.status == -7
        s.poll()                                   # the word was cleared by the poll that reported it
        ek, ev, el, tally = compare_prefill(s, pair, W, pr)
        assert not tally.mismatches
    finally:
        s.close()


def _full_size(name, seqs, golden=True):
    """kvp_prefill_predict on a benchmark configuration in the launch configuration the benchmark times.  Every
    sequence the stored oracle file follows is compared (logits, first token, sampled cache rows); `seqs` are followed
    by the oracle here, whole cache included."""
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=0)
    pr = wl.prompts(name, seed=0)
    s = make_session(pair, W, pr)
    try:
        logits, first = run_prefill(s, pr)
        lens = [int(x) for x in pr.lengths]
        tol = TOL[pair.dtype]
        g = load_golden(name) if golden else None
        if golden:
            assert g is not None, f"tests/golden/{name}_first_step.npz is missing (tests/golden/make_full_size_refs.py {name})"
            el, er, tally, per_seq = compare_with_golden(s, pair, pr, logits, first, g)
            print(f"{name}: {len(per_seq)} stored sequences, worst logits err {el:.2e}, worst sampled (token, head) slice {er:.2e}, "
                  f"argmax compared {tally.compared}; per sequence: " + " ".join(f"{b}:{e:.1e}" for b, e in per_seq.items()))
            assert_first_tokens(tally, tol, name)
        tally = ArgmaxTally()
        ref = orc.prefill_predict(pair, W, pr, seqs)
        for b, (kv_hat, ref_logits, _) in ref.items():
            worst = 0.0
            for i in range(pair.base.n_layers):
                k, v = s.cache.gather(i, b, lens[b])
                e1, e2, e3 = check_cache_layer(k, v, kv_hat[i][0], kv_hat[i][1], pair.base.layers[i].head_dim, tol, f"{name} seq {b} base layer {i}")
                worst = max(worst, e1, e2)
            e = rel_fro(logits[b], ref_logits)
            assert e <= tol, f"{name} seq {b}: logits err {e:.3e}"
            tally.add(b, first[b], logits[b], ref_logits)
            print(f"{name} seq {b} ({lens[b]} tokens), whole cache: worst K/V layer err {worst:.2e}, logits {e:.2e}")
        assert_first_tokens(tally, tol, name)
    finally:
        s.close()


def test_config_2_full_size_matches_oracle():
    """The 1.1B-shaped base with the 270M-shaped auxiliary model on the 1024-token prompt."""
    _full_size("c2", [0], golden=False)


def test_paper_shaped_batch_full_size_sampled_sequences_match_oracle():
    """64 prompts of 59 tokens (the TriviaQA 1-shot length of Sec. 6) on the 1.1B / 270M-shaped pair (step pieces on
    their own stream, tensor-core step projections); the oracle follows three sampled sequences."""
    _full_size("qa", [0, 31, 63], golden=False)


def test_layer_pruned_pair_full_size_sampled_sequences_match_oracle():
    """KVP-LP-0.25 of Table 1 (auxiliary = 7 of the base model's 28 layers) on the 64 x 59 batch."""
    _full_size("lp25", [5, 40], golden=False)


def test_prompt_length_sweep_batch_8_matches_oracle():
    """The batch-8 prompt-length sweep of Sec. 6 (TTFT against prompt length) at one of its lengths, 8 x 256 tokens."""
    pair = wl.pair("c2")
    W = wl.make_weights(pair, seed=0)
    pr = wl.sweep_prompts(256, seed=0)
    s = make_session(pair, W, pr)
    try:
        ek, ev, el, tally = compare_prefill(s, pair, W, pr, seqs=[0, 7])
        print(f"sweep8 256: K {ek:.2e} V {ev:.2e} logits {el:.2e} argmax compared {tally.compared}")
        assert not tally.mismatches, tally.report()
    finally:
        s.close()


def test_train_forward_config_2_sampled_rows_match_oracle():
    """Training-time forward at the benchmark's size (C2 pair); the oracle runs the first 192 tokens of the prompt:
    rows of a causal forward do not depend on later tokens, so they must equal the rows of the full-size run."""
    import torch
    pair = wl.pair("c2")
    W = wl.make_weights(pair, seed=0)
    pr = wl.prompts("c2", seed=0)
    lens = [int(x) for x in pr.lengths]
    s = make_session(pair, W, pr)
    try:
        toks = torch.from_numpy(pr.tokens).to(s.device)
        s.prefill_predict(toks, lens)
        logits, l1_k, l1_v = s.train_forward(toks, lens)
        s.poll()
        n = 192
        ref_logits, _, _, _ = orc.train_forward(pair, W, pr.seq(0)[:n])
        got = logits[:n].cpu().numpy()
        # every projection operand of this forward travels as a bf16 value plus its bf16 remainder and the attention takes
        # IEEE halves, so the ordinary tolerance holds for the whole block of rows and for every row on its own
        e_all = rel_fro(got, ref_logits)
        e_row = max(rel_fro(got[t], ref_logits[t]) for t in range(n))
        print(f"c2 training-time forward, first {n} rows: logits err {e_all:.2e}, worst row {e_row:.2e}")
        assert e_all <= TOL[pair.dtype] and e_row <= TOL[pair.dtype]
        assert bool((l1_k > 0).all()) and bool((l1_v > 0).all())
    finally:
        s.close()


def test_config_3_full_size_all_sequences_match_oracle():
    """3B-shaped base, 450M-shaped auxiliary model, 8 ragged prompts (25 240 tokens): all 8 sequences against the
    stored oracle results, the shortest one against the oracle run here with its whole cache."""
    pr = wl.prompts("c3", seed=0)
    _full_size("c3", [int(np.argmin(pr.lengths))])


def test_config_4_full_size_all_sequences_match_oracle():
    """Layer-wise scaled pair, non-uniform map, 32 x 2048 tokens: all 32 sequences against the stored oracle results
    (logits, first token, sampled cache rows); the sequence whose logits are the most sensitive to the cache's
    storage rounding (largest stored `floor_f16`) is followed by the oracle here with its whole cache."""
    g = load_golden("c4")
    assert g is not None
    _full_size("c4", [int(g["seqs"][int(np.argmax(g["floor_f16"]))])])


def test_config_5_long_prompts_match_oracle():
    """4 x 16 384 tokens, the launch shape of the long-cache step (key-range splits over 256 pages).
    (1) One whole sequence against the stored oracle run: first-step logits, first token, 24 sampled cache rows over the
        whole length in every base layer.
    (2) Every sequence: the GPU's own predicted cache is downloaded and the ORACLE's base step runs on it
        (b <- B(I[-1], KV_B_hat), Fig. 2(b)); logits and first token of the GPU's step must match it.  This isolates the
        step over 16 384 cached entries from the prefill.
    (3) Causality makes cache rows < n a function of the first n tokens: the oracle runs the first 4096 tokens of another
        sequence and every row of the GPU's cache prefix is compared, page tails included."""
    pair = wl.pair("c5")
    W = wl.make_weights(pair, seed=0)
    pr = wl.prompts("c5", seed=0)
    s = make_session(pair, W, pr)
    tol = TOL[pair.dtype]
    try:
        logits, first = run_prefill(s, pr)
        assert np.isfinite(logits).all()
        lens = [int(x) for x in pr.lengths]
        g = load_golden("c5")
        assert g is not None, "tests/golden/c5_first_step.npz is missing"
        el, er, tally, per_seq = compare_with_golden(s, pair, pr, logits, first, g)
        print(f"c5 stored sequence(s) {list(per_seq)}: logits err {el:.2e}, worst sampled (token, head) slice {er:.2e}, argmax compared {tally.compared}")
        assert_first_tokens(tally, tol, "c5")
        tally = ArgmaxTally()
        for b in range(pr.batch):
            kv = []
            for i in range(pair.base.n_layers):
                k, v = s.cache.gather(i, b, lens[b])
                kv.append((k.astype(np.float64), v.astype(np.float64)))
            ref_logits = orc.base_first_step(pair, W, int(pr.seq(b)[-1]), kv)
            e = rel_fro(logits[b], ref_logits)
            print(f"c5 seq {b}: step on the GPU's own cache vs oracle step on the same cache: logits err {e:.2e}, gap {orc.top2_gap(ref_logits):.2e}")
            assert e <= tol
            tally.add(b, first[b], logits[b], ref_logits)
        assert_first_tokens(tally, tol, "c5 step on the GPU's own cache")
        n, b = 4096, 1
        kv_hat = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, pr.seq(b)[:n]))
        worst = 0.0
        for i in range(pair.base.n_layers):
            k, v = s.cache.gather(i, b, n)
            e1, e2, _ = check_cache_layer(k, v, kv_hat[i][0], kv_hat[i][1], pair.base.layers[i].head_dim, tol, f"c5 seq {b} prefix base layer {i}")
            worst = max(worst, e1, e2)
        print(f"c5 seq {b} prefix {n}: worst K/V err {worst:.2e}")
    finally:
        s.close()
