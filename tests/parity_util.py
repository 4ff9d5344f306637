"""Shared by the GPU parity tests: run the CUDA path through the C ABI and the CPU oracle on
the same seeded inputs and compare them the way the acceptance rule states it:
per base layer, separately for K_hat and V_hat over valid rows, and per sequence for logits,
||gpu - oracle||_F / ||oracle||_F <= 1e-2 in bf16 mode, <= 1e-4 in fp32 mode; the first token
must be identical wherever the oracle's top-2 logit gap exceeds 1e-3."""
import numpy as np

import workloads as wl
from oracle import kvp_oracle as orc

TOL = {"bf16": 1e-2, "f32": 1e-4}
GAP = 1e-3


def rel_fro(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def make_session(pair, W, prompts, extra_len=0):
    import paper_2410_08391_b200 as kvp
    return kvp.Session(pair, W, max_batch=prompts.batch, max_total_tokens=prompts.total,
                       max_len=int(prompts.lengths.max()), extra_len=extra_len)


def compare_prefill(sess, pair, W, prompts, seqs=None, gap=GAP):
    """Runs kvp_prefill_predict on the whole batch; compares the listed sequences with the oracle.
    Returns (worst K error, worst V error, worst logits error, n argmax compared)."""
    import torch
    toks = torch.from_numpy(prompts.tokens).to(sess.device)
    lens = [int(x) for x in prompts.lengths]
    logits, first = sess.prefill_predict(toks, lens)
    sess.poll()
    logits = logits.cpu().numpy()
    first = first.cpu().numpy()
    assert sess.cache.seq_lens[:len(lens)].cpu().tolist() == lens
    tol = TOL[pair.dtype]
    ek = ev = el = 0.0
    n_arg = 0
    ref = orc.prefill_predict(pair, W, prompts, seqs)
    for b, (kv_hat, ref_logits, ref_tok) in ref.items():
        for i in range(pair.base.n_layers):
            k, v = sess.cache.gather(i, b, lens[b])
            e1, e2 = rel_fro(k, kv_hat[i][0]), rel_fro(v, kv_hat[i][1])
            assert e1 <= tol and e2 <= tol, f"seq {b} base layer {i}: K err {e1:.3e} V err {e2:.3e} > {tol}"
            ek, ev = max(ek, e1), max(ev, e2)
        e3 = rel_fro(logits[b], ref_logits)
        assert e3 <= tol, f"seq {b}: logits err {e3:.3e} > {tol}"
        el = max(el, e3)
        assert int(first[b]) == int(np.argmax(logits[b])), "first token is not the argmax of the returned logits"
        if orc.top2_gap(ref_logits) > gap:
            assert int(first[b]) == ref_tok, f"seq {b}: first token {first[b]} != oracle {ref_tok}"
            n_arg += 1
    return ek, ev, el, n_arg
