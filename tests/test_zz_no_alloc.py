"""kvp_decode_step_static: the generation step for callers that cannot hand the library a workspace
because they must not allocate device memory at that point (a frozen memory pool, a serving loop
where cudaMalloc would stall the device, a host application that owns the allocator).  Its scratch
is an array built into the library, shared by all calls, so the test runs two steps in a row and
checks each against kvp_decode_step with an ordinary workspace."""
import numpy as np
import pytest

import workloads as wl
from oracle import kvp_oracle as orc
from parity_util import TOL, make_session, rel_fro

pytestmark = pytest.mark.gpu


def test_static_scratch_step_matches_workspace_step_twice_in_a_row():
    import torch
    import __graft_entry__ as ge
    ge.build()
    import paper_2410_08391_b200 as kvp

    pair = wl.pair("t_small")
    W = wl.make_weights(pair, seed=11, regime="fanin")
    lens = [150, 9, 64]          # 150 keys: the split-attention partials in the scratch are exercised
    pr = wl.custom_prompts(pair.base.vocab, lens, seed=11)
    a = make_session(pair, W, pr, extra_len=2)      # reference: caller-provided workspace
    b = make_session(pair, W, pr, extra_len=2)      # under test: built-in scratch
    try:
        toks = torch.from_numpy(pr.tokens).to(a.device)
        for s in (a, b):
            s.prefill_predict(toks, lens)
            s.poll()
        status = torch.full((1,), -1, dtype=torch.int32, device=a.device)
        cur = list(lens)
        g = np.random.default_rng(3)
        ref = orc.prefill_predict(pair, W, pr)
        caches = {i: ref[i][0] for i in range(len(lens))}
        for step in range(2):
            forced = g.integers(0, pair.base.vocab, size=len(lens)).astype(np.int32)
            nxt = torch.from_numpy(forced).to(a.device)
            la, ta = a.decode_step(nxt, cur)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            c = b.enter()
            kvp.kvp_decode_step_static(b.h, nxt, cur, b.cache, b.logits, b.first, status, b.stream)
            b.leave(c)
            torch.cuda.synchronize()
            # (the very first call makes the driver load the library image that holds the array: once per process)
            assert step == 0 or torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
            assert int(status.item()) == 0
            for i in range(len(lens)):       # and against the oracle's generation step
                ref_logits, caches[i] = orc.decode_step(pair, W, int(forced[i]), caches[i])
                assert rel_fro(b.logits[i].cpu().numpy(), ref_logits) <= TOL[pair.dtype]
            la, lb = la.cpu().numpy(), b.logits[:len(lens)].cpu().numpy()
            for i in range(len(lens)):
                assert rel_fro(lb[i], la[i].astype(np.float64)) <= TOL[pair.dtype]
            assert ta.cpu().tolist() == b.first[:len(lens)].cpu().tolist()
            cur = [c + 1 for c in cur]
            assert b.cache.seq_lens[:len(lens)].cpu().tolist() == cur
            for i in range(pair.base.n_layers):
                ka, va = a.cache.gather(i, 0, cur[0])
                kb, vb = b.cache.gather(i, 0, cur[0])
                # the two sessions' prefills differ by the order of fp32 atomic adds, hence not bit for bit
                assert rel_fro(kb, ka.astype(np.float64)) <= TOL[pair.dtype]
                assert rel_fro(vb, va.astype(np.float64)) <= TOL[pair.dtype]
        # a smaller step (batch 1) right after the batch-3 steps, on the array's stale contents
        one = wl.custom_prompts(pair.base.vocab, [77], seed=12)
        a1, b1 = make_session(pair, W, one, extra_len=2), make_session(pair, W, one, extra_len=2)
        try:
            t1 = torch.from_numpy(one.tokens).to(a.device)
            for s in (a1, b1):
                s.prefill_predict(t1, [77])
                s.poll()
            n1 = torch.tensor([5], dtype=torch.int32, device=a.device)
            l1, _ = a1.decode_step(n1, [77])
            c = b1.enter()
            kvp.kvp_decode_step_static(b1.h, n1, [77], b1.cache, b1.logits, b1.first, status, b1.stream)
            b1.leave(c)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert rel_fro(b1.logits[0].cpu().numpy(), l1[0].cpu().numpy().astype(np.float64)) <= TOL[pair.dtype]
            # an out-of-range token id: the access is skipped and status_out carries the code (2 = bad token id)
            bad = torch.tensor([pair.base.vocab + 7], dtype=torch.int32, device=a.device)
            c = b1.enter()
            kvp.kvp_decode_step_static(b1.h, bad, [78], b1.cache, b1.logits, b1.first, status, b1.stream)
            b1.leave(c)
            torch.cuda.synchronize()
            assert int(status.item()) == 2
        finally:
            a1.close()
            b1.close()
        # a step that does not fit the built-in array is refused with a message, nothing is launched
        big = wl.pair("c3")
        h = kvp.kvp_create(big.aux, big.base, big.layer_map, big.dtype)
        n0 = kvp.kvp_launch_count(h)
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_decode_step_static(h, nxt, [5] * 256, b.cache, b.logits, b.first, status, b.stream)
        assert e.value.status == -8 and "built-in array" in str(e.value)
        assert kvp.kvp_launch_count(h) == n0
        kvp.kvp_destroy(h)
    finally:
        a.close()
        b.close()
