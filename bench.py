#!/usr/bin/env python
"""Benchmark of the KV Prediction time-to-first-token path.

A step is one kvp_prefill_predict call: auxiliary prefill over the whole prompt batch, KV
prediction into the paged base cache, and the base model's first step.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

N > 1 runs N independent replicas (the path has no cross-sequence exchange; one process per
GPU, launched by torch.distributed.run); value = N * tokens / max-over-ranks time.
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as wl  # noqa: E402

METRIC = "prompt tok/s over TTFT (aux prefill + KV predict + base first step)"
UNIT = "tok/s"
REF_SAMPLE_TOKENS = 256


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for ts, r in self.rows if t0 - 0.02 <= ts <= t1 + 0.05 and len(r) >= 7] or [r for _, r in self.rows if len(r) >= 7][-3:]
        if not rows:
            return None
        sm = [float(r[0]) for r in rows]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=float(rows[0][1]), samples=len(rows), reasons=reasons)


def time_oracle(pair, W, prompts, seqs=None):
    from oracle import kvp_oracle as orc
    t = time.perf_counter()
    orc.prefill_predict(pair, W, prompts, seqs)
    return time.perf_counter() - t


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the replicas run side by side, the job is done when the last one is."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Prompt tokens per second of all replicas together."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def measured_traffic(workload: str, kernel_class: str):
    """DRAM bytes per launch of a kernel class from the committed ncu capture, or None when there is no
    capture for this workload / class or the kernel's source has changed since it was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    for rec in json.load(open(path)):
        if rec["workload"] == workload and rec["kernel_class"] == kernel_class:
            src = os.path.join(ROOT, rec["source"])
            if os.path.exists(src) and hashlib.sha256(open(src, "rb").read()).hexdigest() == rec["source_sha256"]:
                return rec["dram_bytes_per_launch"]
    return None


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pair = wl.pair(args.workload)
    W = wl.make_weights(pair, seed=0)
    full = wl.prompts(args.workload, seed=0)
    n = min(REF_SAMPLE_TOKENS, int(full.lengths[0]))
    sample = wl.Prompts(full.seq(0)[:n].copy(), np.array([n], np.int32))
    for _ in range(args.warmup):
        time_oracle(pair, W, sample)
    ts = [time_oracle(pair, W, sample) for _ in range(args.steps)]
    t = sum(ts) / len(ts)
    val = n / t
    desc = f"first {n} tokens of sequence 0 of workload {args.workload}, whole path, fp64 numpy"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4", "c5", "qa", "lp75", "lp50", "lp25"])
    ap.add_argument("--impl", default="kvp", choices=["kvp", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--train-forward", action="store_true",
                    help="also time the training-time forward (base model over the whole prompt on the predicted cache)")
    ap.add_argument("--decode-steps", type=int, default=16, help="generation steps timed after the TTFT measurement (0 = none)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "kvp" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import __graft_entry__ as ge
    ge.build()
    import paper_2410_08391_b200 as kvp

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = f"cuda:{local}"
    torch.cuda.set_device(dev)

    pair = wl.pair(args.workload)
    W = wl.make_weights(pair, seed=0)
    pr = wl.prompts(args.workload, seed=0)
    lens = [int(x) for x in pr.lengths]
    work = wl.algorithmic_work(pair, lens)
    sess = kvp.Session(pair, W, max_batch=pr.batch, max_total_tokens=pr.total, max_len=max(lens), device=dev,
                       extra_len=2 * max(args.decode_steps, 0) + 4)
    toks = torch.from_numpy(pr.tokens).to(dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def step():
        sess.prefill_predict(toks, lens)

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    sess.poll()
    # ---- timed region: K steps, device time by CUDA events on the launching stream ----
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = kvp.kvp_launch_count(sess.h)
    barrier()
    t0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    t1 = time.time()
    launches = kvp.kvp_launch_count(sess.h) - n0
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None
    sess.poll()
    ms = max_over_ranks(ms, dist, dev)
    ms_step = ms / args.steps
    value = whole_job_value(work["tokens"], world, ms_step)

    # ---- end to end through the host entry point: pinned host tokens in, host logits out ----
    th = torch.from_numpy(pr.tokens).pin_memory()
    lh = torch.empty((pr.batch, pair.base.vocab), dtype=torch.float32).pin_memory()
    fh = torch.empty(pr.batch, dtype=torch.int32).pin_memory()

    def step_host():
        kvp.kvp_prefill_predict_host(sess.h, th, lens, sess.cache, sess.workspace, sess.logits, lh, fh, sess.stream)

    for _ in range(args.warmup):
        step_host()
    barrier()
    w0 = time.perf_counter()
    for _ in range(args.steps):
        step_host()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - w0) * 1e3 / args.steps
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    e2e_value = whole_job_value(work["tokens"], world, e2e_ms)

    # ---- generation loop after the first token (Fig. 2(b), loop body): secondary figure ----
    decode = None
    if args.decode_steps > 0:
        step()                                  # a fresh predicted cache and first tokens
        cur = list(lens)
        tok = sess.first[:pr.batch].clone()
        for _ in range(3):                      # warm-up steps (they extend the cache too)
            _, nxt = sess.decode_step(tok, cur)
            tok = nxt.clone()
            cur = [c + 1 for c in cur]
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        d0.record(stream)
        for _ in range(args.decode_steps):
            _, nxt = sess.decode_step(tok, cur)
            tok.copy_(nxt)
            cur = [c + 1 for c in cur]
        d1.record(stream)
        torch.cuda.synchronize()
        sess.poll()
        dms = max_over_ranks(d0.elapsed_time(d1) / args.decode_steps, dist, dev)
        decode = {"steps": args.decode_steps, "ms_per_step": dms, "tok_per_s": world * pr.batch / (dms * 1e-3),
                  "ttft_over_step": ms_step / dms}
        # the same loop as ONE recorded step replayed: positions live in seq_lens on the device, the fed-back token
        # in `tok`, so a recorded kvp_decode_step stays valid while the block table has room
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=sess.torch_stream):
            _, nxt = sess.decode_step(tok, cur)
            tok.copy_(nxt)
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(sess.torch_stream)
        with torch.cuda.stream(sess.torch_stream):
            for _ in range(args.decode_steps):
                graph.replay()
        g1.record(sess.torch_stream)
        torch.cuda.synchronize()
        sess.poll()
        want = [c + args.decode_steps for c in cur]
        assert sess.cache.seq_lens[:pr.batch].cpu().tolist() == want, "replayed steps did not advance the cache"
        gms = max_over_ranks(g0.elapsed_time(g1) / args.decode_steps, dist, dev)
        decode.update({"graph_ms_per_step": gms, "graph_tok_per_s": world * pr.batch / (gms * 1e-3)})

    # ---- training-time forward (Sec. 4.1 "Training"): secondary figure, on request ----
    train = None
    if args.train_forward:
        step()
        for _ in range(2):
            sess.train_forward(toks, lens)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        n_tf = max(3, min(args.steps, 10))
        t0.record(stream)
        for _ in range(n_tf):
            sess.train_forward(toks, lens)
        t1.record(stream)
        torch.cuda.synchronize()
        sess.poll()
        tms = max_over_ranks(t0.elapsed_time(t1) / n_tf, dist, dev)
        tf = wl.train_forward_flops(pair, lens)
        pk = measured_peaks()
        pk_tf = (pk["bf16_tflops_sustained"] or pk["bf16_tflops"]) / (16.0 if pair.dtype == "f32" else 1.0)
        train = {"ms": tms, "tok_per_s": world * work["tokens"] / (tms * 1e-3), "tflops": tf / (tms * 1e-3) / 1e12,
                 "algorithmic_tflop": tf / 1e12, "frac_of_tensor_peak": tf / (tms * 1e-3) / 1e12 / pk_tf,
                 "peak": pk_tf, "peak_source": pk["source"]}

    # ---- per-kernel-class device times (separate pass: events around every launch) ----
    kvp.kvp_timing_enable(sess.h, True)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize()
    classes = kvp.kvp_timing_read(sess.h)
    kvp.kvp_timing_enable(sess.h, False)
    per_step = {c: (v[0] / args.steps, v[1] // args.steps) for c, v in classes.items()}
    peaks = measured_peaks()
    alg = {  # algorithmic work of each class per step: (amount, bound, unit scale)
        "aux_gemm": (work["aux_gemm_flops"], "tensor"), "aux_attn": (work["attn_flops"], "tensor"),
        "predictor": (work["pred_flops"], "tensor"), "step_gemv": (work["step_weight_bytes"], "hbm"),
        "step_attn": (work["cache_bytes"], "hbm"), "step_fused": (work["step_bytes"], "hbm"),
    }
    dom = max(alg, key=lambda c: per_step[c][0])
    amount, bound = alg[dom]
    t_dom = per_step[dom][0] * 1e-3
    if bound == "tensor":
        # kernels are timed inside a long step: the sustained figure is the denominator
        peak = peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]
        if pair.dtype == "f32":
            peak = peak / 16.0      # fp32 CUDA-core path; nominal ratio, context only
        achieved, unit = amount / t_dom / 1e12, "TFLOP/s"
    else:
        peak, achieved, unit = peaks["hbm_gbs"], amount / t_dom / 1e9, "GB/s"
    roofline = {"kernel_class": dom, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": measured_traffic(args.workload, dom),
                "algorithmic_per_launch": amount / max(per_step[dom][1], 1), "peak_source": peaks["source"],
                "launches_per_step": per_step[dom][1], "avg_launch_ms": per_step[dom][0] / max(per_step[dom][1], 1),
                "class_ms_per_step": {c: round(v[0], 4) for c, v in per_step.items()},
                "timing": "separate pass with CUDA events around every launch"}
    def frac_of(c):
        amt, bnd = alg[c]
        t = per_step[c][0] * 1e-3
        if t <= 0:
            return None
        if bnd == "tensor":
            pk = (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]) / (16.0 if pair.dtype == "f32" else 1.0)
            return {"bound": bnd, "achieved": amt / t / 1e12, "peak": pk, "unit": "TFLOP/s", "frac": amt / t / 1e12 / pk}
        return {"bound": bnd, "achieved": amt / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": amt / t / 1e9 / peaks["hbm_gbs"]}
    roofline["per_class"] = {c: frac_of(c) for c in alg if per_step[c][0] > 0}
    t12 = (per_step["aux_gemm"][0] + per_step["aux_attn"][0] + per_step["predictor"][0]) * 1e-3
    tensor_frac = work["tensor_flops"] / max(t12, 1e-12) / 1e12 / (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"])

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "ttft_ms": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": pair.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "batch": pr.batch, "prompt_tokens": work["tokens"],
                   "lengths": lens if len(lens) <= 8 else f"{len(lens)} x {lens[0]}",
                   "l2": "inputs larger than L2 (weights + cache read every step)", "parallelism": "replicas only"},
        "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": int(pr.total * 4),
                "d2h_bytes_per_step": int(pr.batch * pair.base.vocab * 4 + pr.batch * 4)},
        "roofline": roofline,
        "tensor_frac_stage12": tensor_frac,
        "decode": decode,
        "train_forward": train,
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands, on the host cores, on a bounded sample of the same workload
        b = int(np.argmin(pr.lengths))
        n = min(int(pr.lengths[b]), 1024)
        sample = wl.Prompts(pr.seq(b)[:n].copy(), np.array([n], np.int32))
        t = time_oracle(pair, W, sample)
        out["cpu_baseline"] = {"value": n / t, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                               "sample": f"{n} tokens of sequence {b} of workload {args.workload}, whole path, {t:.1f} s"}
    sess.close()
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
