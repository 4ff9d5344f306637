#!/usr/bin/env python
"""Benchmark of the KV Prediction time-to-first-token path.

A step is one kvp_prefill_predict call: auxiliary prefill over the whole prompt batch, KV
prediction into the paged base cache, and the base model's first step.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--also c3,c4,c2,qa,sweep8]
                  [--impl reference]

The headline (`value`, `ms_per_step`, `roofline`, `e2e`) is measured on --workload (default: the
largest single-GPU configuration, 4 x 16 384 tokens on the 3B / 450M-shaped pair).  The other
configurations named by --also are measured in the same run with fewer steps and reported under
`configs` (TTFT, tok/s, per-class roofline fractions against both measured tensor peaks, clocks).
N > 1 runs N independent replicas (the path has no cross-sequence exchange; one process per GPU;
when the script is not already running under torch.distributed.run it starts it itself);
value = N * tokens / max-over-ranks time.
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
WORKLOADS = ["c1", "c2", "c3", "c4", "c5", "qa", "lp75", "lp50", "lp25", "sweep8"]
ALSO_DEFAULT = "c3,c4,c2,qa,sweep8"      # c3 shares the headline pair, the last three share the 1.1B / 270M-shaped pair


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained") or d["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU for the whole run; window() summarises
    the samples that fall inside one timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

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

    def window(self, t0: float, t1: float):
        if not self.proc:
            return None
        time.sleep(0.06)
        good = [(ts, r) for ts, r in list(self.rows) if len(r) >= 7]
        rows = [r for ts, r in good if t0 - 0.02 <= ts <= t1 + 0.05] or [r for ts, r in good if ts <= t1 + 0.05][-3:]
        if not rows:
            return None
        sm = [float(r[0]) for r in rows]
        reasons = [n for i, n in enumerate(self.NAMES) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=float(rows[0][1]), samples=len(rows), reasons=reasons)

    def stop(self):
        if self.proc:
            self.proc.terminate()


def tensor_denominator(peaks, clocks):
    """Which measured tensor peak a region is held against: the burst figure when the sampled SM clock stayed at
    its maximum with no power-cap reason active, the sustained one otherwise."""
    if clocks and "sw_power_cap" not in clocks["reasons"] and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"]:
        return peaks["bf16_tflops"], "burst"
    return peaks["bf16_tflops_sustained"], "sustained"


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


def replica_command(argv, n_gpus: int, port: int):
    """Command line that runs this script as n_gpus replicas, one process per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), *argv]


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
    name = "c2" if args.workload == "sweep8" else args.workload
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=0)
    full = wl.prompts(name, seed=0)
    n = min(REF_SAMPLE_TOKENS, int(full.lengths[0]))
    sample = wl.Prompts(full.seq(0)[:n].copy(), np.array([n], np.int32))
    # One oracle step on the 3B-shaped pair takes tens of seconds whatever the sample (its base step converts every
    # weight to fp64), so the number of steps is bounded to keep the whole run within a few minutes; the line says so.
    big = pair.base.d_model > 2048
    warmup, steps = (min(args.warmup, 1), min(args.steps, 3)) if big else (args.warmup, args.steps)
    for _ in range(warmup):
        time_oracle(pair, W, sample)
    ts = [time_oracle(pair, W, sample) for _ in range(max(steps, 1))]
    t = sum(ts) / len(ts)
    val = n / t
    desc = f"first {n} tokens of sequence 0 of workload {args.workload}, whole path, fp64 numpy"
    if (warmup, steps) != (args.warmup, args.steps):
        desc += f"; {steps} timed steps after {warmup} warm-up (asked for {args.steps} / {args.warmup}: bounded to a few minutes)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Bench:
    """One process's view of the run: device, replicas, peaks, clock sampler."""

    def __init__(self, args):
        import torch
        import __graft_entry__ as ge
        ge.build()
        import paper_2410_08391_b200 as kvp
        self.torch, self.kvp, self.args = torch, kvp, args
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{self.local}"))
            self.dist = dist
        self.dev = f"cuda:{self.local}"
        torch.cuda.set_device(self.dev)
        self.peaks = measured_peaks()
        self.sampler = ClockSampler(self.local) if self.rank == 0 else None
        self._weights = {}

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def weights(self, pair):
        key = (pair.aux, pair.base, pair.layer_map, pair.dtype)
        if key not in self._weights:
            self._weights.clear()               # one pair's weights on the host at a time
            self._weights[key] = wl.make_weights(pair, seed=0)
        return self._weights[key]

    def measure(self, name: str, pair, pr, steps: int, warmup: int, full: bool):
        """Times kvp_prefill_predict on one prompt batch.  full: also the end-to-end host entry point, the generation
        loop and (on request) the training-time forward."""
        torch, kvp, args = self.torch, self.kvp, self.args
        dev, dist, world = self.dev, self.dist, self.world
        W = self.weights(pair)
        lens = [int(x) for x in pr.lengths]
        work = wl.algorithmic_work(pair, lens)
        decode_steps = max(args.decode_steps, 0) if full else 0
        sess = kvp.Session(pair, W, max_batch=pr.batch, max_total_tokens=pr.total, max_len=max(lens), device=dev,
                           extra_len=2 * decode_steps + 4, flags=args.opt_flags)
        toks = torch.from_numpy(pr.tokens).to(dev)

        def step():
            sess.prefill_predict(toks, lens)

        for _ in range(warmup):
            step()
        sess.poll()
        # ---- timed region: K steps, device time by CUDA events on the launching stream ----
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = kvp.kvp_launch_count(sess.h)
        self.barrier()
        t0 = time.time()
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        self.barrier()
        t1 = time.time()
        launches = kvp.kvp_launch_count(sess.h) - n0
        ms = e0.elapsed_time(e1)
        clocks = self.sampler.window(t0, t1) if self.sampler else None
        sess.poll()
        ms_step = max_over_ranks(ms, dist, dev) / steps
        out = {"workload": name, "batch": pr.batch, "prompt_tokens": work["tokens"],
               "lengths": lens if len(lens) <= 8 else f"{len(lens)} x {lens[0]}",
               "steps": steps, "ttft_ms": ms_step, "tok_per_s": whole_job_value(work["tokens"], world, ms_step),
               "gpu_launches": launches, "clocks": clocks}

        # ---- end to end through the host entry point: pinned host tokens in, host logits out ----
        th = torch.from_numpy(pr.tokens).pin_memory()
        lh = torch.empty((pr.batch, pair.base.vocab), dtype=torch.float32).pin_memory()
        fh = torch.empty(pr.batch, dtype=torch.int32).pin_memory()

        def step_host():
            kvp.kvp_prefill_predict_host(sess.h, th, lens, sess.cache, sess.workspace, sess.logits, lh, fh, sess.stream)

        for _ in range(warmup):
            step_host()
        self.barrier()
        w0 = time.perf_counter()
        for _ in range(steps):
            step_host()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks((time.perf_counter() - w0) * 1e3 / steps, dist, dev)
        out["e2e"] = {"value": whole_job_value(work["tokens"], world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                      "h2d_bytes_per_step": int(pr.total * 4),
                      "d2h_bytes_per_step": int(pr.batch * pair.base.vocab * 4 + pr.batch * 4)}

        # ---- generation loop after the first token (Fig. 2(b), loop body): secondary figure ----
        if decode_steps > 0:
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
            for _ in range(decode_steps):
                _, nxt = sess.decode_step(tok, cur)
                tok.copy_(nxt)
                cur = [c + 1 for c in cur]
            d1.record(stream)
            torch.cuda.synchronize()
            sess.poll()
            dms = max_over_ranks(d0.elapsed_time(d1) / decode_steps, dist, dev)
            decode = {"steps": decode_steps, "ms_per_step": dms, "tok_per_s": world * pr.batch / (dms * 1e-3),
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
                for _ in range(decode_steps):
                    graph.replay()
            g1.record(sess.torch_stream)
            torch.cuda.synchronize()
            sess.poll()
            want = [c + decode_steps for c in cur]
            assert sess.cache.seq_lens[:pr.batch].cpu().tolist() == want, "replayed steps did not advance the cache"
            gms = max_over_ranks(g0.elapsed_time(g1) / decode_steps, dist, dev)
            decode.update({"graph_ms_per_step": gms, "graph_tok_per_s": world * pr.batch / (gms * 1e-3),
                           "step_bytes": work["step_bytes"], "graph_hbm_gbs": work["step_bytes"] / (gms * 1e-3) / 1e9,
                           "graph_frac_of_hbm_peak": work["step_bytes"] / (gms * 1e-3) / 1e9 / self.peaks["hbm_gbs"]})
            out["decode"] = decode

        # ---- training-time forward (Sec. 4.1 "Training"): secondary figure, on request ----
        if full and args.train_forward:
            step()
            for _ in range(2):
                sess.train_forward(toks, lens)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            n_tf = max(3, min(steps, 10))
            a0.record(stream)
            for _ in range(n_tf):
                sess.train_forward(toks, lens)
            a1.record(stream)
            torch.cuda.synchronize()
            sess.poll()
            tms = max_over_ranks(a0.elapsed_time(a1) / n_tf, dist, dev)
            tf = wl.train_forward_flops(pair, lens)
            pk_tf = self.peaks["bf16_tflops_sustained"] / (16.0 if pair.dtype == "f32" else 1.0)
            out["train_forward"] = {"ms": tms, "tok_per_s": world * work["tokens"] / (tms * 1e-3), "tflops": tf / (tms * 1e-3) / 1e12,
                                    "algorithmic_tflop": tf / 1e12, "frac_of_tensor_peak": tf / (tms * 1e-3) / 1e12 / pk_tf,
                                    "peak": pk_tf, "peak_source": self.peaks["source"]}

        # ---- per-kernel-class device times (separate pass: events around every launch) ----
        kvp.kvp_timing_enable(sess.h, True)
        n_cls = min(steps, 5)
        for _ in range(n_cls):
            step()
        torch.cuda.synchronize()
        classes = kvp.kvp_timing_read(sess.h)
        kvp.kvp_timing_enable(sess.h, False)
        per_step = {c: (v[0] / n_cls, v[1] // n_cls) for c, v in classes.items()}
        peaks = self.peaks
        tpeak, which = tensor_denominator(peaks, clocks)
        scale = 16.0 if pair.dtype == "f32" else 1.0       # fp32 CUDA-core path; nominal ratio, context only
        alg = {  # algorithmic work of each class per step and the roofline that bounds it
            "aux_gemm": (work["aux_gemm_flops"], "tensor"), "aux_attn": (work["attn_flops"], "tensor"),
            "predictor": (work["pred_flops"], "tensor"), "step_gemv": (work["step_weight_bytes"], "hbm"),
            "step_attn": (work["cache_bytes"], "hbm"), "step_fused": (work["step_bytes"], "hbm"),
        }

        def frac_of(c):
            amt, bnd = alg[c]
            t = per_step[c][0] * 1e-3
            if t <= 0:
                return None
            if bnd == "tensor":
                a = amt / t / 1e12
                return {"bound": bnd, "achieved": a, "unit": "TFLOP/s", "peak": tpeak / scale, "peak_kind": which,
                        "frac": a / (tpeak / scale), "frac_of_burst": a / (peaks["bf16_tflops"] / scale),
                        "frac_of_sustained": a / (peaks["bf16_tflops_sustained"] / scale),
                        "ms": per_step[c][0], "launches": per_step[c][1]}
            a = amt / t / 1e9
            return {"bound": bnd, "achieved": a, "unit": "GB/s", "peak": peaks["hbm_gbs"], "frac": a / peaks["hbm_gbs"],
                    "ms": per_step[c][0], "launches": per_step[c][1]}

        dom = max(alg, key=lambda c: per_step[c][0])
        d = frac_of(dom)
        out["roofline"] = {
            "kernel_class": dom, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
            "frac": d["frac"], "traffic": measured_traffic(name, dom), "peak_source": peaks["source"],
            "peak_kind": d.get("peak_kind", "copy bandwidth"),
            "algorithmic_per_launch": alg[dom][0] / max(per_step[dom][1], 1), "launches_per_step": per_step[dom][1],
            "avg_launch_ms": per_step[dom][0] / max(per_step[dom][1], 1),
            "class_ms_per_step": {c: round(v[0], 4) for c, v in per_step.items()},
            "timing": ("separate pass with CUDA events around every launch; that pass runs the SERIAL schedule (predictor and base "
                       "step after the kernels they follow, every kernel on the whole GPU), so the class times are those of the "
                       "kernels alone and their sum exceeds ms_per_step where the timed schedule overlaps them"),
            "per_class": {c: frac_of(c) for c in alg if per_step[c][0] > 0},
        }
        t12 = (per_step["aux_gemm"][0] + per_step["aux_attn"][0] + per_step["predictor"][0] + per_step.get("kv_pred", (0.0, 0))[0]) * 1e-3
        f12 = work["tensor_flops"] / max(t12, 1e-12) / 1e12
        out["tensor_frac_stage12"] = {"achieved_tflops": f12, "frac": f12 / (tpeak / scale), "peak_kind": which,
                                      "frac_of_burst": f12 / (peaks["bf16_tflops"] / scale),
                                      "frac_of_sustained": f12 / (peaks["bf16_tflops_sustained"] / scale)}
        sess.close()
        del sess, toks
        torch.cuda.empty_cache()
        return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5", choices=WORKLOADS)
    ap.add_argument("--also", default=ALSO_DEFAULT,
                    help="comma-separated configurations measured beside the headline with fewer steps ('none' = only the headline)")
    ap.add_argument("--impl", default="kvp", choices=["kvp", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--train-forward", action="store_true",
                    help="also time the training-time forward (base model over the whole prompt on the predicted cache)")
    ap.add_argument("--prompt-lengths", default="",
                    help="comma-separated prompt lengths replacing the headline workload's batch (same pair, same token recipe): "
                         "cut-down shapes for profiler captures")
    ap.add_argument("--opt-flags", type=int, default=0, help="kvp_options.flags: optional kernel variants (see include/kvp.h)")
    ap.add_argument("--decode-steps", type=int, default=16, help="generation steps timed after the TTFT measurement (0 = none)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "kvp" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start the replicas ourselves, one process per GPU
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        return sys.exit(subprocess.call(replica_command(sys.argv[1:], args.gpus, port)))

    B = Bench(args)
    head_pair = wl.pair("c2" if args.workload == "sweep8" else args.workload)
    if args.workload == "sweep8":
        head_prompts = wl.sweep_prompts(wl.SWEEP8_LENGTHS[-1], seed=0)
    else:
        head_prompts = wl.prompts(args.workload, seed=0)
    if args.prompt_lengths:
        lens = [int(x) for x in args.prompt_lengths.split(",")]
        head_prompts = wl.custom_prompts(head_pair.base.vocab, lens, seed=0, zipf=args.workload != "c5")
    head = B.measure(args.workload, head_pair, head_prompts, args.steps, args.warmup, full=True)

    cpu_baseline = None
    if B.rank == 0 and B.world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands, on the host cores, on a bounded sample of the headline workload
        pr, pair = head_prompts, head_pair
        b = int(np.argmin(pr.lengths))
        n = min(int(pr.lengths[b]), 512 if pair.base.d_model > 2048 else 1024)
        sample = wl.Prompts(pr.seq(b)[:n].copy(), np.array([n], np.int32))
        t = time_oracle(pair, B.weights(pair), sample)
        cpu_baseline = {"value": n / t, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                        "sample": f"first {n} tokens of sequence {b} of workload {args.workload}, whole path, {t:.1f} s"}

    configs = {}
    also = [] if args.also.strip().lower() in ("", "none") else [w.strip() for w in args.also.split(",")]
    for name in also:
        if name == args.workload or name not in WORKLOADS or B.world > 1:
            continue
        few = max(3, min(args.steps, 5))
        if name == "sweep8":
            # Sec. 6, "TTFT vs prompt length at batch 8" (the paper's curve is on a CPU): the 1.1B / 270M-shaped pair
            pair = wl.pair("c2")
            rows = []
            for L in wl.SWEEP8_LENGTHS:
                m = B.measure(f"sweep8_{L}", pair, wl.sweep_prompts(L, seed=0), few, 3, full=False)
                rows.append({"prompt_len": L, "ttft_ms": m["ttft_ms"], "tok_per_s": m["tok_per_s"], "e2e_ms": m["e2e"]["ms_per_step"],
                             "class_ms_per_step": m["roofline"]["class_ms_per_step"], "clocks": m["clocks"],
                             "tensor_frac_stage12": m["tensor_frac_stage12"]})
            configs[name] = {"batch": 8, "pair": "c2", "rows": rows}
            continue
        m = B.measure(name, wl.pair(name), wl.prompts(name, seed=0), few, 3, full=(name in ("c2", "qa")))
        configs[name] = m

    pr, pair = head_prompts, head_pair
    out = {
        "metric": METRIC, "value": head["tok_per_s"], "unit": UNIT, "n_gpus": B.world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ttft_ms"], "ttft_ms": head["ttft_ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": pair.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "batch": pr.batch, "prompt_tokens": head["prompt_tokens"], "lengths": head["lengths"],
                   "l2": "inputs larger than L2 (weights + cache read every step)", "parallelism": "replicas only"},
        "gpu_launches": head["gpu_launches"],
        "e2e": head["e2e"],
        "roofline": head["roofline"],
        "tensor_frac_stage12": head["tensor_frac_stage12"],
        "decode": head.get("decode"),
        "train_forward": head.get("train_forward"),
        "clocks": head["clocks"],
        "configs": configs,
    }
    if cpu_baseline:
        out["cpu_baseline"] = cpu_baseline
    if B.sampler:
        B.sampler.stop()
    if B.rank == 0:
        print(json.dumps(out))
    if B.dist is not None:
        B.dist.destroy_process_group()


if __name__ == "__main__":
    main()
