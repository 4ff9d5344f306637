"""Test infrastructure, CPU only: how far do the first-step logits move when nothing but the storage
format of the predicted cache (bf16) is applied to the oracle's exact result?

    python oracle/cache_rounding_floor.py c2 0      # workload, sequence

The predicted cache K_hat, V_hat (Sec. 4.1: the keys and values the base model attends to) is
computed in fp64, rounded once to bf16, and the base model's first step is run on both versions.
The relative Frobenius distance of the two logit vectors is the part of the GPU-vs-oracle logits
error that no kernel can remove while the cache is stored in bf16.
"""
import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import workloads as wl  # noqa: E402
from oracle import kvp_oracle as orc  # noqa: E402


def floor(name: str, b: int) -> float:
    pair = wl.pair(name)
    W = wl.make_weights(pair, seed=0)
    toks = wl.prompts(name, seed=0).seq(b)
    kv = orc.predict_kv(pair, W, orc.aux_prefill(pair, W, toks))
    ref = orc.base_first_step(pair, W, int(toks[-1]), kv)
    rounded = [(wl.round_to_bf16(k.astype(np.float32)).astype(np.float64),
                wl.round_to_bf16(v.astype(np.float32)).astype(np.float64)) for k, v in kv]
    got = orc.base_first_step(pair, W, int(toks[-1]), rounded)
    return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))


if __name__ == "__main__":
    name, b = sys.argv[1], int(sys.argv[2])
    t = time.time()
    print(f"{name} sequence {b}: logits move by {floor(name, b):.3e} from bf16 rounding of the exact cache ({time.time() - t:.0f} s)")
