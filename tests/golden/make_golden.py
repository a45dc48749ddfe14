#!/usr/bin/env python
"""Writes the full-size expected values used by tests/test_gpu_fullsize.py.

    python tests/golden/make_golden.py cfg2 2        # -> tests/golden/cfg2_n2.json

It runs the fp64 CPU oracle (oracle/il_oracle.py) — and nothing else — on the seeded synthetic workload
of workloads.py at the configuration's full size, and stores a compact summary of the result: the K head
losses and, for every parameter tensor, the L2 norm of its n-wise gradient, its values at seeded sample
positions and its inner products with seeded +-1 vectors.  Takes minutes (GPT-2-small shape) to tens of
minutes (GPT-2-medium shape) on 8 cores and up to ~45 GB of host memory.
"""
from __future__ import annotations

import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402
from oracle import il_oracle as orc  # noqa: E402

N_SAMPLES = 8
N_SKETCH = 2


def summarize(name: str, index: int, g: np.ndarray) -> dict:
    flat = g.reshape(-1)
    idx = wl.sample_indices(name, index, flat.size, N_SAMPLES)
    return {
        "norm": float(np.linalg.norm(flat)),
        "samples": [float(flat[i]) for i in idx],
        "sketch": [float(np.dot(flat, wl.rademacher(index, flat.size, j).astype(np.float64))) for j in range(N_SKETCH)],
    }


def main():
    cfg, n = sys.argv[1], int(sys.argv[2])
    w = wl.CONFIGS[cfg]
    t0 = time.time()
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    losses, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=w.rule, head_layers=w.Lh)
    out = {"config": cfg, "n": n, "rule": w.rule, "head_layers": w.Lh, "weight_seed": wl.WEIGHT_SEED, "token_seed": wl.TOKEN_SEED,
           "oracle_seconds": None, "losses": [float(x) for x in losses], "tensors": {}}
    for i, (name, _, _, _) in enumerate(wl.tensor_specs(w)):
        out["tensors"][name] = summarize(name, i, G[name])
    out["oracle_seconds"] = round(time.time() - t0, 1)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"{cfg}_n{n}.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=0)
    print(path, out["oracle_seconds"], "s", losses)


if __name__ == "__main__":
    main()
