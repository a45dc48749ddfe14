#!/usr/bin/env python
"""Writes the full-size expected values used by tests/test_gpu_fullsize.py.

    python tests/golden/make_golden.py cfg2 2        # -> tests/golden/cfg2_n2.json, cfg2_n2.npz
    python tests/golden/make_golden.py cfg5 2 bounded  # the oracle's bounded-memory form of the same step (cfg5)

It runs the fp64 CPU oracle (oracle/il_oracle.py) — and nothing else — on the seeded synthetic workload
of workloads.py at the configuration's full size, and stores a compact summary of the result.
<cfg>_n<n>.json: the K head losses, the oracle's run time and core count and, per parameter tensor, the L2 norm
of its n-wise gradient and its values at seeded sample positions.  <cfg>_n<n>.npz (float32 / float64 arrays,
see tests/golden/sketch.py): per tensor a 64-bucket count sketch (64 seeded +-1 projections with disjoint
supports, whose squared distance estimates the squared L2 distance), the whole gradient of every rank-1 tensor
and four full rows of every matrix.  Takes minutes (GPT-2-small shape) to tens of minutes (GPT-2-medium
shape) on 8 cores and up to ~45 GB of host memory; the 2.7B-parameter shape takes half an hour on 16 cores and more
than 62 GB in the plain form (the bounded form trades time for memory).
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
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import sketch  # noqa: E402

N_SAMPLES = 8


def summarize(name: str, index: int, g: np.ndarray, arrays: dict) -> dict:
    flat = g.reshape(-1)
    idx = wl.sample_indices(name, index, flat.size, N_SAMPLES)
    for key, val in sketch.summarize(name, index, g).items():
        if key != "norm":
            arrays[f"{index}:{key}"] = val
    return {"norm": float(np.linalg.norm(flat)), "samples": [float(flat[i]) for i in idx]}


def main():
    cfg, n = sys.argv[1], int(sys.argv[2])
    w = wl.CONFIGS[cfg]
    t0 = time.time()
    P = wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    bounded = len(sys.argv) > 3 and sys.argv[3] == "bounded"
    out = {"config": cfg, "n": n, "rule": w.rule, "head_layers": w.Lh, "weight_seed": wl.WEIGHT_SEED, "token_seed": wl.TOKEN_SEED,
           "oracle_seconds": None, "oracle_cores": os.cpu_count(), "oracle_form": "bounded memory" if bounded else "plain",
           "losses": None, "tensors": {}}
    arrays = {}
    index = {name: i for i, (name, _, _, _) in enumerate(wl.tensor_specs(w))}
    if bounded:
        # gradients are summarised and dropped as the oracle declares them final (the 2.7B-shaped step does not fit
        # the host otherwise); the time therefore includes the summaries
        def emit(name, g):
            out["tensors"][name] = summarize(name, index[name], g, arrays)
        losses = orc.nwise_gradients_bounded(P, tok, tgt, w.K, w.Lc, w.H, n, emit, rule=w.rule, head_layers=w.Lh)
        out["oracle_seconds"] = round(time.time() - t0, 1)
        out["tensors"] = {name: out["tensors"][name] for name in index}       # registry order
    else:
        losses, G = orc.nwise_gradients(P, tok, tgt, w.K, w.Lc, w.H, n, rule=w.rule, head_layers=w.Lh)
        out["oracle_seconds"] = round(time.time() - t0, 1)
        for name, i in index.items():
            out["tensors"][name] = summarize(name, i, G[name], arrays)
    out["losses"] = [float(x) for x in losses]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"{cfg}_n{n}.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=0)
    np.savez(path[:-5] + ".npz", **arrays)
    print(path, out["oracle_seconds"], "s", losses)


if __name__ == "__main__":
    main()
