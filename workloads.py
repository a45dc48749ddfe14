"""Workload shapes and seeded synthetic inputs for the n-wise training step.

This module holds no arithmetic of the method: only the model shapes, the list
of parameter tensors (names and shapes are the shared *specification* of the
parameter registry) and counter-based random draws for weights and tokens.
Both the fp64 CPU oracle's tests and the CUDA path's tests draw their inputs
here so that the two sides see identical values.

Synthetic inputs stand in for the One Billion Word benchmark the paper trains
its Transformer on (Sec. 4.3): token ids follow a Zipf(s=1.1) law over the
vocabulary (uniform for the tiny configuration), and every weight tensor is
N(0, 0.02^2); LayerNorm gains are 1 + N(0, 0.02^2) so that every path of the
network carries signal in a parity run.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np

WEIGHT_SEED = 20100411
TOKEN_SEED = WEIGHT_SEED + 1


@dataclass(frozen=True)
class Workload:
    """Shape of one training step.  K components of Lc pre-LN blocks each."""

    name: str
    K: int            # components ("modules" in the paper, Sec. 3)
    Lc: int           # Transformer blocks per component
    d: int            # d_model
    H: int            # attention heads
    F: int            # d_ff
    V: int            # vocabulary
    T: int            # sequence length
    B: int            # sequences per step
    n: int            # n-wise parameter (1 = local learning, K = full backprop)
    zipf: bool = True  # token law: Zipf(1.1) if True, uniform otherwise
    adamw: bool = False
    Lh: int = 0       # Transformer blocks inside every auxiliary head (App. B.3: 2); 0 = LayerNorm + linear head
    M: int = 1        # micro-batches a mini-batch of B sequences is processed in (Sec. 3.1)
    rule: str = "sum"  # head weighting: "sum", "far" (Sec. 3 main text) or "mean" (App. B.3)
    weight_decay: float = 0.01   # decoupled decay of the AdamW step; 0 gives the paper's Adam (App. B.3)

    @property
    def ntok(self) -> int:
        return self.B * self.T

    @property
    def dh(self) -> int:
        return self.d // self.H

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations (index 0 = the tiny case the oracle finishes in seconds).
CONFIGS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", K=2, Lc=2, d=128, H=4, F=512, V=512, T=64, B=4, n=2, zipf=False),
    "cfg2": Workload("cfg2", K=4, Lc=3, d=768, H=12, F=3072, V=50257, T=1024, B=8, n=2),
    "cfg3": Workload("cfg3", K=4, Lc=3, d=768, H=12, F=3072, V=50257, T=1024, B=8, n=1),
    "cfg4": Workload("cfg4", K=8, Lc=3, d=1024, H=16, F=4096, V=50257, T=1024, B=8, n=2, adamw=True),
    "cfg5": Workload("cfg5", K=8, Lc=4, d=2560, H=32, F=10240, V=50257, T=2048, B=4, n=2, adamw=True),
    # cfg4's widths, sequence length, batch and vocabulary with only two one-layer components: every kernel
    # runs at cfg4's shapes while the model holds ~3 GB, small enough for profiler captures.
    "cfg4-2x1": Workload("cfg4-2x1", K=2, Lc=1, d=1024, H=16, F=4096, V=50257, T=1024, B=8, n=2, adamw=True),
    # The shape of the paper's own Transformer runs (App. B.3): modules of 6 blocks, d 1024, 4 attention heads,
    # sequence length 128, an auxiliary network of 2 blocks + embedding matrix per module, the mean-of-two-heads
    # rule, Adam; A = 4 modules, a mini-batch of 1024 sequences in 4 micro-batches (Sec. 3.1).  The vocabulary
    # size is not printed in the paper; the other configurations' 50257 is used.
    "cfgP": Workload("cfgP", K=4, Lc=6, d=1024, H=4, F=4096, V=50257, T=128, B=1024, n=2, adamw=True, Lh=2, M=4,
                     rule="mean", weight_decay=0.0),
    # cfgP's model at full size on a mini-batch of 8 sequences (4 micro-batches of 2): what the fp64 oracle can
    # run at full widths, depth and vocabulary in minutes, for the stored expected values.
    "cfgP-b8": Workload("cfgP-b8", K=4, Lc=6, d=1024, H=4, F=4096, V=50257, T=128, B=8, n=2, adamw=True, Lh=2, M=4,
                        rule="mean", weight_decay=0.0),
}


def tensor_specs(w: Workload, max_seq: int | None = None) -> List[Tuple[str, int, bool, Tuple[int, ...]]]:
    """Ordered parameter registry: (name, component, is_head, shape).

    component is 0-based; the embeddings belong to component 0 (the paper's
    first module holds the input projection, App. B.3).  Matrices are stored
    [out_features, in_features].  wqkv rows are [Q; K; V], each split into H
    consecutive blocks of dh rows.
    """
    T = w.T if max_seq is None else max_seq
    specs: List[Tuple[str, int, bool, Tuple[int, ...]]] = [
        ("wte", 0, False, (w.V, w.d)),
        ("wpe", 0, False, (T, w.d)),
    ]
    for k in range(w.K):
        for l in range(w.Lc):
            p = f"c{k}.l{l}."
            specs += [
                (p + "ln1.g", k, False, (w.d,)),
                (p + "ln1.b", k, False, (w.d,)),
                (p + "attn.wqkv", k, False, (3 * w.d, w.d)),
                (p + "attn.bqkv", k, False, (3 * w.d,)),
                (p + "attn.wo", k, False, (w.d, w.d)),
                (p + "attn.bo", k, False, (w.d,)),
                (p + "ln2.g", k, False, (w.d,)),
                (p + "ln2.b", k, False, (w.d,)),
                (p + "mlp.w1", k, False, (w.F, w.d)),
                (p + "mlp.b1", k, False, (w.F,)),
                (p + "mlp.w2", k, False, (w.d, w.F)),
                (p + "mlp.b2", k, False, (w.d,)),
            ]
    for k in range(w.K):
        for l in range(w.Lh):
            p = f"head{k}.l{l}."
            specs += [
                (p + "ln1.g", k, True, (w.d,)),
                (p + "ln1.b", k, True, (w.d,)),
                (p + "attn.wqkv", k, True, (3 * w.d, w.d)),
                (p + "attn.bqkv", k, True, (3 * w.d,)),
                (p + "attn.wo", k, True, (w.d, w.d)),
                (p + "attn.bo", k, True, (w.d,)),
                (p + "ln2.g", k, True, (w.d,)),
                (p + "ln2.b", k, True, (w.d,)),
                (p + "mlp.w1", k, True, (w.F, w.d)),
                (p + "mlp.b1", k, True, (w.F,)),
                (p + "mlp.w2", k, True, (w.d, w.F)),
                (p + "mlp.b2", k, True, (w.d,)),
            ]
        specs += [
            (f"head{k}.ln.g", k, True, (w.d,)),
            (f"head{k}.ln.b", k, True, (w.d,)),
            (f"head{k}.w", k, True, (w.V, w.d)),
        ]
    return specs


def num_params(w: Workload) -> int:
    return int(sum(int(np.prod(s)) for _, _, _, s in tensor_specs(w)))


def _rng(seed: int, stream: int) -> np.random.Generator:
    # Philox is counter-based: (seed, stream) selects an independent sequence.
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream]))


def draw_tensor(name: str, index: int, shape: Tuple[int, ...], seed: int = WEIGHT_SEED,
                std: float = 0.02) -> np.ndarray:
    """fp32 N(0, std^2) values (LayerNorm gains: 1 + N(0, std^2)) for tensor #index."""
    g = _rng(seed, index)
    x = g.standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    if name.endswith(".g"):
        x = x + np.float32(1.0)
    return x.astype(np.float32)


def draw_params(w: Workload, seed: int = WEIGHT_SEED, max_seq: int | None = None) -> Dict[str, np.ndarray]:
    return {name: draw_tensor(name, i, shape, seed)
            for i, (name, _, _, shape) in enumerate(tensor_specs(w, max_seq))}


def draw_tokens(w: Workload, seed: int = TOKEN_SEED, step: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """B x (T+1) token ids -> (inputs [B,T], next-token targets [B,T]), int32.

    Zipf: p(r) proportional to r^-1.1 for ranks r = 1..V, drawn by inverse CDF on an
    fp64 cumulative table; token id = r - 1.
    """
    g = _rng(seed, step)
    u = g.random(size=(w.B, w.T + 1))
    if w.zipf:
        p = np.arange(1, w.V + 1, dtype=np.float64) ** -1.1
        cdf = np.cumsum(p)
        cdf /= cdf[-1]
        ids = np.searchsorted(cdf, u, side="right")
        ids = np.minimum(ids, w.V - 1)
    else:
        ids = np.minimum((u * w.V).astype(np.int64), w.V - 1)
    ids = ids.astype(np.int32)
    return np.ascontiguousarray(ids[:, :-1]), np.ascontiguousarray(ids[:, 1:])


def sample_indices(name: str, index: int, size: int, count: int, seed: int = WEIGHT_SEED) -> np.ndarray:
    """Seeded flat indices into a tensor of `size` elements (for sampled full-size checks)."""
    g = _rng(seed ^ 0x5EED5A3D, index)
    return g.integers(0, size, size=min(count, size), dtype=np.int64)


def rademacher(index: int, size: int, which: int, seed: int = WEIGHT_SEED) -> np.ndarray:
    """Seeded +-1 vector (int8) used to sketch a large gradient tensor into one number."""
    g = _rng(seed ^ 0x0BADC0DE, index * 16 + which)
    return (g.integers(0, 2, size=size, dtype=np.int8) * 2 - 1).astype(np.int8)
