"""Compact summaries of large gradient tensors, and the check of a gradient against such a summary.

Test infrastructure shared by tests/golden/make_golden.py (which summarises the fp64 oracle's gradients)
and tests/test_gpu_fullsize.py (which summarises the CUDA path's gradients the same way and compares).
Nothing here belongs to the method: it is seeded random draws and sums.

Summary of one tensor g (flattened, size n):
  * norm            ||g||_2
  * sketch[64]      a count sketch: every element i draws a bucket b_i in [0, 64) and a sign s_i = +-1 from a
                    counter-based generator keyed by the tensor's index; sketch[j] = sum_{i: b_i = j} s_i g_i.
                    These are 64 seeded +-1 projections with disjoint supports, so for any two tensors
                        E sum_j (sketch_j(g) - sketch_j(r))^2 = ||g - r||^2
                    (cross terms vanish in expectation): the squared sketch distance is an unbiased estimate of
                    the squared L2 distance, with a relative standard deviation of about sqrt(2/64) = 18 % when
                    the difference is spread over many elements, i.e. about 9 % on the L2 distance itself.
  * vec             the whole tensor, for rank-1 tensors
  * rows_idx, rows  four full rows of a matrix: the two rows of largest reference norm (the hot rows of an
                    embedding matrix under Zipf-distributed tokens) and two seeded ones
"""
from __future__ import annotations

import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

BUCKETS = 64
N_ROWS = 4
_CHUNK = 1 << 24


def _codes(index: int, size: int) -> np.ndarray:
    """One int8 in [0, 128) per element: bit 0 = sign, bits 1..6 = bucket."""
    g = np.random.Generator(np.random.Philox(key=[(wl.WEIGHT_SEED ^ 0xC0DE5EED) & (2**64 - 1), index]))
    return g.integers(0, 2 * BUCKETS, size=size, dtype=np.int8)


def count_sketch(index: int, flat: np.ndarray) -> np.ndarray:
    """The 64 bucket sums of `flat` (any float dtype; summed in float64)."""
    codes = _codes(index, flat.size)
    out = np.zeros(BUCKETS, dtype=np.float64)
    for a in range(0, flat.size, _CHUNK):
        c = codes[a:a + _CHUNK].astype(np.int64)
        v = flat[a:a + _CHUNK].astype(np.float64)
        v = np.where(c & 1, -v, v)
        out += np.bincount(c >> 1, weights=v, minlength=BUCKETS)
    return out


def pick_rows(name: str, index: int, ref: np.ndarray) -> np.ndarray:
    """Row indices stored for a matrix: the two of largest norm in `ref` and two seeded ones (distinct)."""
    nrows = ref.shape[0]
    if nrows <= N_ROWS:
        return np.arange(nrows, dtype=np.int64)
    norms = np.einsum("ij,ij->i", ref, ref)
    top = np.argsort(-norms, kind="stable")[:2]
    chosen = [int(r) for r in top]
    for r in wl.sample_indices(name + ":rows", index, nrows, 64):
        if int(r) not in chosen:
            chosen.append(int(r))
        if len(chosen) == N_ROWS:
            break
    return np.array(chosen, dtype=np.int64)


def summarize(name: str, index: int, g: np.ndarray) -> dict:
    """Summary of the reference gradient g (float64) of tensor #index."""
    flat = g.reshape(-1)
    out = {"norm": np.float64(np.linalg.norm(flat)), "sketch": count_sketch(index, flat)}
    if g.ndim == 1:
        out["vec"] = flat.astype(np.float32)
    else:
        idx = pick_rows(name, index, g)
        out["rows_idx"] = idx
        out["rows"] = g[idx].astype(np.float32)
    return out


def check_tensor(name: str, index: int, g: np.ndarray, ref: dict, tol: float) -> list:
    """Compare gradient g with the stored summary `ref`; returns a list of findings (empty = within tol).

      * estimated relative L2 error (count sketch) <= tol;
      * | ||g|| - ||ref|| | <= tol ||ref||;
      * rank-1: exact relative L2 error over the whole vector <= tol;
      * matrices: exact L2 error over the four stored rows <= tol x max(norm of those rows, the share of the
        tensor's norm that four average rows carry) — the tolerance is a per-tensor one, so a row much smaller
        than average is held to the tensor's scale, not its own.
    """
    bad = []
    g64 = g.astype(np.float64)
    flat = g64.reshape(-1)
    norm = float(ref["norm"])
    if norm == 0.0:
        if flat.any():
            bad.append((name, "nonzero where the reference is zero", float(np.linalg.norm(flat)), 0.0))
        return bad
    gn = float(np.linalg.norm(flat))
    if abs(gn - norm) > tol * norm:
        bad.append((name, "norm", gn, norm))
    sk = count_sketch(index, flat)
    est = float(np.sqrt(np.sum((sk - np.asarray(ref["sketch"], dtype=np.float64)) ** 2))) / norm
    if not est <= tol:
        bad.append((name, "estimated rel-L2 (count sketch)", est, tol))
    if g.ndim == 1:
        r = np.asarray(ref["vec"], dtype=np.float64)
        err = float(np.linalg.norm(flat - r)) / norm
        if not err <= tol:
            bad.append((name, "rel-L2 (whole vector)", err, tol))
    else:
        idx = np.asarray(ref["rows_idx"], dtype=np.int64)
        r = np.asarray(ref["rows"], dtype=np.float64)
        rows_norm = float(np.linalg.norm(r))
        share = norm * np.sqrt(r.size / flat.size)
        err = float(np.linalg.norm(g64[idx] - r)) / max(rows_norm, share)
        if not err <= tol:
            bad.append((name, f"rel-L2 (rows {idx.tolist()})", err, tol))
    return bad
