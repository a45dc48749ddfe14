"""The full-size gradient check (tests/golden/sketch.py) on synthetic arrays: a tensor that is 5 % off in
relative L2 must fail, one that is 0.7 % off (the size of bf16 compute error seen on the small configurations)
must pass, for matrices and vectors, whether the error is spread out or concentrated in a few rows."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden"))
import sketch

TOL = 2e-2


def _ref(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape) * 1e-3


def _summary(name, index, ref):
    return sketch.summarize(name, index, ref)


@pytest.mark.parametrize("shape", [(3000, 512), (4096,), (50, 768)])
@pytest.mark.parametrize("rel,ok", [(0.007, True), (0.05, False), (0.03, False)])
def test_spread_error(shape, rel, ok):
    ref = _ref(shape, 1)
    noise = np.random.default_rng(2).standard_normal(shape)
    noise *= rel * np.linalg.norm(ref) / np.linalg.norm(noise)
    bad = sketch.check_tensor("t", 7, (ref + noise).astype(np.float32), _summary("t", 7, ref), TOL)
    assert (not bad) == ok, bad


def test_error_confined_to_a_few_rows_is_seen_by_the_sketch():
    """5 % of the tensor's norm placed in three rows that are not among the stored ones."""
    ref = _ref((2000, 256), 3)
    summ = _summary("t", 3, ref)
    rows = [r for r in range(2000) if r not in set(summ["rows_idx"].tolist())][:3]
    g = ref.copy()
    noise = np.random.default_rng(4).standard_normal((3, 256))
    g[rows] += noise * 0.05 * np.linalg.norm(ref) / np.linalg.norm(noise)
    bad = sketch.check_tensor("t", 3, g.astype(np.float32), summ, TOL)
    assert any("count sketch" in b[1] for b in bad), bad


def test_scaled_tensor_and_sign_flip_fail():
    ref = _ref((512, 512), 5)
    summ = _summary("t", 1, ref)
    assert sketch.check_tensor("t", 1, (1.05 * ref).astype(np.float32), summ, TOL)
    assert sketch.check_tensor("t", 1, (-ref).astype(np.float32), summ, TOL)
    assert not sketch.check_tensor("t", 1, ref.astype(np.float32), summ, TOL)


def test_hot_rows_are_stored():
    """The two rows of largest reference norm (an embedding's hot rows) are among the stored ones, and an error
    confined to them fails the row check."""
    ref = _ref((1000, 64), 6)
    ref[17] *= 50.0
    ref[400] *= 30.0
    summ = _summary("wte", 0, ref)
    assert {17, 400} <= set(summ["rows_idx"].tolist())
    g = ref.copy()
    g[17] *= 1.04
    bad = sketch.check_tensor("wte", 0, g.astype(np.float32), summ, TOL)
    assert any(b[1].startswith("rel-L2 (rows") for b in bad), bad


def test_sketch_estimate_is_unbiased_on_average():
    """Mean of the squared sketch distance over many tensor indices equals the squared L2 distance."""
    delta = np.random.default_rng(8).standard_normal(20000)
    est = [np.sum(sketch.count_sketch(i, delta) ** 2) for i in range(200)]
    assert abs(np.mean(est) / np.sum(delta ** 2) - 1.0) < 0.05


def test_zero_reference_demands_zero():
    ref = np.zeros((8, 16))
    summ = _summary("t", 2, ref)
    assert not sketch.check_tensor("t", 2, np.zeros((8, 16), np.float32), summ, TOL)
    g = np.zeros((8, 16), np.float32)
    g[3, 3] = 1e-9
    assert sketch.check_tensor("t", 2, g, summ, TOL)
