"""The paper's time-per-batch model (Sec. 3.1, App. C): the oracle against what the paper prints, and the
library's host function against the oracle.  No GPU needed."""
import os

import pytest

from oracle import timing_model as tm
from paper_2010_04116_b200 import binding as il

C0, C1 = 0.025, 1.279            # the paper's fit to its Transformer runs (Sec. 3.1)
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "optimal_microbatches.txt")


def test_unit_slot_table_under_fig3():
    """Time per batch in slots without micro-batching: end-to-end 2A, 1-wise 2, 2-wise 4, 3-wise 6, n-wise 2N."""
    for A in (3, 4, 6, 10):
        assert tm.time_per_batch(A, 1, A, 1.0, 0.0) == 2 * A
        for N in range(1, A + 1):
            assert tm.time_per_batch(A, 1, N, 1.0, 0.0) == 2 * N


def test_end_to_end_special_case():
    """N = A degenerates to 2 (M + A - 1) c(M) for every M >= 2 (GPipe)."""
    for A in (2, 3, 5, 8, 16):
        for M in (2, 3, 4, 8, 32):
            ref = 2 * (M + A - 1) * tm.microbatch_cost(M, C0, C1)
            assert abs(tm.time_per_batch(A, M, A, C0, C1) - ref) < 1e-12


def test_independent_of_depth_for_short_windows():
    """For N < 1 + A/2 the time per batch does not depend on the number of modules (Sec. 3.1)."""
    for N in (1, 2, 3):
        for M in (1, 2, 4, 8):
            vals = {round(tm.time_per_batch(A, M, N, C0, C1), 12) for A in range(2 * N - 1, 40)}
            assert len(vals) == 1


def test_optimal_microbatch_table_of_appendix_c():
    rows = [tuple(map(int, ln.split())) for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 25
    for n, A, M in rows:
        assert tm.optimal_microbatches(A, A if n == 0 else n, C0, C1) == M, (n, A, M)


def test_two_wise_speedup_over_gpipe_reaches_half_at_fifteen_accelerators():
    def speedup(A):
        gpipe = min(tm.time_per_batch(A, 1 << e, A, C0, C1) for e in range(11))
        return gpipe / tm.time_per_batch(A, 2, 2, C0, C1)
    assert speedup(14) < 1.49 < speedup(15) < 1.51        # "a 50% speed-up ... at 15 or more accelerators"
    assert all(speedup(A + 1) > speedup(A) for A in range(4, 40))


def test_library_matches_oracle_everywhere():
    for A in range(1, 13):
        for N in range(1, 15):
            for M in (1, 2, 3, 4, 7, 8, 16, 64):
                ref = tm.time_per_batch(A, M, N, C0, C1)
                assert abs(il.time_per_batch(A, M, N, C0, C1) - ref) <= 1e-12 * ref
            assert il.optimal_microbatches(A, N, C0, C1) == tm.optimal_microbatches(A, N, C0, C1)
    with pytest.raises(il.ILError):
        il.time_per_batch(0, 1, 1, C0, C1)
    with pytest.raises(il.ILError):
        il.optimal_microbatches(4, 2, -1.0, C1)


def test_lr_schedule_matches_the_paper_formula():
    """App. B.3: lr = 1024^-0.5 min(step^-0.5, step warmup^-1.5) with 4000 warm-up steps: linear warm-up to
    the peak (d warmup)^-0.5 at step = warmup, inverse square root decay afterwards."""
    import math

    from oracle import il_oracle as orc
    assert il.lr_schedule(4000, 1024, 4000) == pytest.approx((1024 * 4000) ** -0.5, rel=1e-14)
    assert il.lr_schedule(1, 1024, 4000) == pytest.approx(1024 ** -0.5 * 4000 ** -1.5, rel=1e-14)
    assert il.lr_schedule(16000, 1024, 4000) == pytest.approx(0.5 * il.lr_schedule(4000, 1024, 4000), rel=1e-14)
    for step in (1, 7, 3999, 4000, 4001, 123456):
        assert il.lr_schedule(step, 1024, 4000) == pytest.approx(orc.inverse_sqrt_lr(step, 1024, 4000), rel=1e-14)
        assert il.lr_schedule(step, 768, 100) == pytest.approx(
            768 ** -0.5 * min(1 / math.sqrt(step), step / 100 ** 1.5), rel=1e-14)
    with pytest.raises(il.ILError):
        il.lr_schedule(0, 1024, 4000)
