"""Time-per-batch model of synchronous depthwise model parallelism (Sec. 3.1 of the paper).

TEST INFRASTRUCTURE ONLY: the plain statement of the closed form, used to check the library's
il_time_per_batch.  Parameters: A sequential accelerators (modules), M micro-batches per mini-batch,
N the n-wise parameter in [1, A] (N = 1 local learning, N = A end-to-end / GPipe), and the micro-batch
processing cost c(M) = c0 + c1 / M.  The paper fits c0 = 0.025 s, c1 = 1.279 s to its Transformer runs.

Pins (tests/test_timing_model.py): the slot counts of the table under Fig. 3 (2A, 2, 4, 6, 2N for M = 1),
the end-to-end special case 2 (M + A - 1) c(M), the optimal-M rows of App. C's table that follow from the
printed formula (end-to-end, 1-wise, 2-wise; stored in tests/golden/optimal_microbatches.txt), and the
50 % speed-up of 2-wise over GPipe at 15 accelerators.  The 3-, 4- and 5-wise rows of that table do not
follow from the printed formula where A < 2N - 1 and are unpinned.
"""
from __future__ import annotations


def microbatch_cost(M: int, c0: float, c1: float) -> float:
    return c0 + c1 / M


def time_per_batch(A: int, M: int, N: int, c0: float, c1: float) -> float:
    """T(A, M, N) of Sec. 3.1 (N > A is read as N = A: a window cannot exceed the network)."""
    if A < 1 or M < 1 or N < 1:
        raise ValueError("A, M, N must be positive")
    N = min(N, A)
    c = microbatch_cost(M, c0, c1)
    if M == 1:
        return 2 * N * M * c
    if M == 2:
        return (N + 1) * M * c
    if A < 2 * N - 1:
        return (2 + A - N) * M * c + 2 * (2 * N - A - 1) * c
    return (N + 1) * M * c


def optimal_microbatches(A: int, N: int, c0: float, c1: float, max_log2: int = 10) -> int:
    """The power of two M in [1, 2^max_log2] with the smallest time per batch (App. C)."""
    best, best_t = 1, None
    for e in range(max_log2 + 1):
        t = time_per_batch(A, 1 << e, N, c0, c1)
        if best_t is None or t < best_t - 1e-15:
            best, best_t = 1 << e, t
    return best
