// Time-per-batch model of synchronous depthwise model parallelism (Sec. 3.1 of the paper): host-only closed
// form, no device work.  T(A, M, N) with micro-batch cost c(M) = c0 + c1 / M, in the same unit as c0 and c1.
#include "../../include/il.h"

namespace {

double time_per_batch(int A, int M, int N, double c0, double c1) {
  if (N > A) N = A;                       // a window cannot be longer than the network
  const double c = c0 + c1 / (double)M;   // cost of one time slot (one micro-batch through one module)
  if (M == 1) return 2.0 * N * c;                                  // no micro-batching: 2N slots
  if (M == 2 || A >= 2 * N - 1) return (N + 1.0) * M * c;          // windows do not reach across the pipeline fill
  return (2.0 + A - N) * M * c + 2.0 * (2 * N - A - 1) * c;        // M > 2 and A < 2N - 1
}

}  // namespace

extern "C" il_status il_time_per_batch(int A, int M, int N, double c0, double c1, double* out) {
  if (A < 1 || M < 1 || N < 1 || !out || !(c0 >= 0.0) || !(c1 >= 0.0)) return IL_ERR_INVALID_ARG;
  *out = time_per_batch(A, M, N, c0, c1);
  return IL_OK;
}

extern "C" il_status il_optimal_microbatches(int A, int N, double c0, double c1, int max_log2, int* M_out) {
  if (A < 1 || N < 1 || max_log2 < 0 || max_log2 > 30 || !M_out || !(c0 >= 0.0) || !(c1 >= 0.0)) return IL_ERR_INVALID_ARG;
  int best = 1;
  double best_t = time_per_batch(A, 1, N, c0, c1);
  for (int e = 1; e <= max_log2; ++e) {
    const double t = time_per_batch(A, 1 << e, N, c0, c1);
    if (t < best_t - 1e-15) { best_t = t; best = 1 << e; }
  }
  *M_out = best;
  return IL_OK;
}
