// Host-side interface of the tcgen05 GEMM: C[M,N] = A[M,K] * B[N,K]^T with bf16 operands, fp32
// accumulation in tensor memory, operands staged by TMA, and a fused epilogue.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace il {

enum GemmEpilogue : int {
  EPI_BF16 = 0,        // C(bf16) = acc + bias
  EPI_BF16_GELU = 1,   // pre = acc + bias ; C(bf16) = gelu'(pre) ; C2(bf16) = gelu(pre)
  EPI_F32_RESID = 2,   // C(f32)  = resid(f32) + acc + bias        (C may alias resid)
  EPI_BF16_DGELU = 3,  // C(bf16) = acc * aux[row % aux_rows, col]   (aux = saved gelu'(pre))
  EPI_F32 = 4,         // C(f32)  = acc * rowscale[row] (+ C if accumulate); rowscale optional
  EPI_LSE = 5,         // online-softmax partials per (row, column tile) + logit of the target column; C (bf16, optional) =
                       // acc, or exp(acc) with store_exp
  EPI_DZ = 6,          // C(bf16) = (exp(acc - lse[row]) - [col + col0 == target[row]]) * scale
  EPI_COUNT = 7
};

// Operand storage.  "K-major": the contraction index is contiguous (row-major [rows, K]).
// "MN-major": the row index of the operand is contiguous (memory is row-major [K, rows]).
struct GemmOperand {
  const void* ptr;   // bf16, 16-byte aligned
  int ld;            // leading dimension in elements (multiple of 8)
  int mn_major;      // 0 = K-major, 1 = MN-major
};

struct GemmArgs {
  int M, N, K;
  GemmOperand A, B;
  int epilogue;
  void* C;            // [M, ldc]
  int ldc;
  void* C2;           // EPI_BF16_GELU: activated output gelu(pre), same ld as C (C gets gelu'(pre))
  const float* bias;  // [N] or NULL
  const float* resid; // EPI_F32_RESID: [M, ldc] fp32
  const void* aux;    // EPI_BF16_DGELU: bf16 [aux_rows, ld_aux]
  int ld_aux, aux_rows;
  float* colsum;      // EPI_BF16_DGELU: [N] fp32, += column sums of the (unrounded) output over rows < aux_rows;
                      // NULL = off.  Used for the bias gradient of the layer that produced aux.
  int accumulate;     // EPI_F32
  int split_k;        // EPI_F32 without accumulate: > 1 splits K over that many work units per tile; C must be
                      // zero on entry (partial sums are added atomically).  0/1 = off
  // EPI_LSE / EPI_DZ (vocabulary chunk starting at column col0 of the full vocabulary)
  const int* targets; // [M]
  float* part_max;    // [M, part_ld]  written at column (col0 / 128 + 128-column block)
  float* part_sum;    // [M, part_ld]
  int part_ld;
  float* tgt_logit;   // [M]
  const float* lse;   // [M]
  float scale;        // EPI_DZ: 1 / Ntok
  int col0;
  const float* rowscale;  // EPI_F32: [M] fp32 or NULL
  int store_exp;      // EPI_LSE with C: store exp(acc) instead of acc
  int tile_blocks;    // 256-column blocks per output tile: 1 (256 x 256), 2 (256 x 512), 0 = chosen from the shape
};

// Enqueue one GEMM on `stream`.  `err_word` is a device word set non-zero when a bounded wait in
// the kernel expired.  Returns a cudaError_t (argument errors are reported as cudaErrorInvalidValue).
cudaError_t gemm_launch(const GemmArgs& a, unsigned* err_word, int num_sms, cudaStream_t stream);
// One-time per-process setup (driver entry point for tensor-map encoding, smem opt-in).
cudaError_t gemm_init();

}  // namespace il
