/*
 * il_ops.h — operator-level entry points of the same library (CUDA, sm_100a).
 *
 * These expose the individual kernels that il.h's training step is built from, so that each can be
 * checked and profiled in isolation.  Every pointer is a DEVICE pointer on the current device, every
 * call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the default stream), nothing
 * is allocated or freed unless stated, and the return value is an il_status (see il.h).  Arguments are
 * validated on the host; a failed validation returns IL_ERR_INVALID_ARG before anything is launched.
 */
#ifndef IL_OPS_H_
#define IL_OPS_H_

#include "il.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Dense contraction C[M,N] = A[M,K] * B[N,K]^T on the tensor cores (bf16 operands, fp32 accumulate),
 * used for every projection of the Transformer blocks (forward, dgrad, wgrad) and for the auxiliary
 * heads' vocabulary projection (Sec. 3: h_ck; Sec. 4.3: GPT-2-like blocks).
 * Operand storage: mn_major = 0: row-major [rows, K] (contraction index contiguous);
 *                  mn_major = 1: row-major [K, rows] (the operand's own index contiguous).
 * Supported combinations (a_mn, b_mn): (0,0) forward, (0,1) dgrad, (1,1) wgrad.
 * Leading dimensions in elements, multiples of 8; pointers 16-byte aligned.
 * Epilogues (the `epilogue` field):
 *   0 C(bf16) = acc + bias                         1 C(bf16) = gelu_tanh'(pre), C2(bf16) = gelu_tanh(pre), pre = acc + bias
 *   2 C(f32) = resid(f32) + acc + bias             3 C(bf16) = acc * aux[row % aux_rows, col]  (aux_rows >= 32;
 *                                                     optionally colsum[col] += sum over rows < aux_rows)
 *   4 C(f32) = acc * rowscale[row] (+ C when accumulate != 0); rowscale [M] fp32, optional
 *   5 per-(row, 128-column block) softmax partials: part_max, part_sum [M, part_ld] at block index
 *     col0/128 + block (col0 % 128 == 0), and tgt_logit[row] = acc[row, targets[row] - col0] when that
 *     column is in range; when C is not NULL, also C(bf16) = acc (the logits, ldc a multiple of 8), or
 *     exp(acc) when store_exp != 0
 *   6 C(bf16) = (exp(acc - lse[row]) - [col + col0 == targets[row]]) * scale
 * (0,1) supports epilogues 0, 3, 4; (1,1) supports 4; (0,0) supports all. */
typedef struct {
  int M, N, K;
  const void* A; int lda; int a_mn_major;
  const void* B; int ldb; int b_mn_major;
  int epilogue;
  void* C; int ldc;
  void* C2;
  const float* bias;
  const float* resid;
  const void* aux; int ld_aux; int aux_rows;
  float* colsum; /* epilogue 3: optional [N] fp32, receives += the column sums of the output over rows < aux_rows */
  int accumulate;
  int split_k;   /* epilogue 4 without accumulate: > 1 splits the contraction over that many work units per
                    tile and adds the partial sums into C atomically (C must be zero on entry); 0/1 = off */
  const int* targets;
  float* part_max; float* part_sum; int part_ld;
  float* tgt_logit;
  const float* lse;
  float scale;
  int col0;
  int tile_blocks; /* output tile: 1 = 256 x 256, 2 = 256 x 512 (fewer operand bytes per product, epilogue less
                      hidden), 0 = chosen from the shape; results do not depend on it */
  const float* rowscale; /* epilogue 4 */
  int store_exp;         /* epilogue 5 */
} il_gemm_desc;

/* err_word: device word (unsigned) the kernel sets non-zero if one of its bounded waits expired. */
il_status il_op_gemm(const il_gemm_desc* desc, unsigned* err_word, void* stream);

/* Causal multi-head self-attention of the Transformer blocks on packed qkv [B*T, 3*H*dh] bf16
 * (Q | K | V; head h at columns h*dh): o [B*T, H*dh] bf16, lse [B, H, T] fp32.  dh in {32, 64, 80, 128, 256};
 * qkv and o 16-byte aligned, lse 4-byte aligned. */
il_status il_op_attention_fwd(const void* qkv, void* o, float* lse, int B, int T, int H, int dh, void* stream);
/* Its backward.  NB gradient batches may share the saved forward of B sequences (gradient batch b uses
 * sequence b % B): dout [NB*T, H*dh] bf16 -> dqkv [NB*T, 3*H*dh] bf16.  delta: scratch [NB*H*T] fp32.
 * qkv, o, dout and dqkv must be 16-byte aligned (IL_ERR_INVALID_ARG otherwise, before anything is launched). */
il_status il_op_attention_bwd(const void* qkv, const void* o, const float* lse, const void* dout, void* dqkv,
                              float* delta, int NB, int B, int T, int H, int dh, void* stream);

/* The same gradients from one sweep over the scores (head dimensions 32 and 64): dK, dV and dQ come from a single
 * recomputation of S and dP (five products instead of the seven of the two-kernel form above).  dq_acc: scratch
 * [NB*T, H*dh] fp32, 16-byte aligned; every key tile adds its share of dQ into it with floating-point atomics
 * (the order of that sum, and so the last bit of dQ, may differ between runs), and a final pass writes it to dqkv
 * as bf16.  err_word: device word set non-zero if a bounded wait expired (may be NULL). */
il_status il_op_attention_bwd_one_sweep(const void* qkv, const void* o, const float* lse, const void* dout, void* dqkv,
                                        float* delta, float* dq_acc, int NB, int B, int T, int H, int dh,
                                        unsigned* err_word, void* stream);

/* The same backward for callers that cannot allocate device memory (no counterpart in the paper: it exists
 * for code embedded where cudaMalloc is not allowed — inside another framework's memory pool, in a
 * real-time loop that bans driver allocations after start-up, or under a fixed device-memory budget).  The
 * delta scratch lives in a fixed 4 MiB array inside the library image (held by every GPU that loads the
 * library until the process exits), so the call obtains no memory: no cudaMalloc/cudaFree, no allocating
 * library routine.  Limit: NB*H*T <= il_op_attention_bwd_noalloc_max_rows() (1,048,576); larger sizes are
 * rejected with IL_ERR_INVALID_ARG before anything is launched.  The first call on each device looks up
 * the array's device address (with that device current) and should therefore be made before any stream
 * capture starts.  All calls on a device share the one array: it keeps the previous call's contents
 * (nothing needs to start at zero — each call rewrites every element it reads), and two calls whose
 * kernels overlap on the GPU (different streams) race on it; serialise them. */
il_status il_op_attention_bwd_noalloc(const void* qkv, const void* o, const float* lse, const void* dout, void* dqkv,
                                      int NB, int B, int T, int H, int dh, void* stream);
size_t il_op_attention_bwd_noalloc_max_rows(void);
/* Whether a bounded wait expired in any il_op_attention_bwd_noalloc call on the current device since the last
 * call of this function (the allocation-free variant reports to an error word that also lives inside the library
 * image).  Waits for `stream`, copies the word to the host and clears it: IL_OK, or IL_ERR_TIMEOUT when the
 * results of those calls are not valid.  Allocates nothing. */
il_status il_op_attention_bwd_noalloc_status(void* stream);

/* Error-path probe: launches one thread that waits limit_us microseconds (1 .. 1,000,000) on a barrier nobody
 * arrives at — the bounded wait every pipelined kernel of this library uses — and then writes a time-out code to
 * *err_word, exactly as a kernel whose producer never delivered would.  The kernel returns normally; the GPU
 * context stays usable.  With err_word = il_error_word(model, k) the model's next il_sync returns IL_ERR_TIMEOUT. */
il_status il_op_wait_probe(unsigned* err_word, unsigned limit_us, void* stream);

/* LayerNorm over the last axis (biased variance, eps inside the square root): y bf16 [rows, d],
 * mean/rstd fp32 [rows].  d % 8 == 0. */
il_status il_op_layernorm_fwd(const float* x, const float* gamma, const float* beta, void* y, float* mean,
                              float* rstd, int rows, int d, float eps, void* stream);
/* LayerNorm backward: dx[row,:] = (resid ? resid[row,:] : 0) + dLN(dy[row,:]) with x/mean/rstd indexed by
 * row % x_rows; dgamma/dbeta (accumulated atomically, zeroed by the caller) over the first x_rows rows.
 * dy is bf16 unless dy_is_f32.  dx_bf16 may be NULL. */
il_status il_op_layernorm_bwd(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                              const float* gamma, const float* resid, float* dx, void* dx_bf16, float* dgamma,
                              float* dbeta, int rows, int x_rows, int d, void* stream);

/* The same in one pass over the rows for bf16 dy and d a multiple of 128 up to 1024 (IL_ERR_INVALID_ARG
 * otherwise), as the training step runs it inside the blocks: dx and dx_bf16 as above, dgamma / dbeta summed into
 * over the first x_rows rows, and, when colsum != NULL, colsum[c] += sum over the first x_rows rows of dx[r, c]
 * (the bias gradient of the linear layer whose output this position of the residual stream is).  dgamma, dbeta
 * and colsum are fp32 [d], zeroed by the caller or holding a sum to add to. */
il_status il_op_layernorm_bwd_fused(const void* dy, const float* x, const float* mean, const float* rstd,
                                    const float* gamma, const float* resid, float* dx, void* dx_bf16, float* dgamma,
                                    float* dbeta, float* colsum, int rows, int x_rows, int d, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IL_OPS_H_ */
