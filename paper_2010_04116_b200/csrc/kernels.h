// Host-side launchers of the non-GEMM kernels (HBM-bound elementwise / normalisation / reduction
// kernels and the attention kernels).  All pointers are device pointers; all launches are asynchronous
// on `stream` and return cudaGetLastError().
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace il {

// a_0[i,:] = wte[clamp(tok[i]),:] + wpe[i % T,:]  (fp32 residual stream)
cudaError_t embed_fwd(const int* tok, const float* wte, const float* wpe, float* x, int ntok, int T, int d, int V,
                      cudaStream_t s);
// keys [ntok rounded up to 8192] = the batch's (token, position) pairs in sorted order, for embed_bwd.  V < 2^19.
cudaError_t embed_sort(const int* tok, unsigned* keys, int ntok, int V, cudaStream_t s);
// dwte[t,:] = (accumulate ? dwte[t,:] : 0) + sum over the positions i with tok[i] = t of dx[i,:], summed in position
// order (deterministic; rows of tokens that do not occur are left as they are: zero them first unless accumulating);
// dwpe[t,:] = (accumulate ? dwpe[t,:] : 0) + sum_b dx[b*T+t,:].
cudaError_t embed_bwd(const int* tok, const unsigned* keys, const float* dx, float* dwte, float* dwpe, int ntok, int T,
                      int d, int V, int accumulate, cudaStream_t s);

// y(bf16) = gamma * (x - mean) * rstd + beta per row; mean/rstd saved in fp32.
cudaError_t layernorm_fwd(const float* x, const float* gamma, const float* beta, __nv_bfloat16* y, float* mean,
                          float* rstd, int rows, int d, float eps, cudaStream_t s);
// Row part of the LayerNorm backward.  dy is bf16 or fp32 [rows, d]; x/mean/rstd have x_rows rows and are
// indexed by (row % x_rows) so that several stacked gradient streams can share one saved activation.
//   dx_out[row,:] = (resid ? resid[row,:] : 0) + LNbwd(dy[row,:]);   dx_bf16 (optional) = bf16 copy.
cudaError_t layernorm_bwd_rows(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                               const float* gamma, const float* resid, float* dx_out, __nv_bfloat16* dx_bf16,
                               int rows, int x_rows, int d, cudaStream_t s);
// Column reductions over the first `rows` rows: dgamma[c] += sum_r dy[r,c]*xhat[r,c], dbeta[c] += sum_r dy[r,c].
// Outputs are accumulated atomically and must be zeroed by the caller.
cudaError_t layernorm_bwd_params(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                                 float* dgamma, float* dbeta, int rows, int d, cudaStream_t s);
// Both of the above in one pass for bf16 dy and d a multiple of 128 up to 1024 (cudaErrorNotSupported otherwise),
// plus, when colsum != NULL, colsum[c] += sum over the first x_rows rows of dx_out[r,c].
cudaError_t layernorm_bwd_fused(const __nv_bfloat16* dy, const float* x, const float* mean, const float* rstd,
                                const float* gamma, const float* resid, float* dx_out, __nv_bfloat16* dx_bf16, float* dgamma,
                                float* dbeta, float* colsum, int rows, int x_rows, int d, cudaStream_t s);
// out[c] += sum_r y[r,c] for bf16 y [rows, ld] (bias gradients).  out zeroed by the caller.
cudaError_t colsum_bf16(const __nv_bfloat16* y, int ld, float* out, int rows, int cols, cudaStream_t s);
// out[c] += sum_r y[r,c] for fp32 y.
cudaError_t colsum_f32(const float* y, int ld, float* out, int rows, int cols, cudaStream_t s);

// out_f32 = a + (b ? b : 0); out_bf16 (optional) = bf16 copy.   n elements (multiple of 4).
cudaError_t add_convert(const float* a, const float* b, float* out_f32, __nv_bfloat16* out_bf16, size_t n,
                        cudaStream_t s);
// out = (accumulate ? out : 0) + sum_{i<count} w[i] * x[i]   (count <= 4, host arrays of device pointers / weights);
// out_bf16 (optional) = bf16 copy of the result.
cudaError_t lincomb_convert(const float* const* x, const float* w, int count, int accumulate, float* out_f32,
                            __nv_bfloat16* out_bf16, size_t n, cudaStream_t s);
cudaError_t f32_to_bf16(const float* in, __nv_bfloat16* out, size_t n, cudaStream_t s);

// Merge per-tile online-softmax partials: lse[r] = log sum_t exp(pm[r,t]) * ps[r,t]; nll[r] = lse[r] - tgt_logit[r].
cudaError_t lse_finalize(const float* part_max, const float* part_sum, int part_ld, int ntiles, const float* tgt_logit,
                         float* lse, float* nll, int rows, cudaStream_t s);
// out[0] = mean of x[0..n), summed in a fixed order.
cudaError_t mean_f32(const float* x, int n, float* out, cudaStream_t s);
// Launches one thread that waits `limit_ns` on a barrier nobody arrives at and then sets *err = DEV_TIMEOUT_EPILOGUE.
cudaError_t wait_probe(unsigned* err, unsigned long long limit_ns, cudaStream_t s);
// Head backward set-up on E = exp(logits) (bf16 [rows, ld]): E[r, target_r] -= exp(lse_r); rowscale[r] =
// scale * exp(-lse_r) / rows; u_scaled[r, :] = rowscale[r] * u[r, :].  Sets *err when an lse lies outside [-80, 80].
cudaError_t head_backward_prepare(__nv_bfloat16* e, int ld, const float* lse, const int* targets, const __nv_bfloat16* u,
                                  __nv_bfloat16* u_scaled, float* rowscale, int rows, int d, float scale, unsigned* err,
                                  cudaStream_t s);

// AdamW over a flat range: the first n_decay elements get decoupled weight decay.  Writes the bf16 shadow.
// err (may be NULL): when *err != 0 the kernel changes nothing; applied (may be NULL): += 1 when it does update.
// Elements [skip_begin, skip_end) (multiples of 4) are left alone: another launch updates them.
cudaError_t adamw(float* p, float* m, float* v, const float* g, __nv_bfloat16* p_bf16, size_t n, size_t n_decay,
                  float lr, float beta1, float beta2, float eps, float wd, float bc1, float bc2, const unsigned* err,
                  unsigned* applied, size_t skip_begin, size_t skip_end, cudaStream_t s);

// Causal attention on packed qkv [B*T, 3d] (Q | K | V, head h at columns h*dh) on the tcgen05 tensor cores.
// dh in {32, 64, 80, 128, 256}; pointers 16-byte aligned.
//   o [B*T, d] bf16, lse [B, H, T] fp32 (natural log of the softmax denominator, scores scaled by 1/sqrt(dh)).
// err (may be NULL): device word set non-zero if a bounded wait in the kernel expired.
cudaError_t attention_fwd(const __nv_bfloat16* qkv, __nv_bfloat16* o, float* lse, int B, int T, int H, int dh,
                          unsigned* err, cudaStream_t s);
// Backward.  NB batches of gradients share one saved forward of B sequences: gradient batch b uses saved
// sequence (b % B).  dqkv [NB*T, 3d] bf16; delta is scratch [NB, H, T] fp32.
// dq_acc: NULL = two kernels (dK/dV, then dQ; each recomputes the scores; every sum has a fixed order); otherwise
// scratch [NB*T, d] fp32 (16-byte aligned) for the one-sweep form (head dimensions 32 and 64; other sizes fall back
// to two kernels): one recomputation of the scores, dQ summed over key tiles with floating-point atomics.
cudaError_t attention_bwd(const __nv_bfloat16* qkv, const __nv_bfloat16* o, const float* lse, const __nv_bfloat16* dout,
                          __nv_bfloat16* dqkv, float* delta, float* dq_acc, int NB, int B, int T, int H, int dh,
                          unsigned* err, cudaStream_t s);

}  // namespace il
