// Attention backward for callers that must not allocate device memory.
//
// il_op_attention_bwd needs a scratch vector (delta_i = sum_c dO_ic O_ic, one fp32 per gradient row and
// head) that its caller has to allocate.  Code that runs where cudaMalloc is off limits — a plug-in called
// from inside another framework's memory pool, a real-time loop that forbids driver allocations after
// start-up, a process whose device memory budget is fixed by its host — cannot do that.  This variant keeps
// the scratch in a fixed array that is part of the library image, so the call itself obtains no memory.
#include <mutex>

#include "../../include/il_ops.h"
#include "kernels.h"

namespace {

constexpr size_t kMaxDelta = size_t(1) << 20;   // NB*H*T fp32 values: 4 MiB held by every GPU that loads the library
static __device__ __align__(256) float g_delta_scratch[kMaxDelta];
static __device__ __align__(256) unsigned g_err_word[64];   // word 0: set by a kernel whose bounded wait expired

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_scratch_ptr[kMaxDevices] = {};   // device address of g_delta_scratch, per device ordinal
unsigned* g_err_ptr[kMaxDevices] = {};    // device address of g_err_word, per device ordinal

// The array's name is only a host-side handle here; kernels need the device address, which differs per
// device and is looked up once with that device current.
cudaError_t scratch_for_current_device(float** out, unsigned** err_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_delta_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    unsigned* w = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&w), g_err_word);
    if (e != cudaSuccess) return e;
    if (!w) return cudaErrorInvalidSymbol;
    g_err_ptr[dev] = w;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  *err_out = g_err_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" il_status il_op_attention_bwd_noalloc(const void* qkv, const void* o, const float* lse, const void* dout,
                                                 void* dqkv, int NB, int B, int T, int H, int dh, void* stream) {
  if (!qkv || !o || !lse || !dout || !dqkv || B < 1 || NB < 1 || T < 1 || H < 1) return IL_ERR_INVALID_ARG;
  if (!(dh == 32 || dh == 64 || dh == 80 || dh == 128)) return IL_ERR_INVALID_ARG;
  // beyond the built-in scratch (each factor is bounded first, so the product cannot wrap)
  if ((size_t)NB > kMaxDelta || (size_t)H > kMaxDelta || (size_t)T > kMaxDelta) return IL_ERR_INVALID_ARG;
  if ((size_t)NB * (size_t)H > kMaxDelta || (size_t)NB * (size_t)H * (size_t)T > kMaxDelta) return IL_ERR_INVALID_ARG;
  float* delta = nullptr;
  unsigned* err = nullptr;
  if (scratch_for_current_device(&delta, &err) != cudaSuccess) return IL_ERR_CUDA;
  // Every element of delta that the kernels read is written by the same call first, so nothing has to be cleared.
  cudaError_t e = il::attention_bwd(reinterpret_cast<const __nv_bfloat16*>(qkv), reinterpret_cast<const __nv_bfloat16*>(o),
                                    lse, reinterpret_cast<const __nv_bfloat16*>(dout),
                                    reinterpret_cast<__nv_bfloat16*>(dqkv), delta, nullptr, NB, B, T, H, dh, err,
                                    reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaSuccess) return IL_OK;
  return e == cudaErrorInvalidValue ? IL_ERR_INVALID_ARG : IL_ERR_CUDA;
}

extern "C" size_t il_op_attention_bwd_noalloc_max_rows(void) { return kMaxDelta; }

extern "C" il_status il_op_attention_bwd_noalloc_status(void* stream) {
  float* delta = nullptr;
  unsigned* err = nullptr;
  if (scratch_for_current_device(&delta, &err) != cudaSuccess) return IL_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  unsigned w = 0;
  if (cudaMemcpyAsync(&w, err, sizeof w, cudaMemcpyDeviceToHost, st) != cudaSuccess) return IL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return IL_ERR_CUDA;
  if (w == 0) return IL_OK;
  if (cudaMemsetAsync(err, 0, sizeof w, st) != cudaSuccess) return IL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return IL_ERR_CUDA;
  return IL_ERR_TIMEOUT;
}
