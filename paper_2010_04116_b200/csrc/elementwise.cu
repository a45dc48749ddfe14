// HBM-bound kernels of the training step: embedding, LayerNorm forward/backward, column reductions for
// bias and LayerNorm parameter gradients, gradient-stream sums, softmax-partial merge, AdamW.
// All of them use 16-byte (or 8-byte for bf16x4) coalesced accesses and warp-shuffle reductions.
#include "common.cuh"
#include "kernels.h"

namespace il {

static inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

// ---------------------------------------------------------------------------------------------
// Embedding
// ---------------------------------------------------------------------------------------------
__global__ void embed_fwd_kernel(const int* __restrict__ tok, const float* __restrict__ wte,
                                 const float* __restrict__ wpe, float* __restrict__ x, int ntok, int T, int d, int V) {
  grid_dep_sync();
  const int d4 = d >> 2;
  const size_t total = (size_t)ntok * d4;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / d4);
    const int c = (int)(i % d4);
    int t = tok[row];
    t = t < 0 ? 0 : (t >= V ? V - 1 : t);
    const float4 a = __ldg(reinterpret_cast<const float4*>(wte + (size_t)t * d) + c);
    const float4 b = __ldg(reinterpret_cast<const float4*>(wpe + (size_t)(row % T) * d) + c);
    reinterpret_cast<float4*>(x + (size_t)row * d)[c] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
  }
}

cudaError_t embed_fwd(const int* tok, const float* wte, const float* wpe, float* x, int ntok, int T, int d, int V,
                      cudaStream_t s) {
  const size_t total = (size_t)ntok * (d / 4);
  int blocks = ceil_div(total, 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  launch_dep(embed_fwd_kernel, dim3(blocks), dim3(256), 0, s, tok, wte, wpe, x, ntok, T, d, V);
  return cudaGetLastError();
}

// Deterministic scatter-add of the embedding gradient.  Floating-point atomics would add the rows of a hot token
// (under a Zipf law the most frequent id holds about a tenth of all positions) in whatever order the hardware
// serves them; instead the positions are sorted by token id once per batch, and every token's rows are then
// summed in position order.
//
// embed_sort: chunks of SORT_CHUNK positions; a block builds the keys (token << 13 | position in chunk) of its
// chunk in shared memory and sorts them with a bitonic network (keys are distinct, so the order is total).
constexpr int SORT_CHUNK = 8192;
constexpr int SORT_POS_BITS = 13;

__global__ void __launch_bounds__(1024) embed_sort_kernel(const int* __restrict__ tok, unsigned* __restrict__ keys, int ntok,
                                                          int V) {
  grid_dep_sync();
  __shared__ unsigned sk[SORT_CHUNK];
  const int base = blockIdx.x * SORT_CHUNK;
  for (int i = threadIdx.x; i < SORT_CHUNK; i += 1024) {
    unsigned key = 0xFFFFFFFFu;                       // padding sorts to the end
    if (base + i < ntok) {
      int t = tok[base + i];
      t = t < 0 ? 0 : (t >= V ? V - 1 : t);
      key = ((unsigned)t << SORT_POS_BITS) | (unsigned)i;
    }
    sk[i] = key;
  }
  __syncthreads();
  for (int size = 2; size <= SORT_CHUNK; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < SORT_CHUNK / 2; t += 1024) {
        const int lo = 2 * t - (t & (stride - 1));    // index of the lower element of pair t at this stride
        const int hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned a = sk[lo], b = sk[hi];
        if ((a > b) == up) { sk[lo] = b; sk[hi] = a; }
      }
      __syncthreads();
    }
  for (int i = threadIdx.x; i < SORT_CHUNK; i += 1024) keys[base + i] = sk[i];
}

cudaError_t embed_sort(const int* tok, unsigned* keys, int ntok, int V, cudaStream_t s) {
  if (V > (1 << (32 - SORT_POS_BITS)) - 1) return cudaErrorInvalidValue;
  launch_dep(embed_sort_kernel, dim3(ceil_div(ntok, SORT_CHUNK)), dim3(1024), 0, s, tok, keys, ntok, V);
  return cudaGetLastError();
}

// One block per sorted key of a chunk; the block whose key starts a token's run sums the run.  1024 threads =
// 4 row groups x 256 column lanes (float4): group g adds rows g, g+4, ... of the run in order and the four
// partial sums are combined in a fixed order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(1024) embed_bwd_wte_kernel(const unsigned* __restrict__ keys, const float* __restrict__ dx,
                                                             float* __restrict__ dwte, int chunk_base, int ntok, int d,
                                                             int accumulate) {
  grid_dep_sync();
  __shared__ float4 part[3][256];
  const int i = blockIdx.x;                            // index within the chunk
  const unsigned key = keys[chunk_base + i];
  if (key == 0xFFFFFFFFu) return;
  const unsigned tokid = key >> SORT_POS_BITS;
  if (i > 0 && (keys[chunk_base + i - 1] >> SORT_POS_BITS) == tokid) return;     // not the start of a run
  int len = 1;
  const int limit = min(SORT_CHUNK, ntok - chunk_base);
  while (i + len < limit && (keys[chunk_base + i + len] >> SORT_POS_BITS) == tokid) ++len;
  const int g = threadIdx.x >> 8, lane = threadIdx.x & 255;
  const int d4 = d >> 2;
  constexpr unsigned POS_MASK = (1u << SORT_POS_BITS) - 1u;
  for (int c0 = 0; c0 < d4; c0 += 256) {
    const int c = c0 + lane;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < d4) {
      int r = g;
      for (; r + 12 < len; r += 16) {                  // four rows of this group in flight
        float4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int pos = chunk_base + (int)(keys[chunk_base + i + r + 4 * q] & POS_MASK);
          v[q] = reinterpret_cast<const float4*>(dx + (size_t)pos * d)[c];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) { acc.x += v[q].x; acc.y += v[q].y; acc.z += v[q].z; acc.w += v[q].w; }
      }
      for (; r < len; r += 4) {
        const int pos = chunk_base + (int)(keys[chunk_base + i + r] & POS_MASK);
        const float4 v = reinterpret_cast<const float4*>(dx + (size_t)pos * d)[c];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
    }
    if (g > 0) part[g - 1][lane] = acc;
    __syncthreads();
    if (g == 0 && c < d4) {
      const float4 p1 = part[0][lane], p2 = part[1][lane], p3 = part[2][lane];
      acc.x = (acc.x + p1.x) + (p2.x + p3.x); acc.y = (acc.y + p1.y) + (p2.y + p3.y);
      acc.z = (acc.z + p1.z) + (p2.z + p3.z); acc.w = (acc.w + p1.w) + (p2.w + p3.w);
      float4* out = reinterpret_cast<float4*>(dwte + (size_t)tokid * d) + c;
      if (accumulate) {
        const float4 o = *out;
        acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
      }
      *out = acc;
    }
    __syncthreads();
  }
}
__global__ void embed_bwd_wpe_kernel(const float* __restrict__ dx, float* __restrict__ dwpe, int B, int T, int d,
                                     int accumulate) {
  grid_dep_sync();
  const int d4 = d >> 2;
  const size_t total = (size_t)T * d4;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float4 acc = accumulate ? reinterpret_cast<const float4*>(dwpe)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int b = 0; b < B; ++b) {
      const float4 v = reinterpret_cast<const float4*>(dx + (size_t)b * T * d)[i];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    reinterpret_cast<float4*>(dwpe)[i] = acc;
  }
}

cudaError_t embed_bwd(const int* tok, const unsigned* keys, const float* dx, float* dwte, float* dwpe, int ntok, int T,
                      int d, int V, int accumulate, cudaStream_t s) {
  (void)tok; (void)V;
  // chunk after chunk on the one stream: a token that occurs in several chunks is added to in chunk order
  for (int base = 0; base < ntok; base += SORT_CHUNK)
    launch_dep(embed_bwd_wte_kernel, dim3(min(SORT_CHUNK, ntok - base)), dim3(1024), 0, s, keys, dx, dwte, base, ntok, d,
                                                                        (accumulate || base > 0) ? 1 : 0);
  int blocks2 = ceil_div((size_t)T * (d / 4), 256);
  launch_dep(embed_bwd_wpe_kernel, dim3(blocks2), dim3(256), 0, s, dx, dwpe, ntok / T, T, d, accumulate);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// LayerNorm forward: one warp per row
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) layernorm_fwd_kernel(const float* __restrict__ x, const float* __restrict__ gamma,
                                                            const float* __restrict__ beta, bf16* __restrict__ y,
                                                            float* __restrict__ mean, float* __restrict__ rstd,
                                                            int rows, int d, float eps) {
  grid_dep_sync();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)row * d);
  const int d4 = d >> 2;
  float s = 0.f;
  for (int c = lane; c < d4; c += 32) {
    const float4 v = xr[c];
    s += (v.x + v.y) + (v.z + v.w);
  }
  const float mu = warp_sum(s) / d;
  float q = 0.f;
  for (int c = lane; c < d4; c += 32) {
    const float4 v = xr[c];
    const float a = v.x - mu, b = v.y - mu, cc = v.z - mu, e = v.w - mu;
    q += (a * a + b * b) + (cc * cc + e * e);
  }
  const float rs = rsqrtf(warp_sum(q) / d + eps);
  if (lane == 0) { mean[row] = mu; rstd[row] = rs; }
  uint2* yr = reinterpret_cast<uint2*>(y + (size_t)row * d);
  for (int c = lane; c < d4; c += 32) {
    const float4 v = xr[c];
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + c);
    const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + c);
    uint2 o;
    o.x = pack_bf16x2((v.x - mu) * rs * g.x + b.x, (v.y - mu) * rs * g.y + b.y);
    o.y = pack_bf16x2((v.z - mu) * rs * g.z + b.z, (v.w - mu) * rs * g.w + b.w);
    yr[c] = o;
  }
}

// The same for d = 128 NV (NV <= 8): a row is read once and held in registers between the passes.
template <int NV>
__global__ void __launch_bounds__(256) layernorm_fwd_reg_kernel(const float* __restrict__ x, const float* __restrict__ gamma,
                                                                const float* __restrict__ beta, bf16* __restrict__ y,
                                                                float* __restrict__ mean, float* __restrict__ rstd,
                                                                int rows, float eps) {
  grid_dep_sync();
  constexpr int d = NV * 128;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)row * d);
  float4 v[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = xr[lane + 32 * i];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  const float mu = warp_sum(s) / d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    v[i].x -= mu; v[i].y -= mu; v[i].z -= mu; v[i].w -= mu;
    q += (v[i].x * v[i].x + v[i].y * v[i].y) + (v[i].z * v[i].z + v[i].w * v[i].w);
  }
  const float rs = rsqrtf(warp_sum(q) / d + eps);
  if (lane == 0) { mean[row] = mu; rstd[row] = rs; }
  uint2* yr = reinterpret_cast<uint2*>(y + (size_t)row * d);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + lane + 32 * i);
    const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + lane + 32 * i);
    uint2 o;
    o.x = pack_bf16x2(v[i].x * rs * g.x + b.x, v[i].y * rs * g.y + b.y);
    o.y = pack_bf16x2(v[i].z * rs * g.z + b.z, v[i].w * rs * g.w + b.w);
    yr[lane + 32 * i] = o;
  }
}

cudaError_t layernorm_fwd(const float* x, const float* gamma, const float* beta, bf16* y, float* mean, float* rstd,
                          int rows, int d, float eps, cudaStream_t s) {
  const int blocks = ceil_div(rows, 8);
#define IL_LNR(NV) \
  case NV: launch_dep(layernorm_fwd_reg_kernel<NV>, dim3(blocks), dim3(256), 0, s, x, gamma, beta, y, mean, rstd, rows, eps); break;
  if (d % 128 == 0 && d <= 1024) {
    switch (d / 128) { IL_LNR(1) IL_LNR(2) IL_LNR(3) IL_LNR(4) IL_LNR(5) IL_LNR(6) IL_LNR(7) IL_LNR(8) }
  } else {
    launch_dep(layernorm_fwd_kernel, dim3(blocks), dim3(256), 0, s, x, gamma, beta, y, mean, rstd, rows, d, eps);
  }
#undef IL_LNR
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// LayerNorm backward, row part: one warp per row
// ---------------------------------------------------------------------------------------------
template <bool DY_F32>
__device__ __forceinline__ float4 load_dy4(const void* dy, size_t row, int d, int c4) {
  if constexpr (DY_F32) {
    return reinterpret_cast<const float4*>(reinterpret_cast<const float*>(dy) + row * d)[c4];
  } else {
    const uint2 u = reinterpret_cast<const uint2*>(reinterpret_cast<const bf16*>(dy) + row * d)[c4];
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
}

template <bool DY_F32>
__global__ void __launch_bounds__(256) layernorm_bwd_rows_kernel(const void* __restrict__ dy, const float* __restrict__ x,
                                                                 const float* __restrict__ mean,
                                                                 const float* __restrict__ rstd,
                                                                 const float* __restrict__ gamma, const float* resid,
                                                                 float* dx_out, bf16* __restrict__ dx_bf16, int rows,
                                                                 int x_rows, int d) {
  grid_dep_sync();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int xrow = row % x_rows;
  const float mu = mean[xrow], rs = rstd[xrow];
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)xrow * d);
  const int d4 = d >> 2;
  float s1 = 0.f, s2 = 0.f;
  for (int c = lane; c < d4; c += 32) {
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + c);
    const float4 dv = load_dy4<DY_F32>(dy, (size_t)row, d, c);
    const float4 xv = xr[c];
    const float a0 = dv.x * g.x, a1 = dv.y * g.y, a2 = dv.z * g.z, a3 = dv.w * g.w;
    s1 += (a0 + a1) + (a2 + a3);
    s2 += (a0 * (xv.x - mu) + a1 * (xv.y - mu)) + (a2 * (xv.z - mu) + a3 * (xv.w - mu));
  }
  const float m1 = warp_sum(s1) / d;
  const float m2 = warp_sum(s2) * rs / d;   // mean of dxhat * xhat
  const float4* rr = resid ? reinterpret_cast<const float4*>(resid + (size_t)row * d) : nullptr;
  float4* outr = reinterpret_cast<float4*>(dx_out + (size_t)row * d);
  uint2* outb = dx_bf16 ? reinterpret_cast<uint2*>(dx_bf16 + (size_t)row * d) : nullptr;
  for (int c = lane; c < d4; c += 32) {
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + c);
    const float4 dv = load_dy4<DY_F32>(dy, (size_t)row, d, c);
    const float4 xv = xr[c];
    float4 o;
    o.x = (dv.x * g.x - m1 - (xv.x - mu) * rs * m2) * rs;
    o.y = (dv.y * g.y - m1 - (xv.y - mu) * rs * m2) * rs;
    o.z = (dv.z * g.z - m1 - (xv.z - mu) * rs * m2) * rs;
    o.w = (dv.w * g.w - m1 - (xv.w - mu) * rs * m2) * rs;
    if (rr) {
      const float4 r = rr[c];
      o.x += r.x; o.y += r.y; o.z += r.z; o.w += r.w;
    }
    outr[c] = o;
    if (outb) {
      uint2 b;
      b.x = pack_bf16x2(o.x, o.y);
      b.y = pack_bf16x2(o.z, o.w);
      outb[c] = b;
    }
  }
}

cudaError_t layernorm_bwd_rows(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                               const float* gamma, const float* resid, float* dx_out, bf16* dx_bf16, int rows, int x_rows,
                               int d, cudaStream_t s) {
  if (dy_is_f32)
    launch_dep(layernorm_bwd_rows_kernel<true>, dim3(ceil_div(rows, 8)), dim3(256), 0, s, dy, x, mean, rstd, gamma, resid, dx_out, dx_bf16,
                                                                       rows, x_rows, d);
  else
    launch_dep(layernorm_bwd_rows_kernel<false>, dim3(ceil_div(rows, 8)), dim3(256), 0, s, dy, x, mean, rstd, gamma, resid, dx_out, dx_bf16,
                                                                        rows, x_rows, d);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// LayerNorm backward in one pass over the rows (bf16 dy, d = 128 NV with NV <= 8): the row part as above and, for
// the rows of the first gradient stream (row < x_rows), the column reductions that otherwise take three more
// kernels over the same data: dgamma += dy * xhat, dbeta += dy, and colsum += the kernel's own output (the bias
// gradient of the linear layer whose output this residual-stream gradient belongs to).  A warp walks rows with a
// grid-wide stride, keeps a row's values in registers between the two passes and its column partials in
// registers across rows; the block combines its eight warps through shared memory and adds one value per
// column and output to global memory.  dgamma / dbeta / colsum must be zeroed (or hold a sum to add to).
// ---------------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(256, 1) layernorm_bwd_fused_kernel(const bf16* __restrict__ dy, const float* __restrict__ x,
                                                                     const float* __restrict__ mean,
                                                                     const float* __restrict__ rstd,
                                                                     const float* __restrict__ gamma, const float* resid,
                                                                     float* dx_out, bf16* __restrict__ dx_bf16,
                                                                     float* __restrict__ dgamma, float* __restrict__ dbeta,
                                                                     float* __restrict__ colsum, int rows, int x_rows) {
  grid_dep_sync();
  constexpr int d = NV * 128;
  __shared__ float4 red[8][NV * 32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int warps = gridDim.x * 8;
  float4 g4[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) g4[i] = __ldg(reinterpret_cast<const float4*>(gamma) + lane + 32 * i);
  float4 ag[NV], ab[NV], ac[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) ag[i] = ab[i] = ac[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int row = blockIdx.x * 8 + w; row < rows; row += warps) {
    const int xrow = row % x_rows;
    const bool first = row < x_rows;              // rows of the first stream feed the parameter gradients
    const float mu = mean[xrow], rs = rstd[xrow];
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)xrow * d);
    float4 dv[NV], xh[NV];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      dv[i] = load_dy4<false>(dy, (size_t)row, d, lane + 32 * i);
      const float4 xv = xr[lane + 32 * i];
      xh[i] = make_float4((xv.x - mu) * rs, (xv.y - mu) * rs, (xv.z - mu) * rs, (xv.w - mu) * rs);
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const float a0 = dv[i].x * g4[i].x, a1 = dv[i].y * g4[i].y, a2 = dv[i].z * g4[i].z, a3 = dv[i].w * g4[i].w;
      s1 += (a0 + a1) + (a2 + a3);
      s2 += (a0 * xh[i].x + a1 * xh[i].y) + (a2 * xh[i].z + a3 * xh[i].w);
      if (first) {
        ag[i].x += dv[i].x * xh[i].x; ag[i].y += dv[i].y * xh[i].y; ag[i].z += dv[i].z * xh[i].z; ag[i].w += dv[i].w * xh[i].w;
        ab[i].x += dv[i].x; ab[i].y += dv[i].y; ab[i].z += dv[i].z; ab[i].w += dv[i].w;
      }
    }
    const float m1 = warp_sum(s1) / d;
    const float m2 = warp_sum(s2) / d;          // mean of dxhat * xhat
    const float4* rr = resid ? reinterpret_cast<const float4*>(resid + (size_t)row * d) : nullptr;
    float4* outr = reinterpret_cast<float4*>(dx_out + (size_t)row * d);
    uint2* outb = dx_bf16 ? reinterpret_cast<uint2*>(dx_bf16 + (size_t)row * d) : nullptr;
    float4 r4[NV];
    if (rr) {
#pragma unroll
      for (int i = 0; i < NV; ++i) r4[i] = rr[lane + 32 * i];
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      float4 o;
      o.x = (dv[i].x * g4[i].x - m1 - xh[i].x * m2) * rs;
      o.y = (dv[i].y * g4[i].y - m1 - xh[i].y * m2) * rs;
      o.z = (dv[i].z * g4[i].z - m1 - xh[i].z * m2) * rs;
      o.w = (dv[i].w * g4[i].w - m1 - xh[i].w * m2) * rs;
      if (rr) { o.x += r4[i].x; o.y += r4[i].y; o.z += r4[i].z; o.w += r4[i].w; }
      outr[lane + 32 * i] = o;
      if (outb) {
        uint2 b;
        b.x = pack_bf16x2(o.x, o.y);
        b.y = pack_bf16x2(o.z, o.w);
        outb[lane + 32 * i] = b;
      }
      if (first) { ac[i].x += o.x; ac[i].y += o.y; ac[i].z += o.z; ac[i].w += o.w; }
    }
  }
  // block-level combination, one quantity after the other through the same buffer
#pragma unroll
  for (int q = 0; q < 3; ++q) {
    float* out = q == 0 ? dgamma : q == 1 ? dbeta : colsum;
    if (!out) continue;                           // uniform across the block
#pragma unroll
    for (int i = 0; i < NV; ++i) red[w][lane + 32 * i] = q == 0 ? ag[i] : q == 1 ? ab[i] : ac[i];
    __syncthreads();
    for (int c = threadIdx.x; c < NV * 32; c += 256) {
      float4 t = red[0][c];
#pragma unroll
      for (int k = 1; k < 8; ++k) {
        const float4 v = red[k][c];
        t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
      }
      red_add_f32x4(out + 4 * c, t);
    }
    __syncthreads();
  }
}

// Fused LayerNorm backward for bf16 dy when d is a multiple of 128 up to 1024; returns cudaErrorNotSupported for
// other widths (the caller then uses the separate row and column kernels).  dgamma, dbeta, colsum: fp32 [d],
// summed into (colsum may be NULL).
cudaError_t layernorm_bwd_fused(const bf16* dy, const float* x, const float* mean, const float* rstd, const float* gamma,
                                const float* resid, float* dx_out, bf16* dx_bf16, float* dgamma, float* dbeta,
                                float* colsum, int rows, int x_rows, int d, cudaStream_t s) {
  if (d % 128 || d > 1024 || d < 128) return cudaErrorNotSupported;
  int blocks = ceil_div(rows, 8);
  if (blocks > 148) blocks = 148;
#define IL_LNF(NV)                                                                                                        \
  case NV:                                                                                                                \
    launch_dep(layernorm_bwd_fused_kernel<NV>, dim3(blocks), dim3(256), 0, s, dy, x, mean, rstd, gamma, resid, dx_out, dx_bf16, dgamma, dbeta, \
                                                          colsum, rows, x_rows);                                          \
    break;
  switch (d / 128) {
    IL_LNF(1) IL_LNF(2) IL_LNF(3) IL_LNF(4) IL_LNF(5) IL_LNF(6) IL_LNF(7) IL_LNF(8)
  }
#undef IL_LNF
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Column reductions.  Block = 32 lanes x 8 warps; a lane owns 4 consecutive columns, a block 128 columns;
// the rows are split over gridDim.y; partial sums are combined through shared memory and one atomicAdd
// per column per block.
// ---------------------------------------------------------------------------------------------
template <bool DY_F32>
__global__ void __launch_bounds__(256) layernorm_bwd_params_kernel(const void* __restrict__ dy, const float* __restrict__ x,
                                                                   const float* __restrict__ mean,
                                                                   const float* __restrict__ rstd,
                                                                   float* __restrict__ dgamma, float* __restrict__ dbeta,
                                                                   int rows, int d, int rows_per_block) {
  grid_dep_sync();
  __shared__ float4 sg[8][32], sb[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c4 = blockIdx.x * 32 + lane;       // float4 column index
  const bool col_ok = c4 * 4 < d;
  const int r0 = blockIdx.y * rows_per_block;
  const int r1 = min(rows, r0 + rows_per_block);
  float4 ag = make_float4(0.f, 0.f, 0.f, 0.f), ab = ag;
  if (col_ok) {
    for (int r = r0 + w; r < r1; r += 8) {
      const float mu = mean[r], rs = rstd[r];
      const float4 dv = load_dy4<DY_F32>(dy, (size_t)r, d, c4);
      const float4 xv = reinterpret_cast<const float4*>(x + (size_t)r * d)[c4];
      ag.x += dv.x * (xv.x - mu) * rs; ag.y += dv.y * (xv.y - mu) * rs;
      ag.z += dv.z * (xv.z - mu) * rs; ag.w += dv.w * (xv.w - mu) * rs;
      ab.x += dv.x; ab.y += dv.y; ab.z += dv.z; ab.w += dv.w;
    }
  }
  sg[w][lane] = ag;
  sb[w][lane] = ab;
  __syncthreads();
  if (w == 0 && col_ok) {
    for (int i = 1; i < 8; ++i) {
      const float4 g = sg[i][lane], b = sb[i][lane];
      ag.x += g.x; ag.y += g.y; ag.z += g.z; ag.w += g.w;
      ab.x += b.x; ab.y += b.y; ab.z += b.z; ab.w += b.w;
    }
    float* pg = dgamma + c4 * 4;
    float* pb = dbeta + c4 * 4;
    atomicAdd(pg, ag.x); atomicAdd(pg + 1, ag.y); atomicAdd(pg + 2, ag.z); atomicAdd(pg + 3, ag.w);
    atomicAdd(pb, ab.x); atomicAdd(pb + 1, ab.y); atomicAdd(pb + 2, ab.z); atomicAdd(pb + 3, ab.w);
  }
}

static inline void colreduce_grid(int rows, int cols_per_block, int cols, dim3* grid, int* rows_per_block) {
  const int bx = ceil_div(cols, cols_per_block);
  int by = ceil_div(148 * 4, bx);
  if (by > ceil_div(rows, 8)) by = ceil_div(rows, 8);
  if (by < 1) by = 1;
  *rows_per_block = ceil_div(rows, by);
  by = ceil_div(rows, *rows_per_block);
  *grid = dim3(bx, by, 1);
}

cudaError_t layernorm_bwd_params(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                                 float* dgamma, float* dbeta, int rows, int d, cudaStream_t s) {
  dim3 grid;
  int rpb;
  colreduce_grid(rows, 128, d, &grid, &rpb);
  if (dy_is_f32)
    launch_dep(layernorm_bwd_params_kernel<true>, dim3(grid), dim3(256), 0, s, dy, x, mean, rstd, dgamma, dbeta, rows, d, rpb);
  else
    launch_dep(layernorm_bwd_params_kernel<false>, dim3(grid), dim3(256), 0, s, dy, x, mean, rstd, dgamma, dbeta, rows, d, rpb);
  return cudaGetLastError();
}

template <bool IN_F32>
__global__ void __launch_bounds__(256) colsum_kernel(const void* __restrict__ y, int ld, float* __restrict__ out, int rows,
                                                     int cols, int rows_per_block) {
  grid_dep_sync();
  __shared__ float4 sm[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c4 = blockIdx.x * 32 + lane;
  const bool col_ok = c4 * 4 < cols;
  const int r0 = blockIdx.y * rows_per_block;
  const int r1 = min(rows, r0 + rows_per_block);
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col_ok) {
    int r = r0 + w;
    for (; r + 24 < r1; r += 32) {               // four independent loads in flight per lane
      const float4 v0 = load_dy4<IN_F32>(y, (size_t)r, ld, c4), v1 = load_dy4<IN_F32>(y, (size_t)r + 8, ld, c4);
      const float4 v2 = load_dy4<IN_F32>(y, (size_t)r + 16, ld, c4), v3 = load_dy4<IN_F32>(y, (size_t)r + 24, ld, c4);
      a.x += (v0.x + v1.x) + (v2.x + v3.x); a.y += (v0.y + v1.y) + (v2.y + v3.y);
      a.z += (v0.z + v1.z) + (v2.z + v3.z); a.w += (v0.w + v1.w) + (v2.w + v3.w);
    }
    for (; r < r1; r += 8) {
      const float4 v = load_dy4<IN_F32>(y, (size_t)r, ld, c4);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
  }
  sm[w][lane] = a;
  __syncthreads();
  if (w == 0 && col_ok) {
    for (int i = 1; i < 8; ++i) {
      const float4 v = sm[i][lane];
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    float* po = out + c4 * 4;
    atomicAdd(po, a.x); atomicAdd(po + 1, a.y); atomicAdd(po + 2, a.z); atomicAdd(po + 3, a.w);
  }
}

cudaError_t colsum_bf16(const bf16* y, int ld, float* out, int rows, int cols, cudaStream_t s) {
  dim3 grid;
  int rpb;
  colreduce_grid(rows, 128, cols, &grid, &rpb);
  launch_dep(colsum_kernel<false>, dim3(grid), dim3(256), 0, s, y, ld, out, rows, cols, rpb);
  return cudaGetLastError();
}
cudaError_t colsum_f32(const float* y, int ld, float* out, int rows, int cols, cudaStream_t s) {
  dim3 grid;
  int rpb;
  colreduce_grid(rows, 128, cols, &grid, &rpb);
  launch_dep(colsum_kernel<true>, dim3(grid), dim3(256), 0, s, y, ld, out, rows, cols, rpb);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Elementwise
// ---------------------------------------------------------------------------------------------
__global__ void add_convert_kernel(const float4* __restrict__ a, const float4* __restrict__ b, float4* out_f32,
                                   uint2* __restrict__ out_bf16, size_t n4) {
  grid_dep_sync();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 v = a[i];
    if (b) {
      const float4 w = b[i];
      v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
    }
    if (out_f32) out_f32[i] = v;
    if (out_bf16) {
      uint2 o;
      o.x = pack_bf16x2(v.x, v.y);
      o.y = pack_bf16x2(v.z, v.w);
      out_bf16[i] = o;
    }
  }
}

cudaError_t add_convert(const float* a, const float* b, float* out_f32, bf16* out_bf16, size_t n, cudaStream_t s) {
  const size_t n4 = n / 4;
  int blocks = ceil_div(n4, 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  launch_dep(add_convert_kernel, dim3(blocks), dim3(256), 0, s, reinterpret_cast<const float4*>(a), reinterpret_cast<const float4*>(b),
                                            reinterpret_cast<float4*>(out_f32), reinterpret_cast<uint2*>(out_bf16), n4);
  return cudaGetLastError();
}

struct LinComb { const float4* x[4]; float w[4]; int count; int accumulate; };

__global__ void lincomb_convert_kernel(LinComb c, float4* out_f32, uint2* __restrict__ out_bf16, size_t n4) {
  grid_dep_sync();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 v = c.accumulate ? out_f32[i] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (j < c.count) {
        const float4 a = c.x[j][i];
        v.x += c.w[j] * a.x; v.y += c.w[j] * a.y; v.z += c.w[j] * a.z; v.w += c.w[j] * a.w;
      }
    out_f32[i] = v;
    if (out_bf16) {
      uint2 o;
      o.x = pack_bf16x2(v.x, v.y);
      o.y = pack_bf16x2(v.z, v.w);
      out_bf16[i] = o;
    }
  }
}

cudaError_t lincomb_convert(const float* const* x, const float* w, int count, int accumulate, float* out_f32, bf16* out_bf16,
                            size_t n, cudaStream_t s) {
  if (count < 1 || count > 4 || !out_f32) return cudaErrorInvalidValue;
  LinComb c;
  for (int j = 0; j < 4; ++j) {
    c.x[j] = reinterpret_cast<const float4*>(j < count ? x[j] : x[0]);
    c.w[j] = j < count ? w[j] : 0.f;
  }
  c.count = count;
  c.accumulate = accumulate;
  const size_t n4 = n / 4;
  int blocks = ceil_div(n4, 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  launch_dep(lincomb_convert_kernel, dim3(blocks), dim3(256), 0, s, c, reinterpret_cast<float4*>(out_f32), reinterpret_cast<uint2*>(out_bf16), n4);
  return cudaGetLastError();
}

cudaError_t f32_to_bf16(const float* in, bf16* out, size_t n, cudaStream_t s) {
  return add_convert(in, nullptr, nullptr, out, n, s);
}

// ---------------------------------------------------------------------------------------------
// Merge of the per-tile softmax partials and the mean cross-entropy: one warp per row
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) lse_finalize_kernel(const float* __restrict__ pm, const float* __restrict__ ps,
                                                           int part_ld, int ntiles, const float* __restrict__ tgt_logit,
                                                           float* __restrict__ lse, float* __restrict__ nll, int rows) {
  grid_dep_sync();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int row = blockIdx.x * 8 + w;
  if (row >= rows) return;
  float m = -INFINITY;
  for (int t = lane; t < ntiles; t += 32) m = fmaxf(m, pm[(size_t)row * part_ld + t]);
  m = warp_max(m);
  float sum = 0.f;
  for (int t = lane; t < ntiles; t += 32) {
    const float tm = pm[(size_t)row * part_ld + t];
    if (tm > -INFINITY) sum += ps[(size_t)row * part_ld + t] * __expf(tm - m);
  }
  sum = warp_sum(sum);
  const float l = m + logf(sum);
  if (lane == 0) {
    lse[row] = l;
    nll[row] = l - tgt_logit[row];
  }
}

cudaError_t lse_finalize(const float* part_max, const float* part_sum, int part_ld, int ntiles, const float* tgt_logit,
                         float* lse, float* nll, int rows, cudaStream_t s) {
  launch_dep(lse_finalize_kernel, dim3(ceil_div(rows, 8)), dim3(256), 0, s, part_max, part_sum, part_ld, ntiles, tgt_logit, lse, nll, rows);
  return cudaGetLastError();
}

// out[0] = mean of x[0..n) with a fixed summation order (one block: strided per-thread sums, then a tree), so the
// value does not depend on scheduling.
__global__ void __launch_bounds__(1024) mean_f32_kernel(const float* __restrict__ x, int n, float* __restrict__ out) {
  grid_dep_sync();
  __shared__ float sm[1024];
  float a = 0.f;
  for (int i = threadIdx.x; i < n; i += 1024) a += x[i];
  sm[threadIdx.x] = a;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[0] = sm[0] / (float)n;
}

cudaError_t mean_f32(const float* x, int n, float* out, cudaStream_t s) {
  launch_dep(mean_f32_kernel, dim3(1), dim3(1024), 0, s, x, n, out);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Head backward set-up.  The loss pass kept E = exp(logits) (bf16).  With s_r = exp(-lse_r) / rows the gradient
// of the mean cross-entropy is dZ[r, c] = s_r * (E[r, c] - [c == target_r] * exp(lse_r)), so one warp per row
//   * subtracts exp(lse_r) from the target's entry of E (the bf16 rounding of that difference is, relative to
//     the entry, what rounding dZ itself would be),
//   * writes s_r for the epilogue of dU = diag(s) (E W),
//   * writes U'[r, :] = s_r * U[r, :] (bf16) for dW = E^T U'.
// exp(logit) must stay inside the bf16 / fp32 range: rows whose lse leaves [-80, 80] raise the error word.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) head_backward_prepare_kernel(bf16* __restrict__ e, int ld, const float* __restrict__ lse,
                                                                    const int* __restrict__ targets, const bf16* __restrict__ u,
                                                                    bf16* __restrict__ u_scaled, float* __restrict__ rowscale,
                                                                    int rows, int d, float inv_rows, unsigned* err) {
  grid_dep_sync();
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float l = lse[row];
  if (!(l >= -80.0f && l <= 80.0f)) {
    if (lane == 0) atomicExch(err, DEV_LOGIT_RANGE);
    return;
  }
  const float s = __expf(-l) * inv_rows;
  if (lane == 0) {
    rowscale[row] = s;
    bf16* et = e + (size_t)row * ld + targets[row];
    *et = __float2bfloat16(__bfloat162float(*et) - __expf(l));
  }
  const uint4* ur = reinterpret_cast<const uint4*>(u + (size_t)row * d);
  uint4* us = reinterpret_cast<uint4*>(u_scaled + (size_t)row * d);
  for (int c8 = lane; c8 < d / 8; c8 += 32) {
    const uint4 raw = ur[c8];
    uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
      w[i] = pack_bf16x2(f.x * s, f.y * s);
    }
    us[c8] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

cudaError_t head_backward_prepare(bf16* e, int ld, const float* lse, const int* targets, const bf16* u, bf16* u_scaled,
                                  float* rowscale, int rows, int d, float scale, unsigned* err, cudaStream_t s) {
  if ((d % 8) || ((uintptr_t)u % 16) || ((uintptr_t)u_scaled % 16) || !err) return cudaErrorInvalidValue;
  launch_dep(head_backward_prepare_kernel, dim3(ceil_div(rows, 8)), dim3(256), 0, s, e, ld, lse, targets, u, u_scaled, rowscale, rows, d,
                                                                 scale / (float)rows, err);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// AdamW: 16 bytes/param read (p, m, v, g), 12 written (p, m, v) + 2 (bf16 shadow) = 30 B/param
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) adamw_kernel(float4* __restrict__ p, float4* __restrict__ m, float4* __restrict__ v,
                                                    const float4* __restrict__ g, uint2* __restrict__ pb, size_t n4,
                                                    size_t n4_decay, float lr, float b1, float b2, float eps, float wd,
                                                    float ibc1, float ibc2, const unsigned* __restrict__ err,
                                                    unsigned* applied, size_t skip0, size_t skip1) {
  grid_dep_sync();
  // a step whose kernels reported an error must not reach the parameters: leave everything as it is
  if (err && *reinterpret_cast<const volatile unsigned*>(err) != 0u) return;
  if (applied && blockIdx.x == 0 && threadIdx.x == 0) *applied += 1u;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    if (i >= skip0 && i < skip1) continue;          // a sub-range updated by another launch
    const float w = i < n4_decay ? wd : 0.f;
    float4 pv = p[i], mv = m[i], vv = v[i];
    const float4 gv = g[i];
#define IL_ADAM1(F)                                                        \
  mv.F = b1 * mv.F + (1.f - b1) * gv.F;                                    \
  vv.F = b2 * vv.F + (1.f - b2) * gv.F * gv.F;                             \
  pv.F = pv.F - lr * ((mv.F * ibc1) / (sqrtf(vv.F * ibc2) + eps) + w * pv.F);
    IL_ADAM1(x) IL_ADAM1(y) IL_ADAM1(z) IL_ADAM1(w)
#undef IL_ADAM1
    p[i] = pv; m[i] = mv; v[i] = vv;
    uint2 o;
    o.x = pack_bf16x2(pv.x, pv.y);
    o.y = pack_bf16x2(pv.z, pv.w);
    pb[i] = o;
  }
}

cudaError_t adamw(float* p, float* m, float* v, const float* g, bf16* p_bf16, size_t n, size_t n_decay, float lr,
                  float beta1, float beta2, float eps, float wd, float bc1, float bc2, const unsigned* err, unsigned* applied,
                  size_t skip_begin, size_t skip_end, cudaStream_t s) {
  const size_t n4 = n / 4;
  if (n4 == 0) return cudaSuccess;
  int blocks = ceil_div(n4, 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  launch_dep(adamw_kernel, dim3(blocks), dim3(256), 0, s, reinterpret_cast<float4*>(p), reinterpret_cast<float4*>(m),
                                      reinterpret_cast<float4*>(v), reinterpret_cast<const float4*>(g),
                                      reinterpret_cast<uint2*>(p_bf16), n4, n_decay / 4, lr, beta1, beta2, eps, wd,
                                      1.0f / bc1, 1.0f / bc2, err, applied, skip_begin / 4, skip_end / 4);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// A wait that cannot succeed: one thread waits, with the given limit, on an mbarrier nobody arrives at, and
// reports the expiry the way the pipelined kernels do.  It exercises the error path (error word -> host status)
// without any kernel having to go wrong.
// ---------------------------------------------------------------------------------------------
__global__ void wait_probe_kernel(unsigned* err, unsigned long long limit_ns) {
  grid_dep_sync();
  __shared__ unsigned long long bar;
  __shared__ int never;
  if (threadIdx.x == 0) {
    never = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
    if (!mbar_wait(smem_u32(&bar), 0, &never, limit_ns)) atomicExch(err, DEV_TIMEOUT_EPILOGUE);
  }
}

cudaError_t wait_probe(unsigned* err, unsigned long long limit_ns, cudaStream_t s) {
  launch_dep(wait_probe_kernel, dim3(1), dim3(32), 0, s, err, limit_ns);
  return cudaGetLastError();
}

}  // namespace il
