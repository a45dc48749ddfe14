// Causal self-attention forward and backward on packed qkv [B*T, 3d] (softmax(Q K^T / sqrt(dh)) V).
//
// Blockwise online-softmax formulation: the T x T score matrix is never stored.  One CTA owns a block of
// 64 query rows (forward, dQ) or 64 key rows (dK/dV) of one (sequence, head) and sweeps the other index in
// blocks of 64; each of its 4 warps owns 16 rows.  Contractions run on the tensor cores through
// mma.sync m16n8k16 (bf16 in, fp32 accumulate) with ldmatrix-fed fragments; softmax statistics are fp32.
// Backward recomputes the probabilities from the saved per-row log-sum-exp and uses
// delta_i = sum_c dO_ic O_ic (= sum_j P_ij dP_ij).
#include "common.cuh"
#include "kernels.h"

namespace il {

constexpr int AT_BLK = 64;        // rows per CTA tile and per sweep step
constexpr int AT_THREADS = 128;
#define LOG2E_F 1.4426950408889634f

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

// Copy a [64, DH] bf16 tile (row stride ld elements, rows >= rows_valid zero-filled) into padded smem.
template <int DH>
__device__ __forceinline__ void load_tile(bf16* dst, const bf16* src, int ld, int row0, int rows_valid) {
  constexpr int LD = DH + 8;
  constexpr int CH = DH / 8;
  for (int i = threadIdx.x; i < AT_BLK * CH; i += AT_THREADS) {
    const int r = i / CH, c = i % CH;
    const bool ok = (row0 + r) < rows_valid;
    const bf16* g = src + (size_t)(ok ? row0 + r : 0) * ld + c * 8;
    cp_async16(smem_u32(dst + r * LD + c * 8), g, ok);
  }
}

// A-operand fragment (16 rows x 16 k) from row-major smem [rows][LD]
template <int LD>
__device__ __forceinline__ void load_a(const bf16* s, int row0, int k0, uint32_t (&a)[4]) {
  const int lane = threadIdx.x & 31;
  const int r = row0 + (lane & 7) + 8 * ((lane >> 3) & 1);
  const int c = k0 + 8 * (lane >> 4);
  ldsm_x4(smem_u32(s + r * LD + c), a[0], a[1], a[2], a[3]);
}
// B-operand fragments for two adjacent n-tiles (16 n x 16 k) where smem holds [n][k] (k contiguous)
template <int LD>
__device__ __forceinline__ void load_b_nk(const bf16* s, int n0, int k0, uint32_t (&b)[4]) {
  const int lane = threadIdx.x & 31;
  const int r = n0 + (lane & 7) + 8 * (lane >> 4);
  const int c = k0 + 8 * ((lane >> 3) & 1);
  ldsm_x4(smem_u32(s + r * LD + c), b[0], b[1], b[2], b[3]);
}
// B-operand fragments for two adjacent n-tiles where smem holds [k][n] (n contiguous): transposing load
template <int LD>
__device__ __forceinline__ void load_b_kn(const bf16* s, int k0, int n0, uint32_t (&b)[4]) {
  const int lane = threadIdx.x & 31;
  const int r = k0 + (lane & 7) + 8 * ((lane >> 3) & 1);
  const int c = n0 + 8 * (lane >> 4);
  ldsm_x4_t(smem_u32(s + r * LD + c), b[0], b[1], b[2], b[3]);
}

// acc[8 n-tiles] (16 x 64) = A[16 x DH] (smem rows a_row0..) * Bs[64 x DH]^T
template <int DH>
__device__ __forceinline__ void mm_16x64_nk(float (&acc)[8][4], const bf16* sA, int a_row0, const bf16* sB) {
  constexpr int LD = DH + 8;
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
#pragma unroll
  for (int ks = 0; ks < DH / 16; ++ks) {
    uint32_t a[4];
    load_a<LD>(sA, a_row0, ks * 16, a);
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      load_b_nk<LD>(sB, np * 16, ks * 16, b);
      mma_bf16(acc[2 * np], a, b[0], b[1]);
      mma_bf16(acc[2 * np + 1], a, b[2], b[3]);
    }
  }
}

// out[DH/8 n-tiles] (16 x DH) += P[16 x 64] (register fragments) * Bs[64 x DH]   (Bs row-major [k][n])
template <int DH>
__device__ __forceinline__ void mm_acc_p(float (&out)[DH / 8][4], const uint32_t (&p)[4][4], const bf16* sB) {
  constexpr int LD = DH + 8;
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
    for (int dp = 0; dp < DH / 16; ++dp) {
      uint32_t b[4];
      load_b_kn<LD>(sB, kk * 16, dp * 16, b);
      mma_bf16(out[2 * dp], p[kk], b[0], b[1]);
      mma_bf16(out[2 * dp + 1], p[kk], b[2], b[3]);
    }
  }
}

__device__ __forceinline__ void pack_p(const float (&s)[8][4], uint32_t (&p)[4][4]) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    p[kk][0] = pack_bf16x2(s[2 * kk][0], s[2 * kk][1]);
    p[kk][1] = pack_bf16x2(s[2 * kk][2], s[2 * kk][3]);
    p[kk][2] = pack_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
    p[kk][3] = pack_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
  }
}

// ---------------------------------------------------------------------------------------------
// Forward
// ---------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(AT_THREADS) attn_fwd_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ o,
                                                              float* __restrict__ lse, int T, int H, float scale) {
  constexpr int LD = DH + 8;
  extern __shared__ __align__(16) uint8_t at_smem[];
  bf16* sQ = reinterpret_cast<bf16*>(at_smem);
  bf16* sK = sQ + AT_BLK * LD;
  bf16* sV = sK + AT_BLK * LD;
  const int qt = gridDim.x - 1 - blockIdx.x;      // longest sweeps first
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  const int d = H * DH;
  const int ld = 3 * d;
  const bf16* qb = qkv + (size_t)b * T * ld + h * DH;
  const bf16* kb = qb + d;
  const bf16* vb = qb + 2 * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const float c = scale * LOG2E_F;

  load_tile<DH>(sQ, qb, ld, qt * AT_BLK, T);
  float oacc[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[j][e] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY};
  float lrow[2] = {0.f, 0.f};

  for (int kt = 0; kt <= qt; ++kt) {
    __syncthreads();   // previous sweep step has finished reading sK/sV
    load_tile<DH>(sK, kb, ld, kt * AT_BLK, T);
    load_tile<DH>(sV, vb, ld, kt * AT_BLK, T);
    cp_async_wait_all();
    __syncthreads();
    float s[8][4];
    mm_16x64_nk<DH>(s, sQ, warp * 16, sK);
    if (kt == qt) {
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = j * 8 + 2 * t4 + (e & 1);
          const int qry = warp * 16 + g + 8 * (e >> 1);
          if (key > qry) s[j][e] = -INFINITY;
        }
    }
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      mx[0] = fmaxf(mx[0], fmaxf(s[j][0], s[j][1]));
      mx[1] = fmaxf(mx[1], fmaxf(s[j][2], s[j][3]));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    float alpha[2], mc[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const float mn = fmaxf(mrow[r], mx[r]);      // finite: key 0 is always visible
      alpha[r] = exp2f((mrow[r] - mn) * c);
      mrow[r] = mn;
      mc[r] = mn * c;
      lrow[r] *= alpha[r];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      s[j][0] = exp2f(s[j][0] * c - mc[0]);
      s[j][1] = exp2f(s[j][1] * c - mc[0]);
      s[j][2] = exp2f(s[j][2] * c - mc[1]);
      s[j][3] = exp2f(s[j][3] * c - mc[1]);
      lrow[0] += s[j][0] + s[j][1];
      lrow[1] += s[j][2] + s[j][3];
    }
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) {
      oacc[j][0] *= alpha[0]; oacc[j][1] *= alpha[0];
      oacc[j][2] *= alpha[1]; oacc[j][3] *= alpha[1];
    }
    uint32_t p[4][4];
    pack_p(s, p);
    mm_acc_p<DH>(oacc, p, sV);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int qry = qt * AT_BLK + warp * 16 + g + 8 * r;
    if (qry < T) {
      const float inv = 1.0f / lrow[r];
      bf16* orow = o + ((size_t)b * T + qry) * d + h * DH;
#pragma unroll
      for (int j = 0; j < DH / 8; ++j)
        *reinterpret_cast<uint32_t*>(orow + j * 8 + 2 * t4) = pack_bf16x2(oacc[j][2 * r] * inv, oacc[j][2 * r + 1] * inv);
      if (t4 == 0) lse[((size_t)b * H + h) * T + qry] = mrow[r] * scale + logf(lrow[r]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Backward: delta, dK/dV, dQ
// ---------------------------------------------------------------------------------------------
// delta[nb, h, t] = sum_c dO[nb*T+t, h*dh+c] * O[(nb%B)*T+t, h*dh+c];  one warp per (row, head)
__global__ void __launch_bounds__(256) attn_delta_kernel(const bf16* __restrict__ dout, const bf16* __restrict__ o,
                                                         float* __restrict__ delta, int NB, int B, int T, int H, int dh) {
  const int wid = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int total = NB * T * H;
  if (wid >= total) return;
  const int h = wid % H;
  const int row = wid / H;               // nb*T + t
  const int nb = row / T, t = row % T;
  const int d = H * dh;
  const bf16* a = dout + (size_t)row * d + h * dh;
  const bf16* bb = o + ((size_t)(nb % B) * T + t) * d + h * dh;
  float s = 0.f;
  for (int c = lane * 2; c < dh; c += 64) {
    const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(a + c));
    const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(bb + c));
    s += x.x * y.x + x.y * y.y;
  }
  s = warp_sum(s);
  if (lane == 0) delta[((size_t)nb * H + h) * T + t] = s;
}

template <int DH>
__global__ void __launch_bounds__(AT_THREADS) attn_bwd_dkv_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                                                                  const bf16* __restrict__ dout,
                                                                  const float* __restrict__ delta, bf16* __restrict__ dqkv,
                                                                  int B, int T, int H, float scale) {
  constexpr int LD = DH + 8;
  extern __shared__ __align__(16) uint8_t at_smem[];
  bf16* sK = reinterpret_cast<bf16*>(at_smem);
  bf16* sV = sK + AT_BLK * LD;
  bf16* sQ = sV + AT_BLK * LD;
  bf16* sdO = sQ + AT_BLK * LD;
  float* sLse = reinterpret_cast<float*>(sdO + AT_BLK * LD);
  float* sDel = sLse + AT_BLK;
  const int kt = blockIdx.x;
  const int nb = blockIdx.y / H, h = blockIdx.y % H;
  const int bs = nb % B;
  const int d = H * DH, ld = 3 * d;
  const bf16* qb = qkv + (size_t)bs * T * ld + h * DH;
  const bf16* dob = dout + (size_t)nb * T * d + h * DH;
  const float* lseb = lse + ((size_t)bs * H + h) * T;
  const float* delb = delta + ((size_t)nb * H + h) * T;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const float c = scale * LOG2E_F;
  const int nq = (T + AT_BLK - 1) / AT_BLK;

  load_tile<DH>(sK, qb + d, ld, kt * AT_BLK, T);
  load_tile<DH>(sV, qb + 2 * d, ld, kt * AT_BLK, T);
  float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) { dk[j][e] = 0.f; dv[j][e] = 0.f; }

  for (int qt = kt; qt < nq; ++qt) {
    __syncthreads();
    load_tile<DH>(sQ, qb, ld, qt * AT_BLK, T);
    load_tile<DH>(sdO, dob, d, qt * AT_BLK, T);
    if (threadIdx.x < AT_BLK) {
      const int q = qt * AT_BLK + threadIdx.x;
      sLse[threadIdx.x] = q < T ? lseb[q] * LOG2E_F : 0.f;
      sDel[threadIdx.x] = q < T ? delb[q] : 0.f;
    }
    cp_async_wait_all();
    __syncthreads();
    // S^T (16 keys x 64 queries) and dP^T
    float st[8][4], dpt[8][4];
    mm_16x64_nk<DH>(st, sK, warp * 16, sQ);
    mm_16x64_nk<DH>(dpt, sV, warp * 16, sdO);
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kt * AT_BLK + warp * 16 + g + 8 * (e >> 1);
        const int ql = j * 8 + 2 * t4 + (e & 1);
        const int qry = qt * AT_BLK + ql;
        const float p = (qry >= key && qry < T) ? exp2f(st[j][e] * c - sLse[ql]) : 0.f;
        st[j][e] = p;
        dpt[j][e] = p * (dpt[j][e] - sDel[ql]);
      }
    uint32_t pf[4][4];
    pack_p(st, pf);
    mm_acc_p<DH>(dv, pf, sdO);
    pack_p(dpt, pf);
    mm_acc_p<DH>(dk, pf, sQ);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int key = kt * AT_BLK + warp * 16 + g + 8 * r;
    if (key < T) {
      bf16* row = dqkv + ((size_t)nb * T + key) * ld + h * DH;
#pragma unroll
      for (int j = 0; j < DH / 8; ++j) {
        *reinterpret_cast<uint32_t*>(row + d + j * 8 + 2 * t4) = pack_bf16x2(dk[j][2 * r] * scale, dk[j][2 * r + 1] * scale);
        *reinterpret_cast<uint32_t*>(row + 2 * d + j * 8 + 2 * t4) = pack_bf16x2(dv[j][2 * r], dv[j][2 * r + 1]);
      }
    }
  }
}

template <int DH>
__global__ void __launch_bounds__(AT_THREADS) attn_bwd_dq_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                                                                 const bf16* __restrict__ dout,
                                                                 const float* __restrict__ delta, bf16* __restrict__ dqkv,
                                                                 int B, int T, int H, float scale) {
  constexpr int LD = DH + 8;
  extern __shared__ __align__(16) uint8_t at_smem[];
  bf16* sQ = reinterpret_cast<bf16*>(at_smem);
  bf16* sdO = sQ + AT_BLK * LD;
  bf16* sK = sdO + AT_BLK * LD;
  bf16* sV = sK + AT_BLK * LD;
  const int qt = gridDim.x - 1 - blockIdx.x;
  const int nb = blockIdx.y / H, h = blockIdx.y % H;
  const int bs = nb % B;
  const int d = H * DH, ld = 3 * d;
  const bf16* qb = qkv + (size_t)bs * T * ld + h * DH;
  const bf16* dob = dout + (size_t)nb * T * d + h * DH;
  const float* lseb = lse + ((size_t)bs * H + h) * T;
  const float* delb = delta + ((size_t)nb * H + h) * T;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const float c = scale * LOG2E_F;

  load_tile<DH>(sQ, qb, ld, qt * AT_BLK, T);
  load_tile<DH>(sdO, dob, d, qt * AT_BLK, T);
  float lrow[2], drow[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int q = qt * AT_BLK + warp * 16 + g + 8 * r;
    lrow[r] = q < T ? lseb[q] * LOG2E_F : 0.f;
    drow[r] = q < T ? delb[q] : 0.f;
  }
  float dq[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) dq[j][e] = 0.f;

  for (int kt = 0; kt <= qt; ++kt) {
    __syncthreads();
    load_tile<DH>(sK, qb + d, ld, kt * AT_BLK, T);
    load_tile<DH>(sV, qb + 2 * d, ld, kt * AT_BLK, T);
    cp_async_wait_all();
    __syncthreads();
    float s[8][4], dp[8][4];
    mm_16x64_nk<DH>(s, sQ, warp * 16, sK);
    mm_16x64_nk<DH>(dp, sdO, warp * 16, sV);
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kt * AT_BLK + j * 8 + 2 * t4 + (e & 1);
        const int r = e >> 1;
        const int qry = qt * AT_BLK + warp * 16 + g + 8 * r;
        const float p = (key <= qry && key < T) ? exp2f(s[j][e] * c - lrow[r]) : 0.f;
        dp[j][e] = p * (dp[j][e] - drow[r]);
      }
    uint32_t pf[4][4];
    pack_p(dp, pf);
    mm_acc_p<DH>(dq, pf, sK);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int qry = qt * AT_BLK + warp * 16 + g + 8 * r;
    if (qry < T) {
      bf16* row = dqkv + ((size_t)nb * T + qry) * ld + h * DH;
#pragma unroll
      for (int j = 0; j < DH / 8; ++j)
        *reinterpret_cast<uint32_t*>(row + j * 8 + 2 * t4) = pack_bf16x2(dq[j][2 * r] * scale, dq[j][2 * r + 1] * scale);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------
template <int DH>
static cudaError_t fwd_launch(const bf16* qkv, bf16* o, float* lse, int B, int T, int H, cudaStream_t s) {
  const int smem = 3 * AT_BLK * (DH + 8) * 2;
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  dim3 grid((T + AT_BLK - 1) / AT_BLK, B * H);
  attn_fwd_kernel<DH><<<grid, AT_THREADS, smem, s>>>(qkv, o, lse, T, H, rsqrtf((float)DH));
  return cudaGetLastError();
}

cudaError_t attention_fwd_legacy(const bf16* qkv, bf16* o, float* lse, int B, int T, int H, int dh, cudaStream_t s) {
  switch (dh) {
    case 32: return fwd_launch<32>(qkv, o, lse, B, T, H, s);
    case 64: return fwd_launch<64>(qkv, o, lse, B, T, H, s);
    case 80: return fwd_launch<80>(qkv, o, lse, B, T, H, s);
    case 128: return fwd_launch<128>(qkv, o, lse, B, T, H, s);
  }
  return cudaErrorInvalidValue;
}

template <int DH>
static cudaError_t bwd_launch(const bf16* qkv, const bf16* o, const float* lse, const bf16* dout, bf16* dqkv, float* delta,
                              int NB, int B, int T, int H, cudaStream_t s) {
  const int smem_kv = 4 * AT_BLK * (DH + 8) * 2 + 2 * AT_BLK * 4;
  const int smem_q = 4 * AT_BLK * (DH + 8) * 2;
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_dkv_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_kv);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_bwd_dq_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_q);
  if (e != cudaSuccess) return e;
  const int nwarps = NB * T * H;
  attn_delta_kernel<<<(nwarps + 7) / 8, 256, 0, s>>>(dout, o, delta, NB, B, T, H, DH);
  dim3 grid((T + AT_BLK - 1) / AT_BLK, NB * H);
  const float scale = rsqrtf((float)DH);
  attn_bwd_dkv_kernel<DH><<<grid, AT_THREADS, smem_kv, s>>>(qkv, lse, dout, delta, dqkv, B, T, H, scale);
  attn_bwd_dq_kernel<DH><<<grid, AT_THREADS, smem_q, s>>>(qkv, lse, dout, delta, dqkv, B, T, H, scale);
  return cudaGetLastError();
}

cudaError_t attention_bwd_legacy(const bf16* qkv, const bf16* o, const float* lse, const bf16* dout, bf16* dqkv, float* delta,
                          int NB, int B, int T, int H, int dh, cudaStream_t s) {
  switch (dh) {
    case 32: return bwd_launch<32>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, s);
    case 64: return bwd_launch<64>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, s);
    case 80: return bwd_launch<80>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, s);
    case 128: return bwd_launch<128>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace il
