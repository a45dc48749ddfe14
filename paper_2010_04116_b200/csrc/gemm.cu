// tcgen05 GEMM for sm_100a: C[M,N] = A[M,K] * B[N,K]^T, bf16 operands, fp32 accumulation in TMEM.
//
// One persistent CTA per SM walks a static list of 128 x 256 output tiles.  Warp roles:
//   warp 0    : TMA producer — one elected thread streams 128x64 (A) and 256x64 (B) bf16 slabs into a
//               4-stage shared-memory ring (128-byte swizzle), signalling "full" mbarriers by byte count.
//   warp 1    : MMA issuer — allocates 512 TMEM columns (two 128x256 fp32 accumulators), one thread
//               issues tcgen05.mma (M128 N256 K16) four times per slab, commits to the slab's "empty"
//               barrier and, per tile, to the accumulator's "full" barrier.
//   warps 2-5 : epilogue — tcgen05.ld the accumulator (32 lanes x 32 columns per load), apply the fused
//               epilogue and store to global memory, then release the accumulator.  The second
//               accumulator lets the next tile's main loop overlap this epilogue.
// Operands may be K-major or MN-major in global memory (forward: K/K, dgrad: K/MN, wgrad: MN/MN); the
// major-ness goes into the TMA box shape, the shared-memory descriptor and the instruction descriptor.
// Ragged M/N/K edges rely on TMA zero fill for loads and on bounds checks in the epilogue.
// Every wait is bounded; on expiry the CTA sets the error word, drains and returns.
#include <cstdio>
#include <mutex>

#include "common.cuh"
#include "gemm.h"

namespace il {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;             // 16 KB
constexpr int B_BYTES = BN * BK * 2;             // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 48 KB
constexpr int TMEM_COLS = 2 * BN;                // 512 columns: two accumulators
constexpr int GEMM_THREADS = 192;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct GemmDev {
  int M, N, K;
  int tiles_m, tiles_n;
  void* C;
  int ldc;
  void* C2;
  const float* bias;
  const float* resid;
  const bf16* aux;
  int ld_aux, aux_rows;
  int accumulate;
  const int* targets;
  float* part_max;
  float* part_sum;
  int part_ld;
  float* tgt_logit;
  const float* lse;
  float scale;
  int col0;
  unsigned* err;
};

struct RowState {   // per-thread state carried across the 32-column chunks of one tile row (EPI_LSE)
  float m, s, tl;
  int tgt;
};

template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmDev& p, int row, int col, const uint32_t (&r)[32],
                                               RowState& st) {
  const bool full = (col + 32 <= p.N);
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);

  if constexpr (EPI == EPI_BF16 || EPI == EPI_BF16_GELU || EPI == EPI_F32_RESID) {
    if (p.bias) {
      if (full) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col + j));
          v[j] += b.x; v[j + 1] += b.y; v[j + 2] += b.z; v[j + 3] += b.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col + j < p.N) v[j] += __ldg(p.bias + col + j);
      }
    }
  }

  if constexpr (EPI == EPI_BF16 || EPI == EPI_BF16_GELU) {
    bf16* c = reinterpret_cast<bf16*>(p.C) + (size_t)row * p.ldc + col;
    bf16* c2 = (EPI == EPI_BF16_GELU) ? reinterpret_cast<bf16*>(p.C2) + (size_t)row * p.ldc + col : nullptr;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 o;
        o.x = pack_bf16x2(v[j], v[j + 1]); o.y = pack_bf16x2(v[j + 2], v[j + 3]);
        o.z = pack_bf16x2(v[j + 4], v[j + 5]); o.w = pack_bf16x2(v[j + 6], v[j + 7]);
        *reinterpret_cast<uint4*>(c + j) = o;
        if constexpr (EPI == EPI_BF16_GELU) {
          uint4 g;
          g.x = pack_bf16x2(gelu_tanh(v[j]), gelu_tanh(v[j + 1]));
          g.y = pack_bf16x2(gelu_tanh(v[j + 2]), gelu_tanh(v[j + 3]));
          g.z = pack_bf16x2(gelu_tanh(v[j + 4]), gelu_tanh(v[j + 5]));
          g.w = pack_bf16x2(gelu_tanh(v[j + 6]), gelu_tanh(v[j + 7]));
          *reinterpret_cast<uint4*>(c2 + j) = g;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col + j < p.N) {
          c[j] = __float2bfloat16(v[j]);
          if constexpr (EPI == EPI_BF16_GELU) c2[j] = __float2bfloat16(gelu_tanh(v[j]));
        }
    }
  } else if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
    float* c = reinterpret_cast<float*>(p.C) + (size_t)row * p.ldc + col;
    const float* add = nullptr;
    if constexpr (EPI == EPI_F32_RESID) add = p.resid + (size_t)row * p.ldc + col;
    else if (p.accumulate) add = c;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        float4 o = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        if (add) {
          float4 a = *reinterpret_cast<const float4*>(add + j);
          o.x += a.x; o.y += a.y; o.z += a.z; o.w += a.w;
        }
        *reinterpret_cast<float4*>(c + j) = o;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col + j < p.N) c[j] = v[j] + (add ? add[j] : 0.0f);
    }
  } else if constexpr (EPI == EPI_BF16_DGELU) {
    bf16* c = reinterpret_cast<bf16*>(p.C) + (size_t)row * p.ldc + col;
    const bf16* h = p.aux + (size_t)(row % p.aux_rows) * p.ld_aux + col;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 hv = *reinterpret_cast<const uint4*>(h + j);
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&hv);
        float g[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float2 f = __bfloat1622float2(h2[q]);
          g[2 * q] = v[j + 2 * q] * gelu_tanh_grad(f.x);
          g[2 * q + 1] = v[j + 2 * q + 1] * gelu_tanh_grad(f.y);
        }
        uint4 o;
        o.x = pack_bf16x2(g[0], g[1]); o.y = pack_bf16x2(g[2], g[3]);
        o.z = pack_bf16x2(g[4], g[5]); o.w = pack_bf16x2(g[6], g[7]);
        *reinterpret_cast<uint4*>(c + j) = o;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col + j < p.N) c[j] = __float2bfloat16(v[j] * gelu_tanh_grad(__bfloat162float(h[j])));
    }
  } else if constexpr (EPI == EPI_LSE) {
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (full || col + j < p.N) cm = fmaxf(cm, v[j]);
    if (cm > -INFINITY) {
      float nm = fmaxf(st.m, cm);
      float acc = 0.0f;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (full || col + j < p.N) acc += __expf(v[j] - nm);
      st.s = st.s * __expf(st.m - nm) + acc;
      st.m = nm;
    }
    int tj = st.tgt - (p.col0 + col);
    if (tj >= 0 && tj < 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j == tj) st.tl = v[j];
    }
  } else if constexpr (EPI == EPI_DZ) {
    bf16* c = reinterpret_cast<bf16*>(p.C) + (size_t)row * p.ldc + col;
    const float l = st.m;   // lse of this row
    const int tj = st.tgt - (p.col0 + col);
    float g[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) g[j] = (__expf(v[j] - l) - (j == tj ? 1.0f : 0.0f)) * p.scale;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 o;
        o.x = pack_bf16x2(g[j], g[j + 1]); o.y = pack_bf16x2(g[j + 2], g[j + 3]);
        o.z = pack_bf16x2(g[j + 4], g[j + 5]); o.w = pack_bf16x2(g[j + 6], g[j + 7]);
        *reinterpret_cast<uint4*>(c + j) = o;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col + j < p.N) c[j] = __float2bfloat16(g[j]);
    }
  }
}

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmDev p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_smem;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
  // barriers: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
  auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + 2 + s); };
  const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(acc_full_bar(s), 1);
      mbar_init(acc_empty_bar(s), 4);
    }
    mbar_init(drain_bar, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_smem), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const int m0 = (t % p.tiles_m) * BM;
        const int n0 = (t / p.tiles_m) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          const int k0 = kb * BK;
          if constexpr (!A_MN) {
            tma_load_2d(sa, &tmA, k0, m0, full_bar(stage));
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d(sa + i * 8192, &tmA, m0 + 64 * i, k0, full_bar(stage));
          }
          if constexpr (!B_MN) {
            tma_load_2d(sb, &tmB, k0, n0, full_bar(stage));
          } else {
#pragma unroll
            for (int i = 0; i < BN / 64; ++i) tma_load_2d(sb + i * 8192, &tmB, n0 + 64 * i, k0, full_bar(stage));
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(p.err, DEV_TIMEOUT_PRODUCER);
        abort_flag = 1;
        // let copies already in flight land before the CTA (and its shared memory) goes away
        int s = stage;
        uint32_t ph = phase;
        for (int i = 0; i < STAGES && i < issued; ++i) {
          if (--s < 0) { s = STAGES - 1; ph ^= 1u; }
          int never = 0;
          mbar_wait(full_bar(s), ph, &never, 20000000ull);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(acc_empty_bar(as), aphase ^ 1u, abortp)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            // K-major: 16 k-elements = 32 bytes along the swizzled row; 8-row groups 1024 B apart.
            // MN-major: 16 k = two groups of 8 k-rows (1024 B each); 64-element MN chunks 8192 B apart.
            const uint64_t ad = A_MN ? make_smem_desc(sa + k * 2048, 8192, 1024) : make_smem_desc(sa + k * 32, 16, 1024);
            const uint64_t bd = B_MN ? make_smem_desc(sb + k * 2048, 8192, 1024) : make_smem_desc(sb + k * 32, 16, 1024);
            umma_bf16(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));   // slab reusable once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(acc_full_bar(as));
      }
      if (!ok) {
        atomicExch(p.err, DEV_TIMEOUT_MMA);
        abort_flag = 1;
      }
      // all issued MMAs must have retired before TMEM is released
      umma_commit(drain_bar);
      int never = 0;
      mbar_wait(drain_bar, 0, &never);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                  // TMEM lane quarter this warp may access
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
      const int m_blk = t % p.tiles_m;
      const int n_blk = t / p.tiles_m;
      const int as = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      if (!mbar_wait(acc_full_bar(as), aphase, abortp)) { ok = false; break; }
      tc_fence_after();
      const int row = m_blk * BM + q * 32 + lane;
      const bool row_ok = row < p.M;
      RowState st;
      st.m = -INFINITY; st.s = 0.0f; st.tl = 0.0f; st.tgt = -1;
      if constexpr (EPI == EPI_LSE || EPI == EPI_DZ) {
        if (row_ok) {
          st.tgt = __ldg(p.targets + row);
          if constexpr (EPI == EPI_DZ) st.m = __ldg(p.lse + row);
        }
      }
      const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        const int col = n_blk * BN + c * 32;
        if (col >= p.N) break;               // uniform across the warp
        uint32_t r[32];
        tmem_ld_32x32(t_addr + (uint32_t)(c * 32), r);
        tmem_ld_wait();
        if (row_ok) epilogue_chunk<EPI>(p, row, col, r, st);
      }
      if constexpr (EPI == EPI_LSE) {
        if (row_ok) {
          const size_t pi = (size_t)row * p.part_ld + (p.col0 / BN + n_blk);
          p.part_max[pi] = st.m;
          p.part_sum[pi] = st.s;
          const int tt = st.tgt - p.col0 - n_blk * BN;
          if (tt >= 0 && tt < BN && tt + n_blk * BN < p.N) p.tgt_logit[row] = st.tl;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty_bar(as));
    }
    if (!ok && lane == 0) {
      atomicExch(p.err, DEV_TIMEOUT_EPILOGUE);
      abort_flag = 1;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;
static std::once_flag g_once;
static cudaError_t g_init_err = cudaSuccess;

typedef void (*KernelFn)(const CUtensorMap, const CUtensorMap, const GemmDev);

template <bool A_MN, bool B_MN>
static KernelFn pick_epi(int epi) {
  switch (epi) {
    case EPI_BF16: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16>;
    case EPI_BF16_GELU: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16_GELU>;
    case EPI_F32_RESID: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_F32_RESID>;
    case EPI_BF16_DGELU: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16_DGELU>;
    case EPI_F32: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_F32>;
    case EPI_LSE: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_LSE>;
    case EPI_DZ: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_DZ>;
  }
  return nullptr;
}

// Only the operand layouts the training step uses are instantiated:
//   forward (K/K): every epilogue but the wgrad-only ones; dgrad (K/MN): bf16, dgelu, f32;
//   wgrad (MN/MN): f32.
static KernelFn pick_kernel(int a_mn, int b_mn, int epi) {
  if (!a_mn && !b_mn) return pick_epi<false, false>(epi);
  if (!a_mn && b_mn) {
    switch (epi) {
      case EPI_BF16: return gemm_tcgen05_kernel<false, true, EPI_BF16>;
      case EPI_BF16_DGELU: return gemm_tcgen05_kernel<false, true, EPI_BF16_DGELU>;
      case EPI_F32: return gemm_tcgen05_kernel<false, true, EPI_F32>;
    }
    return nullptr;
  }
  if (a_mn && b_mn && epi == EPI_F32) return gemm_tcgen05_kernel<true, true, EPI_F32>;
  return nullptr;
}

cudaError_t gemm_init() {
  std::call_once(g_once, []() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
      g_init_err = (e != cudaSuccess) ? e : cudaErrorNotSupported;
      return;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    for (int a = 0; a < 2; ++a)
      for (int b = 0; b < 2; ++b)
        for (int epi = 0; epi < EPI_COUNT; ++epi) {
          KernelFn k = pick_kernel(a, b, epi);
          if (!k) continue;
          e = cudaFuncSetAttribute(reinterpret_cast<const void*>(k), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   SMEM_BYTES);
          if (e != cudaSuccess) { g_init_err = e; return; }
        }
  });
  return g_init_err;
}

// rows = extent of the operand's own index (M or N), kdim = contraction extent, box_rows = tile rows.
static bool encode_operand(CUtensorMap* tm, const GemmOperand& op, int rows, int kdim, int box_rows) {
  cuuint64_t dims[2], strides[1];
  cuuint32_t box[2], estr[2] = {1, 1};
  if (!op.mn_major) {            // memory [rows, kdim], k contiguous
    dims[0] = (cuuint64_t)kdim; dims[1] = (cuuint64_t)rows;
    box[0] = BK; box[1] = (cuuint32_t)box_rows;
  } else {                       // memory [kdim, rows], rows contiguous
    dims[0] = (cuuint64_t)rows; dims[1] = (cuuint64_t)kdim;
    box[0] = 64; box[1] = BK;
  }
  strides[0] = (cuuint64_t)op.ld * 2;
  CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(op.ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

cudaError_t gemm_launch(const GemmArgs& a, unsigned* err_word, int num_sms, cudaStream_t stream) {
  cudaError_t e = gemm_init();
  if (e != cudaSuccess) return e;
  if (a.M <= 0 || a.N <= 0 || a.K <= 0 || !a.A.ptr || !a.B.ptr || !err_word) return cudaErrorInvalidValue;
  if ((a.A.ld % 8) || (a.B.ld % 8) || ((uintptr_t)a.A.ptr % 16) || ((uintptr_t)a.B.ptr % 16)) return cudaErrorInvalidValue;
  KernelFn kern = pick_kernel(a.A.mn_major, a.B.mn_major, a.epilogue);
  if (!kern) return cudaErrorInvalidValue;
  const bool out_f32 = (a.epilogue == EPI_F32 || a.epilogue == EPI_F32_RESID);
  if (a.epilogue != EPI_LSE) {
    if (!a.C || (a.ldc % (out_f32 ? 4 : 8)) || ((uintptr_t)a.C % 16)) return cudaErrorInvalidValue;
  }
  if (a.epilogue == EPI_BF16_GELU && (!a.C2 || ((uintptr_t)a.C2 % 16))) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_F32_RESID && (!a.resid || ((uintptr_t)a.resid % 16))) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_BF16_DGELU && (!a.aux || a.aux_rows <= 0 || (a.ld_aux % 8) || ((uintptr_t)a.aux % 16)))
    return cudaErrorInvalidValue;
  if (a.bias && ((uintptr_t)a.bias % 16)) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_LSE && (!a.targets || !a.part_max || !a.part_sum || !a.tgt_logit || (a.col0 % BN)))
    return cudaErrorInvalidValue;
  if (a.epilogue == EPI_DZ && (!a.targets || !a.lse)) return cudaErrorInvalidValue;

  CUtensorMap tmA, tmB;
  if (!encode_operand(&tmA, a.A, a.M, a.K, BM)) return cudaErrorInvalidValue;
  if (!encode_operand(&tmB, a.B, a.N, a.K, BN)) return cudaErrorInvalidValue;

  GemmDev p;
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.tiles_m = (a.M + BM - 1) / BM;
  p.tiles_n = (a.N + BN - 1) / BN;
  p.C = a.C; p.ldc = a.ldc; p.C2 = a.C2; p.bias = a.bias; p.resid = a.resid;
  p.aux = reinterpret_cast<const bf16*>(a.aux); p.ld_aux = a.ld_aux; p.aux_rows = a.aux_rows > 0 ? a.aux_rows : 1;
  p.accumulate = a.accumulate;
  p.targets = a.targets; p.part_max = a.part_max; p.part_sum = a.part_sum; p.part_ld = a.part_ld;
  p.tgt_logit = a.tgt_logit; p.lse = a.lse; p.scale = a.scale; p.col0 = a.col0;
  p.err = err_word;
  const long long tiles = (long long)p.tiles_m * p.tiles_n;
  const int grid = (int)(tiles < num_sms ? tiles : num_sms);
  kern<<<grid, GEMM_THREADS, SMEM_BYTES, stream>>>(tmA, tmB, p);
  return cudaGetLastError();
}

}  // namespace il
