// tcgen05 GEMM for sm_100a: C[M,N] = A[M,K] * B[N,K]^T, bf16 operands, fp32 accumulation in TMEM.
//
// Persistent kernel of CTA pairs (clusters of two, cta_group::2): a pair owns a 256 x 256 output tile and
// walks a static tile list.  Each CTA stages its own 128 rows of A and its own 128 of the 256 rows of B
// (32 KB per 64-wide k-slab instead of the 48 KB a lone CTA needs for 128 x 256), the leader issues one
// tcgen05.mma.cta_group::2 (M256 N256 K16) that reads both CTAs' shared memory and accumulates rows 0-127
// in its own TMEM and rows 128-255 in the peer's.  Warp roles in each CTA:
//   warp 0    : TMA producer — one thread streams the slabs into a ring of 6 stages (256 x 256 tiles) or 4 (256 x 512), 128-byte swizzle; the byte
//               counts of both CTAs are credited to the leader's "full" mbarrier.
//   warp 1    : allocates 512 TMEM columns (two 128 x 256 fp32 accumulators per CTA); in the leader one thread
//               issues the MMAs and commits (multicast to both CTAs) to the slab's "empty" barriers and,
//               per tile, to the accumulator's "full" barriers.
//   warps 2-9 : epilogue — tcgen05.ld this CTA's half of the accumulator (32 lanes x 32 columns per load, two
//               warps per TMEM lane quarter, one per 128-column half), row-wise math in that layout, then a
//               transpose through shared memory so that every global load and store of the fused epilogue is
//               coalesced; finally the accumulator is released on the leader's barrier.  The second
//               accumulator lets the next tile's main loop overlap this epilogue.
// Operands may be K-major or MN-major in global memory (forward: K/K, dgrad: K/MN, wgrad: MN/MN); the
// major-ness goes into the TMA box shape, the shared-memory descriptor and the instruction descriptor.
// Ragged M/N/K edges rely on TMA zero fill for loads and on bounds checks in the epilogue.
// Every CTA issues its own TMA loads (none is shared across a cluster).  Every wait is bounded; on expiry the CTA sets the error word, and
// both CTAs meet at a cluster barrier before they return.
#include <mutex>

#include "common.cuh"
#include "gemm.h"

namespace il {

constexpr int BM = 128;                          // rows of A (and of the accumulator) held by one CTA
constexpr int TILE_M = 2 * BM;                   // rows of the output tile of a CTA pair
constexpr int BN = 256;                          // columns of the output tile; each CTA stages half of B
constexpr int BK = 64;
constexpr int A_BYTES = BM * BK * 2;             // 16 KB
constexpr int B_BYTES = (BN / 2) * BK * 2;       // 16 KB
constexpr int TMEM_COLS = 2 * BN;                // 512 columns: two accumulators
// NT = accumulators (256-column blocks) per tile.  NT 1: a tile is 256 x 256 and the two accumulators alternate
// between consecutive tiles, so a tile's epilogue hides behind the next tile's main loop.  NT 2: a tile is
// 256 x 512, both accumulators belong to it and every A slab feeds two MMAs: a CTA takes 48 KB instead of
// 64 KB from L2 per 2 x (128 x 256 x 64) products.  One SM's L2 port delivers a 32 KB slab in about the time the
// tensor pipe needs for it, so with NT 1 the two run neck and neck and stall each other; NT 2 leaves the loads
// 25 % slack at the price of an epilogue that overlaps only the start of the next tile.
template <int NT> struct TileCfg {
  static constexpr int STAGES = (NT == 1) ? 6 : 4;
  static constexpr int STAGE_BYTES = A_BYTES + NT * B_BYTES;   // 32 / 48 KB per CTA and stage
};
constexpr int EPI_WARPS = 8;
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;   // producer warp, MMA warp, epilogue warps
constexpr int BAR_BYTES = 256;
constexpr int STG_LD = 32;                       // floats per row of an epilogue warp's 32 x 32 staging tile (16-byte slots XOR-swizzled by row)
constexpr int STG_BYTES = EPI_WARPS * 32 * STG_LD * 4;
template <int NT> constexpr int smem_bytes() {
  return TileCfg<NT>::STAGES * TileCfg<NT>::STAGE_BYTES + 1024 /*alignment slack*/ + BAR_BYTES + STG_BYTES;
}

struct GemmDev {
  int M, N, K;
  int tiles_m, tiles_n;
  int group_m;                   // row blocks per group of the tile order
  int split_k, kb_per_split;     // work unit = (tile, k-range); split_k > 1 adds into C with red.add
  void* C;
  int ldc;
  void* C2;
  const float* bias;
  const float* resid;
  const bf16* aux;
  int ld_aux, aux_rows;
  float* colsum;                 // EPI_BF16_DGELU: += column sums of the output over rows < aux_rows (or NULL)
  int accumulate;
  const int* targets;
  float* part_max;
  float* part_sum;
  int part_ld;
  float* tgt_logit;
  const float* lse;
  float scale;
  int col0;
  const float* rowscale;
  int store_exp;
  unsigned* err;
};

// Tile order: groups of group_m row blocks are swept across all column blocks before the next group starts, so
// that the pairs running at the same time share a small set of A rows and the whole of B in L2.  B is read from
// DRAM once per group, A once in total: the host makes the group as tall as the matrix when all of A fits in
// L2 beside the streams passing through it (the heads' [Ntok, V, d] projection: W would otherwise be read four
// times), and 8 row blocks otherwise.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int group_m, int& m_blk, int& n_blk) {
  const int per_group = group_m * tiles_n;
  const int g = t / per_group;
  const int within = t - g * per_group;
  const int gm = min(group_m, tiles_m - g * group_m);
  m_blk = g * group_m + within % gm;
  n_blk = within / gm;
}

struct RowState {   // per-thread state carried across the 32-column chunks of one tile row (EPI_LSE)
  float m, s, tl;
  int tgt;
};

// Row-wise part of the epilogue, in the accumulator's own layout (thread = one row, v = 32 consecutive
// columns starting at `col`): the softmax statistics (EPI_LSE; the logits themselves are stored only when
// C is given) and dZ (EPI_DZ, in place).
template <int EPI>
__device__ __forceinline__ void epilogue_rowwise(const GemmDev& p, int col, float (&v)[32], RowState& st) {
  const bool full = (col + 32 <= p.N);
  if constexpr (EPI == EPI_LSE) {
    constexpr float L2E = 1.4426950408889634f;
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (full || col + j < p.N) cm = fmaxf(cm, v[j]);
    int tj = st.tgt - (p.col0 + col);
    if (tj >= 0 && tj < 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j == tj) st.tl = v[j];
    }
    if (p.store_exp) {
      // What is kept for the backward is E = exp(logit) (softmax up to a per-row factor), so each element needs
      // one exponential only: while the running maximum stays where exp() of it is far from the fp32 range, the
      // chunk's share of the softmax sum is the sum of the stored values times one factor per chunk.
      const float nm = fmaxf(st.m, cm);
      const bool direct = fabsf(nm) < 64.0f;      // nm = -inf (nothing valid yet) takes the general branch
      float acc = 0.0f;
      if (direct) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          v[j] = ex2_fast(v[j] * L2E);
          if (full || col + j < p.N) acc += v[j];
        }
        acc *= ex2_fast(-nm * L2E);
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if (full || col + j < p.N) acc += ex2_fast((v[j] - nm) * L2E);
          v[j] = ex2_fast(v[j] * L2E);
        }
      }
      if (cm > -INFINITY) {
        st.s = st.s * ex2_fast((st.m - nm) * L2E) + acc;
        st.m = nm;
      }
    } else if (cm > -INFINITY) {
      const float nm = fmaxf(st.m, cm);
      float acc = 0.0f;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (full || col + j < p.N) acc += ex2_fast((v[j] - nm) * L2E);
      st.s = st.s * ex2_fast((st.m - nm) * L2E) + acc;
      st.m = nm;
    }
  } else if constexpr (EPI == EPI_DZ) {
    const float l = st.m;   // lse of this row
    const int tj = st.tgt - (p.col0 + col);
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = (ex2_fast((v[j] - l) * 1.4426950408889634f) - (j == tj ? 1.0f : 0.0f)) * p.scale;
  }
}

// Element-wise part of the epilogue, after the 32 x 32 chunk has been transposed through shared memory: a
// lane now holds 4 consecutive columns (gcol..gcol+3) of row grow, 8 lanes cover 128 contiguous bytes of
// fp32 output (64 of bf16), so every global access is coalesced.  The loads of the second operand
// (residual, saved pre-activation, or C itself when accumulating) are split from the stores so that all of
// a chunk's loads are in flight before the first store (C may alias the residual).
template <int EPI>
__device__ __forceinline__ float4 epilogue_load4(const GemmDev& p, int grow, int arow, int gcol) {
  float4 e = make_float4(0.f, 0.f, 0.f, 0.f);
  const bool vec = (gcol + 4 <= p.N);
  if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
    const float* add = nullptr;
    if constexpr (EPI == EPI_F32_RESID) add = p.resid + (size_t)grow * p.ldc + gcol;
    else if (p.accumulate) add = reinterpret_cast<const float*>(p.C) + (size_t)grow * p.ldc + gcol;
    if (add) {
      if (vec) {
        e = *reinterpret_cast<const float4*>(add);
      } else {
        e.x = add[0];
        if (gcol + 1 < p.N) e.y = add[1];
        if (gcol + 2 < p.N) e.z = add[2];
      }
    }
  } else if constexpr (EPI == EPI_BF16_DGELU) {
    const bf16* h = p.aux + (size_t)arow * p.ld_aux + gcol;   // arow = grow % aux_rows
    if (vec) {
      const uint2 hv = *reinterpret_cast<const uint2*>(h);
      const float2 h0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hv.x));
      const float2 h1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hv.y));
      e = make_float4(h0.x, h0.y, h1.x, h1.y);
    } else {
      e.x = __bfloat162float(h[0]);
      if (gcol + 1 < p.N) e.y = __bfloat162float(h[1]);
      if (gcol + 2 < p.N) e.z = __bfloat162float(h[2]);
    }
  }
  return e;
}

template <int EPI>
__device__ __forceinline__ void epilogue_store4(const GemmDev& p, int grow, int gcol, float4 a, float4 e) {
  const bool vec = (gcol + 4 <= p.N);
  float v[4] = {a.x, a.y, a.z, a.w};
  if constexpr (EPI == EPI_BF16 || EPI == EPI_BF16_GELU || EPI == EPI_F32_RESID) {
    if (p.bias) {
      if (vec) {
        const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + gcol));
        v[0] += b.x; v[1] += b.y; v[2] += b.z; v[3] += b.w;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (gcol + j < p.N) v[j] += __ldg(p.bias + gcol + j);
      }
    }
  }
  if constexpr (EPI == EPI_BF16 || EPI == EPI_BF16_GELU || EPI == EPI_DZ || EPI == EPI_BF16_DGELU || EPI == EPI_LSE) {
    bf16* c = reinterpret_cast<bf16*>(p.C) + (size_t)grow * p.ldc + gcol;
    if constexpr (EPI == EPI_BF16_DGELU) {
      v[0] *= e.x; v[1] *= e.y; v[2] *= e.z; v[3] *= e.w;
      if (p.colsum && grow < p.aux_rows) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (gcol + j < p.N) atomicAdd(p.colsum + gcol + j, v[j]);
      }
    }
    float y[4] = {0.f, 0.f, 0.f, 0.f};
    if constexpr (EPI == EPI_BF16_GELU) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float d;
        gelu_tanh_both(v[j], y[j], d);
        v[j] = d;                                   // C receives gelu'(pre), C2 gelu(pre)
      }
    }
    if (vec) {
      uint2 o;
      o.x = pack_bf16x2(v[0], v[1]);
      o.y = pack_bf16x2(v[2], v[3]);
      *reinterpret_cast<uint2*>(c) = o;
      if constexpr (EPI == EPI_BF16_GELU) {
        uint2 g;
        g.x = pack_bf16x2(y[0], y[1]);
        g.y = pack_bf16x2(y[2], y[3]);
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(p.C2) + (size_t)grow * p.ldc + gcol) = g;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (gcol + j < p.N) {
          c[j] = __float2bfloat16(v[j]);
          if constexpr (EPI == EPI_BF16_GELU)
            (reinterpret_cast<bf16*>(p.C2) + (size_t)grow * p.ldc + gcol)[j] = __float2bfloat16(y[j]);
        }
    }
  } else if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
    float* c = reinterpret_cast<float*>(p.C) + (size_t)grow * p.ldc + gcol;
    v[0] += e.x; v[1] += e.y; v[2] += e.z; v[3] += e.w;
    if (EPI == EPI_F32 && p.split_k > 1) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (gcol + j < p.N) atomicAdd(c + j, v[j]);
    } else if (vec) {
      *reinterpret_cast<float4*>(c) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (gcol + j < p.N) c[j] = v[j];
    }
  }
}

template <bool A_MN, bool B_MN, int EPI, int NT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmDev p) {
  constexpr int STAGES = TileCfg<NT>::STAGES;
  constexpr int STAGE_BYTES = TileCfg<NT>::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_smem;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
  // barriers: full[STAGES] (leader's are used), empty[STAGES], acc_full[2], acc_empty[2] (leader's), drain
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
  auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + 2 + s); };
  const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();           // 0 = leader of the pair (issues the MMAs)
  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n * p.split_k;    // work units: unit u = (tile u / split_k, k-range u % split_k)
  const int num_kb_all = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(acc_full_bar(s), 1);
      mbar_init(acc_empty_bar(s), 2 * EPI_WARPS);      // the epilogue warps of both CTAs of the pair
    }
    mbar_init(drain_bar, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_smem), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();       // the peer's barriers are initialised before anything is signalled remotely
  tc_fence_after();
  grid_dep_sync();          // tensor memory is held, nothing in global memory has been touched yet
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = pair; t < num_tiles && ok; t += num_pairs) {
        int m_blk, n_blk;
        tile_coords(t / p.split_k, p.tiles_m, p.tiles_n, p.group_m, m_blk, n_blk);
        const int m0 = m_blk * TILE_M + (int)rank * BM;       // this CTA's 128 rows of A
        const int n0 = n_blk * (NT * BN) + (int)rank * (BN / 2);   // this CTA's 128 rows of the (first) 256-row block of B
        const int kb0 = (t % p.split_k) * p.kb_per_split;
        const int kb1 = min(num_kb_all, kb0 + p.kb_per_split);
        // a wide tile whose second 256-column block lies wholly past N carries that block neither through shared
        // memory nor through the tensor pipe
        const int nh = (NT == 2 && n_blk * (NT * BN) + BN >= p.N) ? 1 : NT;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          // both CTAs' bytes are credited to the leader's barrier, which expects the pair's total
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * (A_BYTES + nh * B_BYTES));
          const uint32_t fb = mapa_cluster(full_bar(stage), 0);
          const int k0 = kb * BK;
          if constexpr (!A_MN) {
            tma_load_2d_pair(sa, &tmA, k0, m0, fb);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(sa + i * 8192, &tmA, m0 + 64 * i, k0, fb);
          }
#pragma unroll
          for (int h = 0; h < NT; ++h) {          // block h of the tile's columns (past N: zero fill)
            if (h >= nh) break;
            if constexpr (!B_MN) {
              tma_load_2d_pair(sb + h * B_BYTES, &tmB, k0, n0 + h * BN, fb);
            } else {
#pragma unroll
              for (int i = 0; i < BN / 128; ++i) tma_load_2d_pair(sb + h * B_BYTES + i * 8192, &tmB, n0 + h * BN + 64 * i, k0, fb);
            }
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(p.err, DEV_TIMEOUT_PRODUCER);
        abort_flag = 1;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(TILE_M, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int t = pair; t < num_tiles && ok; t += num_pairs, ++it) {
        // NT 1: the tile uses accumulator it % 2.  NT 2: it uses both; block 0 is waited for first and handed to
        // the epilogue as soon as its last MMAs are issued, block 1 is only waited for before its first MMA, so
        // the first products of a tile overlap the draining of the previous tile's second block.
        const int as = (NT == 1) ? (it & 1) : 0;
        const uint32_t aphase = (NT == 1) ? ((uint32_t)(it >> 1) & 1u) : ((uint32_t)it & 1u);
        if (!mbar_wait(acc_empty_bar(as), aphase ^ 1u, abortp)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        const int kb0 = (t % p.split_k) * p.kb_per_split;
        const int kb1 = min(num_kb_all, kb0 + p.kb_per_split);
        int m_blk_, n_tile_;
        tile_coords(t / p.split_k, p.tiles_m, p.tiles_n, p.group_m, m_blk_, n_tile_);
        const bool skip_h1 = (NT == 2 && n_tile_ * (NT * BN) + BN >= p.N);   // second block wholly past N: not loaded
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int h = 0; h < NT; ++h) {
            if (NT == 2 && h == 1 && kb == kb0) {
              if (!mbar_wait(acc_empty_bar(1), aphase ^ 1u, abortp)) { ok = false; break; }
              tc_fence_after();
            }
            if (h == 1 && skip_h1) continue;      // the accumulator is still handed over below; nothing reads it
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) {
              // K-major: 16 k-elements = 32 bytes along the swizzled row; 8-row groups 1024 B apart.
              // MN-major: 16 k = two groups of 8 k-rows (1024 B each); 64-element MN chunks 8192 B apart.
              const uint32_t sbh = sb + h * B_BYTES;
              const uint64_t ad = A_MN ? make_smem_desc(sa + k * 2048, 8192, 1024) : make_smem_desc(sa + k * 32, 16, 1024);
              const uint64_t bd = B_MN ? make_smem_desc(sbh + k * 2048, 8192, 1024) : make_smem_desc(sbh + k * 32, 16, 1024);
              umma_bf16_pair(d_tmem + (uint32_t)(h * BN), ad, bd, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
            }
            if (NT == 2 && h == 0 && kb == kb1 - 1) umma_commit_pair(acc_full_bar(0), 3);
          }
          if (!ok) break;
          umma_commit_pair(empty_bar(stage), 3);   // slab reusable in both CTAs once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(acc_full_bar(NT == 1 ? as : 1), 3);
      }
      if (!ok) {
        atomicExch(p.err, DEV_TIMEOUT_MMA);
        abort_flag = 1;
      }
      // all issued MMAs must have retired before TMEM is released
      umma_commit_pair(drain_bar, 1);
      int never = 0;
      mbar_wait(drain_bar, 0, &never);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    // Two warps share each TMEM lane quarter (a warp may only read lanes 32*(warp%4)..+31): the first
    // takes columns 0-127 of the tile, the second columns 128-255.
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    float* stg = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)) + STAGES * STAGE_BYTES + BAR_BYTES) +
                 (warp - 2) * (32 * STG_LD);
    int it = 0;
    bool ok = true;
    for (int t = pair; t < num_tiles && ok; t += num_pairs, ++it) {
      int m_blk, n_tile;
      tile_coords(t / p.split_k, p.tiles_m, p.tiles_n, p.group_m, m_blk, n_tile);
      for (int h = 0; h < NT && ok; ++h) {           // the tile's 256-column blocks, one accumulator each
      const int n_blk = n_tile * NT + h;
      const int as = (NT == 1) ? (it & 1) : h;
      const uint32_t aphase = (NT == 1) ? ((uint32_t)(it >> 1) & 1u) : ((uint32_t)it & 1u);
      const int row0 = m_blk * TILE_M + (int)rank * BM + q * 32;     // first row of this warp's 32
      const int col_base = n_blk * BN + half * (BN / 2);
      const int lrow = lane >> 3;                  // row within a group of 4 after the transpose
      const int gcol_off = 4 * (lane & 7);
      const int arow0 = (EPI == EPI_BF16_DGELU) ? row0 % p.aux_rows : 0;
      // While the main loop of this tile is still running, fetch the epilogue's second operand in the
      // coalesced (transposed) layout: the first chunk of the saved gelu' (bf16) or of the fp32 residual /
      // accumulated C; the later chunks are fetched one chunk ahead.
      uint2 cur_h[8], nxt_h[8];      // saved gelu' of the chunk being processed and of the next one
      float4 cur_f[8], nxt_f[8];     // fp32 second operand of the chunk being processed and of the next one
      auto load_f32_chunk = [&](int c, float4 (&dst)[8]) {
        const int gcol = col_base + c * 32 + gcol_off;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int grow = row0 + 4 * i + lrow;
          dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (grow < p.M && gcol < p.N) dst[i] = epilogue_load4<EPI>(p, grow, 0, gcol);
        }
      };
      auto load_h_chunk = [&](int c, uint2 (&dst)[8]) {
        const int gcol = col_base + c * 32 + gcol_off;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int grow = row0 + 4 * i + lrow;
          int arow = arow0 + 4 * i + lrow;          // grow % aux_rows without a division
          while (arow >= p.aux_rows) arow -= p.aux_rows;   // more than once only for fewer than 32 saved rows
          dst[i] = make_uint2(0u, 0u);
          if (grow < p.M && gcol + 4 <= p.N)
            dst[i] = *reinterpret_cast<const uint2*>(p.aux + (size_t)arow * p.ld_aux + gcol);
        }
      };
      if constexpr (EPI == EPI_BF16_DGELU) {
        load_h_chunk(0, cur_h);
      } else if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
        load_f32_chunk(0, cur_f);
      }
      {   // one lane polls the barrier (keeps 255 pollers off the shared-memory pipe the main loop lives on)
        int got = 1;
        if (lane == 0) got = mbar_wait(acc_full_bar(as), aphase, abortp) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        if (!got) { ok = false; break; }
      }
      tc_fence_after();
      const int row = row0 + lane;
      const bool row_ok = row < p.M;
      RowState st;
      st.m = -INFINITY; st.s = 0.0f; st.tl = 0.0f; st.tgt = -1;
      if constexpr (EPI == EPI_LSE || EPI == EPI_DZ) {
        if (row_ok) {
          st.tgt = __ldg(p.targets + row);
          if constexpr (EPI == EPI_DZ) st.m = __ldg(p.lse + row);
        }
      }
      float rs = 1.0f;                           // EPI_F32: factor of this thread's row
      if constexpr (EPI == EPI_F32) {
        if (p.rowscale && row_ok) rs = __ldg(p.rowscale + row);
      }
      const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN + half * (BN / 2));
      // One 32-column chunk of this warp's 32 rows; returns false once the chunk lies past the last column.
      auto do_chunk = [&](const int c) -> bool {
        const int col = col_base + c * 32;
        if (col >= p.N) return false;        // uniform across the warp
        uint32_t r[32];
        tmem_ld_32x32(t_addr + (uint32_t)(c * 32), r);
        const int gcol = col + gcol_off;
        // fast path: the whole 32 x 32 chunk is inside the matrix (uniform across the warp), so nothing below
        // is predicated and the 32 element chains of a lane are independent straight-line code
        const bool interior = (row0 + 32 <= p.M) && (col + 32 <= p.N);
        // the chunk's bias values are requested before the accumulator columns are waited for
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (EPI == EPI_BF16 || EPI == EPI_BF16_GELU || EPI == EPI_F32_RESID)
          if (interior && p.bias) b4 = __ldg(reinterpret_cast<const float4*>(p.bias + gcol));
        float4 extra[8];
        if constexpr (EPI == EPI_BF16_DGELU) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float2 h0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&cur_h[i].x));
            const float2 h1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&cur_h[i].y));
            extra[i] = make_float4(h0.x, h0.y, h1.x, h1.y);
          }
          // the next chunk's values travel while this one is processed
          if (c + 1 < BN / 64 && col + 32 < p.N) load_h_chunk(c + 1, nxt_h);
          if (!interior && gcol < p.N && gcol + 4 > p.N) {    // ragged last columns: element-wise reload
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int grow = row0 + 4 * i + lrow;
              int arow = arow0 + 4 * i + lrow;
              while (arow >= p.aux_rows) arow -= p.aux_rows;   // more than once only for fewer than 32 saved rows
              if (grow < p.M) extra[i] = epilogue_load4<EPI>(p, grow, arow, gcol);
            }
          }
        } else if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
#pragma unroll
          for (int i = 0; i < 8; ++i) extra[i] = cur_f[i];
          if (c + 1 < BN / 64 && col + 32 < p.N) load_f32_chunk(c + 1, nxt_f);
        }
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if constexpr (EPI == EPI_LSE || EPI == EPI_DZ) epilogue_rowwise<EPI>(p, col, v, st);
        if constexpr (EPI == EPI_F32) {
          if (p.rowscale) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] *= rs;
          }
        }
        if (EPI != EPI_LSE || p.C != nullptr) {      // EPI_LSE keeps the logits (bf16) only when asked to
          // transpose through shared memory: lane (= row) writes its 32 columns, then lane l reads 4
          // columns of row 4i + l/8
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<float4*>(stg + lane * STG_LD + 4 * (j ^ (lane & 7))) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          __syncwarp();
          float4 a[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)          // row 4i + lrow, slot (lane & 7) ^ (row & 7); row & 7 = (4i + lrow) & 7
            a[i] = *reinterpret_cast<const float4*>(stg + (4 * i + lrow) * STG_LD + 4 * ((lane & 7) ^ ((4 * i + lrow) & 7)));
          if (interior) {
            if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
              float* cbase = reinterpret_cast<float*>(p.C) + (size_t)(row0 + lrow) * p.ldc + gcol;
              if (EPI == EPI_F32 && p.split_k > 1) {       // partial sums of a k-range: add into the zeroed output
#pragma unroll
                for (int i = 0; i < 8; ++i) red_add_f32x4(cbase + (size_t)(4 * i) * p.ldc, a[i]);
              } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  *reinterpret_cast<float4*>(cbase + (size_t)(4 * i) * p.ldc) =
                      make_float4(a[i].x + b4.x + extra[i].x, a[i].y + b4.y + extra[i].y, a[i].z + b4.z + extra[i].z,
                                  a[i].w + b4.w + extra[i].w);
              }
            } else {
              uint2 o[8], g[8];
              float4 cs = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                float x0 = a[i].x + b4.x, x1 = a[i].y + b4.y, x2 = a[i].z + b4.z, x3 = a[i].w + b4.w;
                if constexpr (EPI == EPI_BF16_DGELU) {
                  x0 *= extra[i].x; x1 *= extra[i].y; x2 *= extra[i].z; x3 *= extra[i].w;
                  if (row0 + 4 * i + lrow < p.aux_rows) { cs.x += x0; cs.y += x1; cs.z += x2; cs.w += x3; }
                }
                if constexpr (EPI == EPI_BF16_GELU) {
                  float y0, y1, y2, y3, d0, d1, d2, d3;
                  gelu_tanh_both(x0, y0, d0); gelu_tanh_both(x1, y1, d1);
                  gelu_tanh_both(x2, y2, d2); gelu_tanh_both(x3, y3, d3);
                  o[i].x = pack_bf16x2(d0, d1);
                  o[i].y = pack_bf16x2(d2, d3);
                  g[i].x = pack_bf16x2(y0, y1);
                  g[i].y = pack_bf16x2(y2, y3);
                } else {
                  o[i].x = pack_bf16x2(x0, x1);
                  o[i].y = pack_bf16x2(x2, x3);
                }
              }
              bf16* cbase = reinterpret_cast<bf16*>(p.C) + (size_t)(row0 + lrow) * p.ldc + gcol;
#pragma unroll
              for (int i = 0; i < 8; ++i) *reinterpret_cast<uint2*>(cbase + (size_t)(4 * i) * p.ldc) = o[i];
              if constexpr (EPI == EPI_BF16_DGELU) {
                if (p.colsum && row0 < p.aux_rows) {     // bias gradient: column sums over the first gradient stream
                  cs.x += __shfl_xor_sync(0xffffffffu, cs.x, 8);  cs.y += __shfl_xor_sync(0xffffffffu, cs.y, 8);
                  cs.z += __shfl_xor_sync(0xffffffffu, cs.z, 8);  cs.w += __shfl_xor_sync(0xffffffffu, cs.w, 8);
                  cs.x += __shfl_xor_sync(0xffffffffu, cs.x, 16); cs.y += __shfl_xor_sync(0xffffffffu, cs.y, 16);
                  cs.z += __shfl_xor_sync(0xffffffffu, cs.z, 16); cs.w += __shfl_xor_sync(0xffffffffu, cs.w, 16);
                  if (lane < 8) red_add_f32x4(p.colsum + gcol, cs);
                }
              }
              if constexpr (EPI == EPI_BF16_GELU) {
                bf16* c2base = reinterpret_cast<bf16*>(p.C2) + (size_t)(row0 + lrow) * p.ldc + gcol;
#pragma unroll
                for (int i = 0; i < 8; ++i) *reinterpret_cast<uint2*>(c2base + (size_t)(4 * i) * p.ldc) = g[i];
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int rr = 4 * i + lrow;
              if (row0 + rr < p.M && gcol < p.N) epilogue_store4<EPI>(p, row0 + rr, gcol, a[i], extra[i]);
            }
          }
          __syncwarp();
        }
        if constexpr (EPI == EPI_BF16_DGELU) {
#pragma unroll
          for (int i = 0; i < 8; ++i) cur_h[i] = nxt_h[i];
        }
        if constexpr (EPI == EPI_F32_RESID || EPI == EPI_F32) {
#pragma unroll
          for (int i = 0; i < 8; ++i) cur_f[i] = nxt_f[i];
        }
        return true;
      };
      // The chunk body is a loop, not four copies: it is the largest code in the kernel and has to stay in the
      // instruction cache beside the main loop's (second operands are handed from chunk to chunk in registers).
#pragma unroll 1
      for (int c = 0; c < BN / 64; ++c)
        if (!do_chunk(c)) break;
      if constexpr (EPI == EPI_LSE) {
        if (row_ok && n_blk * BN + half * (BN / 2) < p.N) {
          const size_t pi = (size_t)row * p.part_ld + (p.col0 / (BN / 2) + n_blk * 2 + half);
          p.part_max[pi] = st.m;
          p.part_sum[pi] = st.s;
          const int tt = st.tgt - p.col0 - n_blk * BN - half * (BN / 2);
          if (tt >= 0 && tt < BN / 2 && st.tgt - p.col0 < p.N) p.tgt_logit[row] = st.tl;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_cluster(acc_empty_bar(as), 0));
      }
    }
    if (!ok && lane == 0) {
      atomicExch(p.err, DEV_TIMEOUT_EPILOGUE);
      abort_flag = 1;
    }
  }

  // Neither CTA may leave while its peer can still read its shared memory or signal its barriers.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
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

template <bool A_MN, bool B_MN, int NT>
static KernelFn pick_epi(int epi) {
  switch (epi) {
    case EPI_BF16: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16, NT>;
    case EPI_BF16_GELU: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16_GELU, NT>;
    case EPI_F32_RESID: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_F32_RESID, NT>;
    case EPI_BF16_DGELU: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_BF16_DGELU, NT>;
    case EPI_F32: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_F32, NT>;
    case EPI_LSE: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_LSE, NT>;
    case EPI_DZ: return gemm_tcgen05_kernel<A_MN, B_MN, EPI_DZ, NT>;
  }
  return nullptr;
}

// Only the operand layouts the training step uses are instantiated:
//   forward (K/K): every epilogue but the wgrad-only ones; dgrad (K/MN): bf16, dgelu, f32;
//   wgrad (MN/MN): f32.
template <int NT>
static KernelFn pick_kernel_nt(int a_mn, int b_mn, int epi) {
  if (!a_mn && !b_mn) return pick_epi<false, false, NT>(epi);
  if (!a_mn && b_mn) {
    switch (epi) {
      case EPI_BF16: return gemm_tcgen05_kernel<false, true, EPI_BF16, NT>;
      case EPI_BF16_DGELU: return gemm_tcgen05_kernel<false, true, EPI_BF16_DGELU, NT>;
      case EPI_F32: return gemm_tcgen05_kernel<false, true, EPI_F32, NT>;
    }
    return nullptr;
  }
  if (a_mn && b_mn && epi == EPI_F32) return gemm_tcgen05_kernel<true, true, EPI_F32, NT>;
  return nullptr;
}
static KernelFn pick_kernel(int a_mn, int b_mn, int epi, int nt) {
  return nt == 2 ? pick_kernel_nt<2>(a_mn, b_mn, epi) : pick_kernel_nt<1>(a_mn, b_mn, epi);
}

// The driver entry point is looked up once per process; the shared-memory opt-in of the kernels is a per-device
// function attribute and is set once for every device the library is used on (with that device current).
static std::mutex g_attr_mu;
static bool g_attr_done[64] = {};

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
  });
  if (g_init_err != cudaSuccess) return g_init_err;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_attr_mu);
  if (g_attr_done[dev]) return cudaSuccess;
  for (int a = 0; a < 2; ++a)
    for (int b = 0; b < 2; ++b)
      for (int epi = 0; epi < EPI_COUNT; ++epi)
        for (int nt = 1; nt <= 2; ++nt) {
          KernelFn k = pick_kernel(a, b, epi, nt);
          if (!k) continue;
          e = cudaFuncSetAttribute(reinterpret_cast<const void*>(k), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   nt == 2 ? smem_bytes<2>() : smem_bytes<1>());
          if (e != cudaSuccess) return e;
        }
  g_attr_done[dev] = true;
  return cudaSuccess;
}

static bool tma_encode_any(CUtensorMap* tm, CUtensorMapDataType dt, const void* ptr, int rank, const unsigned long long* dims,
                           const unsigned long long* strides_bytes, const unsigned* box) {
  if (gemm_init() != cudaSuccess || rank < 2 || rank > 5) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
  for (int i = 0; i < rank - 1; ++i) st[i] = strides_bytes[i];
  return g_encode(tm, dt, (cuuint32_t)rank, const_cast<void*>(ptr), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tma_encode_bf16(CUtensorMap* tm, const void* ptr, int rank, const unsigned long long* dims,
                     const unsigned long long* strides_bytes, const unsigned* box) {
  return tma_encode_any(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ptr, rank, dims, strides_bytes, box);
}

bool tma_encode_f32(CUtensorMap* tm, const void* ptr, int rank, const unsigned long long* dims,
                    const unsigned long long* strides_bytes, const unsigned* box) {
  return tma_encode_any(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ptr, rank, dims, strides_bytes, box);
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
  // Tile width.  256 x 512 tiles cut the operand bytes per product by a quarter but expose most of the epilogue,
  // so they pay when the main loop of a tile is long (K) and the output is at least one such tile wide.
  int nt = a.tile_blocks;
  if (nt < 1 || nt > 2) nt = (a.N > BN && a.K >= 2048) ? 2 : 1;
  if (a.N <= BN) nt = 1;
  KernelFn kern = pick_kernel(a.A.mn_major, a.B.mn_major, a.epilogue, nt);
  if (!kern) return cudaErrorInvalidValue;
  const bool out_f32 = (a.epilogue == EPI_F32 || a.epilogue == EPI_F32_RESID);
  if (a.epilogue != EPI_LSE || a.C) {
    if (!a.C || (a.ldc % (out_f32 ? 4 : 8)) || ((uintptr_t)a.C % 16)) return cudaErrorInvalidValue;
  }
  if (a.epilogue == EPI_BF16_GELU && (!a.C2 || ((uintptr_t)a.C2 % 16))) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_F32_RESID && (!a.resid || ((uintptr_t)a.resid % 16))) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_BF16_DGELU && (!a.aux || a.aux_rows < 1 || (a.ld_aux % 8) || ((uintptr_t)a.aux % 16)))
    return cudaErrorInvalidValue;
  if (a.bias && ((uintptr_t)a.bias % 16)) return cudaErrorInvalidValue;
  if (a.colsum && (a.epilogue != EPI_BF16_DGELU || ((uintptr_t)a.colsum % 16))) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_LSE && (!a.targets || !a.part_max || !a.part_sum || !a.tgt_logit || (a.col0 % (BN / 2))))
    return cudaErrorInvalidValue;
  if (a.epilogue == EPI_DZ && (!a.targets || !a.lse)) return cudaErrorInvalidValue;
  if (a.rowscale && a.epilogue != EPI_F32) return cudaErrorInvalidValue;
  if (a.store_exp && (a.epilogue != EPI_LSE || !a.C)) return cudaErrorInvalidValue;

  CUtensorMap tmA, tmB;
  if (!encode_operand(&tmA, a.A, a.M, a.K, BM)) return cudaErrorInvalidValue;
  if (!encode_operand(&tmB, a.B, a.N, a.K, BN / 2)) return cudaErrorInvalidValue;

  GemmDev p;
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.tiles_m = (a.M + TILE_M - 1) / TILE_M;
  p.tiles_n = (a.N + nt * BN - 1) / (nt * BN);
  p.group_m = ((long long)a.M * a.K * 2 <= (48ll << 20)) ? p.tiles_m : 8;
  {
    // Split the contraction when the tile count leaves most CTA pairs idle (fp32 outputs only; the caller
    // zeroes C and the partial sums are added with red.global.add).
    const int num_kb = (a.K + BK - 1) / BK;
    int split = a.split_k > 1 ? a.split_k : 1;
    if (a.epilogue != EPI_F32 || a.accumulate) split = 1;
    if (split > num_kb) split = num_kb;
    p.kb_per_split = (num_kb + split - 1) / split;
    p.split_k = (num_kb + p.kb_per_split - 1) / p.kb_per_split;
  }
  p.C = a.C; p.ldc = a.ldc; p.C2 = a.C2; p.bias = a.bias; p.resid = a.resid;
  p.aux = reinterpret_cast<const bf16*>(a.aux); p.ld_aux = a.ld_aux; p.aux_rows = a.aux_rows > 0 ? a.aux_rows : 1;
  p.colsum = a.colsum;
  p.accumulate = a.accumulate;
  p.targets = a.targets; p.part_max = a.part_max; p.part_sum = a.part_sum; p.part_ld = a.part_ld;
  p.tgt_logit = a.tgt_logit; p.lse = a.lse; p.scale = a.scale; p.col0 = a.col0;
  p.rowscale = a.rowscale; p.store_exp = a.store_exp;
  p.err = err_word;
  const long long tiles = (long long)p.tiles_m * p.tiles_n * p.split_k;
  const int pairs = (int)(tiles < num_sms / 2 ? tiles : num_sms / 2);
  const int grid = 2 * pairs;
  launch_dep(kern, dim3(grid), dim3(GEMM_THREADS), nt == 2 ? smem_bytes<2>() : smem_bytes<1>(), stream, tmA, tmB, p);
  return cudaGetLastError();
}

}  // namespace il
