// Causal self-attention forward on the tcgen05 tensor cores (sm_100a).
//
// One CTA owns 128 query rows of one (sequence, head) and sweeps the keys in blocks of 64.  Q, K and V
// tiles come in by TMA from the packed qkv tensor viewed as a 4-D tensor (column within head, head slot,
// position, sequence) so that head selection, the ragged last rows of a sequence and head dimensions
// that are not a multiple of 64 are all handled by the tensor map's bounds (zero fill).  Per key block:
//   S = Q K^T        tcgen05.mma (M128 N64, both operands K-major in shared memory) -> TMEM columns [0, 64)
//   softmax          thread r owns query row r: tcgen05.ld its 64 scores, running max / sum in registers
//                    (no cross-lane reduction), P = exp2(...) rounded to bf16, packed in pairs and stored back
//                    over the first 32 of the score columns (tcgen05.st)
//   O += P V         tcgen05.mma (M128 N=dh, A = P read from TMEM, B = V MN-major), accumulated in TMEM columns
//                    [64, 64+dh).  The reference maximum of a row is raised only when a block exceeds it by a
//                    factor 2^8, so the accumulator is rescaled (tcgen05.ld / st) rarely.
// A CTA runs these phases one after the other; several CTAs are resident per SM (128 threads, 64-144 KB of
// shared memory, 128-256 TMEM columns each), which is what overlaps one CTA's softmax with another's MMAs.
// K and V come through a ring of TMA stages filled two or more sweep steps ahead.
// The T x T score matrix is never stored.  Every wait is bounded.
#include "common.cuh"
#include "kernels.h"
#include "tma.h"

namespace il {

namespace {

constexpr int TQ = 128;     // query rows per CTA
constexpr int TK = 64;      // keys per sweep step
#define IL_LOG2E 1.4426950408889634f

template <int DH>
struct FwdCfg {
  static constexpr int NCH = (DH + 63) / 64;            // 64-column chunks of the head dimension
  static constexpr int Q_BYTES = NCH * TQ * 128;
  static constexpr int KV_BYTES = NCH * TK * 128;
  static constexpr int NST = (DH <= 64) ? 3 : 2;               // K/V ring depth: as deep as keeps three (dh <= 64) or two CTAs per SM
  static constexpr int TCOLS = (64 + DH <= 128) ? 128 : (64 + DH <= 256) ? 256 : 512;   // 64 score columns + the O accumulator
  static constexpr int SMEM = Q_BYTES + NST * 2 * KV_BYTES + 1024 + 128;
};

template <int DH>
__global__ void __launch_bounds__(128) attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                          const __grid_constant__ CUtensorMap tmKV, bf16* __restrict__ o,
                                                          float* __restrict__ lse, int T, int H, float scale, unsigned* err) {
  using C = FwdCfg<DH>;
  constexpr int NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_smem;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base;
  const uint32_t sK0 = sQ + C::Q_BYTES;                       // the K stages, then the V stages
  const uint32_t sV0 = sK0 + NST * C::KV_BYTES;
  const uint32_t bars = sV0 + NST * C::KV_BYTES;
  const uint32_t bar_q = bars, bar_s = bars + 8, bar_o = bars + 16, bar_drain = bars + 24, bar_kv0 = bars + 32;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int qb = gridDim.x - 1 - blockIdx.x;                  // longest sweeps first
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  const int d = H * DH;
  const int row = qb * TQ + tid;                              // query position of this thread
  int nkv = (qb * TQ + TQ + TK - 1) / TK;
  const int nkv_all = (T + TK - 1) / TK;
  if (nkv > nkv_all) nkv = nkv_all;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_q, 1);
    for (int s = 0; s < NST; ++s) mbar_init(bar_kv0 + 8 * s, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_init(bar_drain, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmKV);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_base_smem), C::TCOLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  grid_dep_sync();
  const uint32_t tmem_base = tmem_base_smem;                  // scores at columns [0, 64) (then P packed in [0, 32)), O at [64, 64 + dh)
  const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
  volatile int* abortp = &abort_flag;
  constexpr uint32_t idesc_s = make_idesc_bf16(TQ, TK, 0, 0);
  constexpr uint32_t idesc_o = make_idesc_bf16(TQ, DH, 0, 1);
  int fail = 0;

  auto load_kv = [&](int j) {
    const int st = j % NST;
    mbar_expect_tx(bar_kv0 + 8 * st, 2 * C::KV_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) {
      tma_load_4d(sK0 + st * C::KV_BYTES + c * (TK * 128), &tmKV, c * 64, H + h, j * TK, b, bar_kv0 + 8 * st);
      tma_load_4d(sV0 + st * C::KV_BYTES + c * (TK * 128), &tmKV, c * 64, 2 * H + h, j * TK, b, bar_kv0 + 8 * st);
    }
  };
  if (tid == 0) {
    mbar_expect_tx(bar_q, C::Q_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) tma_load_4d(sQ + c * (TQ * 128), &tmQ, c * 64, h, qb * TQ, b, bar_q);
    for (int i = 0; i < NST; ++i)
      if (i < nkv) load_kv(i);
  }

  const float c2 = scale * IL_LOG2E;
  // Running statistics of this thread's row.  m is the reference maximum the exponentials are taken against; it
  // is only raised when a block's maximum exceeds it by more than 8 (in log2 units), so that the accumulator in
  // TMEM rarely needs rescaling; l and O stay consistent with whatever m is, and O / l is exact either way.
  float m = -INFINITY, l = 0.f;
  const float slack = 8.0f / c2;

  // S_j = Q K_j^T; issued by thread 0 one step ahead (right after the previous block's P V) so that each sweep
  // step waits for the tensor pipe only once
  // descriptors of the operands at their first stage; a sweep step adds its stage's offset (one add per MMA:
  // the issuing thread's own instruction stream is on every step's critical path)
  const SmemDescBase dq_k = make_smem_desc_base(sQ, 16, 1024), dk_k = make_smem_desc_base(sK0, 16, 1024);
  const SmemDescBase dv_mn = make_smem_desc_base(sV0, TK * 128, 1024);
  auto issue_s = [&](int j) {
    const int st = j % NST;
    if (!mbar_wait(bar_kv0 + 8 * st, (uint32_t)(j / NST) & 1u, abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
    const uint32_t so = (uint32_t)(st * C::KV_BYTES);
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks)
      umma_bf16(tmem_base, desc_at(dq_k, (ks >> 2) * (TQ * 128) + (ks & 3) * 32),
                desc_at(dk_k, so + (ks >> 2) * (TK * 128) + (ks & 3) * 32), idesc_s, ks ? 1u : 0u);
    umma_commit(bar_s);
  };
  if (tid == 0) {
    if (!mbar_wait(bar_q, 0, abortp)) { fail = 1; abort_flag = 1; }
    issue_s(0);
  }

  for (int j = 0; j < nkv; ++j) {
    const int st = j % NST;
    const uint32_t ph = (uint32_t)j & 1u;
    if (!mbar_wait(bar_s, ph, abortp)) { fail = 1; abort_flag = 1; }
    // the previous block's P V was issued before these scores and the tensor pipe retires in order, so it has
    // landed too (bar_s covers it; only the last P V is committed on its own): the packed P columns, the O
    // accumulator and that block's K/V stage are free
    if (j > 0) {
      if (tid == 0 && j - 1 + NST < nkv) load_kv(j - 1 + NST);
    }
    tc_fence_after();
    // ---- softmax of this thread's row over the 64 keys of the block
    uint32_t r0[32], r1[32];
    tmem_ld_32x32(t_lane, r0);
    tmem_ld_32x32(t_lane + 32, r1);
    tmem_ld_wait();
    float s[64];
#pragma unroll
    for (int i = 0; i < 32; ++i) { s[i] = __uint_as_float(r0[i]); s[32 + i] = __uint_as_float(r1[i]); }
    if (j * TK + TK - 1 > qb * TQ) {              // block touches the diagonal: mask keys after the query
#pragma unroll
      for (int i = 0; i < 64; ++i)
        if (j * TK + i > row) s[i] = -INFINITY;
    }
    float mx4[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
    for (int i = 4; i < 64; i += 4) {
      mx4[0] = fmaxf(mx4[0], s[i]); mx4[1] = fmaxf(mx4[1], s[i + 1]);
      mx4[2] = fmaxf(mx4[2], s[i + 2]); mx4[3] = fmaxf(mx4[3], s[i + 3]);
    }
    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
    if (__any_sync(0xffffffffu, mx > m + slack)) {            // warp-uniform: raise the reference maximum
      const float mn = fmaxf(m, mx);
      const float alpha = ex2_fast((m - mn) * c2);            // 0 on the first block (m = -inf)
      l *= alpha;
      m = mn;
      if (j > 0) {
#pragma unroll
        for (int c0 = 0; c0 < DH; c0 += 32) {
          if (c0 + 32 <= DH) {
            uint32_t r[32];
            tmem_ld_32x32(t_lane + 64 + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st_32x32(t_lane + 64 + c0, r);
          } else {
            uint32_t r[16];
            tmem_ld_32x16(t_lane + 64 + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st_32x16(t_lane + 64 + c0, r);
          }
        }
        tmem_st_wait();
      }
    }
    const float mc = m * c2;
    float ps4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 64; i += 4) {
      s[i] = ex2_fast(fmaf(s[i], c2, -mc)); s[i + 1] = ex2_fast(fmaf(s[i + 1], c2, -mc));
      s[i + 2] = ex2_fast(fmaf(s[i + 2], c2, -mc)); s[i + 3] = ex2_fast(fmaf(s[i + 3], c2, -mc));
      ps4[0] += s[i]; ps4[1] += s[i + 1]; ps4[2] += s[i + 2]; ps4[3] += s[i + 3];
    }
    l += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
    // P (bf16 pairs, even key in the low half) over the first 32 score columns of this thread's lane
    {
      uint32_t pw[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) pw[i] = pack_bf16x2(s[2 * i], s[2 * i + 1]);
      tmem_st_32x32(t_lane, pw);
      tmem_st_wait();
    }
    tc_fence_before();
    if (__syncthreads_or(fail)) { fail = 1; break; }     // uniform exit if any thread's wait expired
    if (tid == 0) {
      tc_fence_after();
      const uint32_t so = (uint32_t)(st * C::KV_BYTES);
#pragma unroll
      for (int ks = 0; ks < TK / 16; ++ks)       // B = V read MN-major; O accumulates in TMEM
        umma_bf16_ts(tmem_base + 64, tmem_base + 8 * ks, desc_at(dv_mn, so + ks * 2048), idesc_o, (j | ks) ? 1u : 0u);
      // every thread has read S_j (barrier above); the tensor pipe runs the P V just issued, which reads the
      // packed columns, before it overwrites them with the next scores
      if (j + 1 < nkv) issue_s(j + 1);
      else umma_commit(bar_o);
    }
  }
  if (!fail && nkv > 0) {
    if (!mbar_wait(bar_o, 0, abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
  }
  fail = __syncthreads_or(fail);
  if (!fail) {
    const float inv = 1.0f / l;
    bf16* orow = o + ((size_t)b * T + row) * d + h * DH;
#pragma unroll
    for (int c0 = 0; c0 < DH; c0 += 32) {
      float v[32];
      if (c0 + 32 <= DH) {
        uint32_t r[32];
        tmem_ld_32x32(t_lane + 64 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) * inv;
      } else {
        uint32_t r[16];
        tmem_ld_32x16(t_lane + 64 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) * inv;
      }
      if (row < T) {
#pragma unroll
        for (int i = 0; i < 32 && c0 + i < DH; i += 8) {
          uint4 pk;
          pk.x = pack_bf16x2(v[i], v[i + 1]);
          pk.y = pack_bf16x2(v[i + 2], v[i + 3]);
          pk.z = pack_bf16x2(v[i + 4], v[i + 5]);
          pk.w = pack_bf16x2(v[i + 6], v[i + 7]);
          *reinterpret_cast<uint4*>(orow + c0 + i) = pk;
        }
      }
    }
    if (row < T) lse[((size_t)b * H + h) * T + row] = m * scale + logf(l);
  }
  if (tid == 0) {
    if (fail && err) atomicExch(err, DEV_TIMEOUT_MMA);
    umma_commit(bar_drain);                      // every MMA issued by this CTA has retired before TMEM goes
    int never = 0;
    mbar_wait(bar_drain, 0, &never);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TCOLS);
  }
}

template <int DH>
cudaError_t fwd_tc_launch(const bf16* qkv, bf16* o, float* lse, int B, int T, int H, unsigned* err, cudaStream_t s) {
  using C = FwdCfg<DH>;
  const unsigned long long d3 = 3ull * H * DH;
  const unsigned long long dims[4] = {(unsigned long long)DH, 3ull * H, (unsigned long long)T, (unsigned long long)B};
  const unsigned long long strides[3] = {(unsigned long long)DH * 2, d3 * 2, (unsigned long long)T * d3 * 2};
  const unsigned boxq[4] = {64, 1, TQ, 1}, boxk[4] = {64, 1, TK, 1};
  CUtensorMap tmQ, tmKV;
  if (!tma_encode_bf16(&tmQ, qkv, 4, dims, strides, boxq)) return cudaErrorInvalidValue;
  if (!tma_encode_bf16(&tmKV, qkv, 4, dims, strides, boxk)) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return e;
  dim3 grid((T + TQ - 1) / TQ, B * H);
  launch_dep(attn_fwd_tc_kernel<DH>, dim3(grid), dim3(128), C::SMEM, s, tmQ, tmKV, o, lse, T, H, rsqrtf((float)DH), err);
  return cudaGetLastError();
}


// ------------------------------------------------------------------------------------------------
// Backward.  Same structure as the forward: a CTA owns 128 rows (keys for dK/dV, queries for dQ), the other
// index is swept in blocks of 64; two threads share a row (32 columns of each block each: the backward has
// no row-wise reduction, so they never need to talk), all products run on tcgen05 and
// — because the backward has no running maximum — every gradient accumulates in TMEM across the sweep.
// Probabilities are recomputed from the saved log-sum-exp; delta_i = sum_c dO_ic O_ic.
// P^T and dS^T (dS for dQ) never touch shared memory: a thread rounds its 32 values to bf16, packs them in
// pairs and stores the 16 words back into the first half of the TMEM columns it has just read, from where
// the next MMA takes them as its A operand.  The tiles of the swept index come through a 4-deep TMA ring.
// ------------------------------------------------------------------------------------------------

template <int DH>
struct BwdCfg {
  static constexpr int NCH = (DH + 63) / 64;
  static constexpr int NST = (DH > 128) ? 1 : 4;        // ring depth of the swept tiles (one 64 KB stage is all that fits at dh 256)
  static constexpr bool AHEAD = NST > 1;                // the next step's scores are issued one step ahead (needs a second stage)
  static constexpr int ROW_BYTES = NCH * TQ * 128;      // a 128-row operand (all chunks)
  static constexpr int BLK_BYTES = NCH * TK * 128;      // a 64-row operand
  // dK/dV: K, V resident; ring of (Q, dO); lse/delta vectors.  TMEM: S^T, dP^T, dV, dK.
  static constexpr int SMEM_KV = 2 * ROW_BYTES + NST * 2 * BLK_BYTES + 1024 + 2 * 2 * 64 * 4 + 128;
  static constexpr int TCOLS_KV = (128 + 2 * DH <= 256) ? 256 : 512;   // dh 256: one accumulator per launch (PART)
  // dQ: Q, dO resident; ring of (K, V).  TMEM: S, dP, dQ.
  static constexpr int SMEM_Q = 2 * ROW_BYTES + NST * 2 * BLK_BYTES + 1024 + 128;
  static constexpr int TCOLS_Q = (128 + DH <= 256) ? 256 : 512;
};

// 32 fp32 values -> 16 words of bf16 pairs (even index in the low half)
__device__ __forceinline__ void pack_row32(const float (&v)[32], uint32_t (&w)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) w[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
}
// TMEM column offset (within a 64-column block whose two 32-column halves each hold their packed values in
// their first 16 columns) of the A operand of K-step ks (16 elements = 8 columns)
__device__ __forceinline__ constexpr uint32_t packed_col(int ks) { return (uint32_t)((ks >> 1) * 32 + (ks & 1) * 8); }

// PART: 0 = dV and dK in one launch; 1 = dV only; 2 = dK only (head dimensions whose two accumulators do not fit
// the 512 TMEM columns together run as two launches, each recomputing the scores).
template <int DH, int PART>
__global__ void __launch_bounds__(256) attn_bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap tmRow,   // qkv, 128-row box
                                                              const __grid_constant__ CUtensorMap tmBlk,   // qkv, 64-row box
                                                              const __grid_constant__ CUtensorMap tmdO,    // dout, 64-row box
                                                              const float* __restrict__ lse, const float* __restrict__ delta,
                                                              bf16* __restrict__ dqkv, int B, int T, int H, float scale,
                                                              unsigned* err) {
  using C = BwdCfg<DH>;
  constexpr int NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_smem;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = base, sV = sK + C::ROW_BYTES;
  const uint32_t sQ0 = sV + C::ROW_BYTES, sdO0 = sQ0 + NST * C::BLK_BYTES;
  const uint32_t vecs = sdO0 + NST * C::BLK_BYTES;               // lse2[2][64], delta[2][64]
  const uint32_t bars = vecs + 2 * 2 * 64 * 4;
  const uint32_t bar_kv = bars, bar_s = bars + 8, bar_acc = bars + 16, bar_drain = bars + 24, bar_q0 = bars + 32;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  float* s_lse = reinterpret_cast<float*>(gen + (vecs - base));  // [2][64]
  float* s_del = s_lse + 128;                                    // [2][64]

  // 256 threads: thread (r, hf) owns row r = tid % 128 and columns [32 hf, 32 hf + 32) of each 64-wide block
  const int tid = threadIdx.x, warp = tid >> 5, r = tid & 127, hf = tid >> 7;
  const int kb = blockIdx.x;
  const int nb = blockIdx.y / H, h = blockIdx.y % H;
  const int bs = nb % B;
  const int d = H * DH;
  const int key = kb * TQ + r;
  const int nq = (T + TK - 1) / TK;
  const int q0 = (kb * TQ) / TK;                                 // first query block that can see these keys
  const float* lse_b = lse + ((size_t)bs * H + h) * T;
  const float* del_b = delta + ((size_t)nb * H + h) * T;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_kv, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_acc, 1);
    mbar_init(bar_drain, 1);
    for (int s = 0; s < NST; ++s) mbar_init(bar_q0 + 8 * s, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmRow);
    tma_prefetch_desc(&tmBlk);
    tma_prefetch_desc(&tmdO);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_base_smem), C::TCOLS_KV);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();          // tensor memory is held by this CTA before the next kernel may become resident
  grid_dep_sync();
  // lse (in log2 units) and delta of a query block: fetched from global memory into a register one sweep
  // step before they are put into shared memory (buffer j&1), two steps before they are used, so that no
  // step waits on that load
  auto fetch_vec = [&](int j) -> float {
    const int q = j * TK + (tid & 63);
    if (j >= nq || q >= T || tid >= 128) return 0.f;
    return tid < 64 ? lse_b[q] * IL_LOG2E : del_b[q];
  };
  auto put_vec = [&](int j, float v) {
    if (tid < 64) s_lse[(j & 1) * 64 + tid] = v;
    else if (tid < 128) s_del[(j & 1) * 64 + (tid & 63)] = v;
  };
  if (q0 < nq) put_vec(q0, fetch_vec(q0));
  float vec_next = fetch_vec(q0 + 1);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // TMEM: S^T [0,64) and dP^T [64,128) (each later overwritten in part by its packed bf16 successor P^T,
  // dS^T), dV [128,128+dh), dK [128+dh, 128+2dh)
  const uint32_t tmem_base = tmem_base_smem;
  const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  volatile int* abortp = &abort_flag;
  constexpr uint32_t idesc_s = make_idesc_bf16(TQ, TK, 0, 0);
  constexpr uint32_t idesc_g = make_idesc_bf16(TQ, DH, 0, 1);
  int fail = 0;

  auto load_q = [&](int j) {
    const int st = (j - q0) % NST;
    mbar_expect_tx(bar_q0 + 8 * st, 2 * C::BLK_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) {
      tma_load_4d(sQ0 + st * C::BLK_BYTES + c * (TK * 128), &tmBlk, c * 64, h, j * TK, bs, bar_q0 + 8 * st);
      tma_load_4d(sdO0 + st * C::BLK_BYTES + c * (TK * 128), &tmdO, c * 64, h, j * TK, nb, bar_q0 + 8 * st);
    }
  };
  if (tid == 0) {
    mbar_expect_tx(bar_kv, 2 * C::ROW_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) {
      tma_load_4d(sK + c * (TQ * 128), &tmRow, c * 64, H + h, kb * TQ, bs, bar_kv);
      tma_load_4d(sV + c * (TQ * 128), &tmRow, c * 64, 2 * H + h, kb * TQ, bs, bar_kv);
    }
    for (int i = 0; i < NST; ++i)
      if (q0 + i < nq) load_q(q0 + i);
  }
  const float c2 = scale * IL_LOG2E;

  // S^T and dP^T of query block j; issued by thread 0 one step ahead (right after the previous block's dV/dK
  // products) so that each sweep step waits for the tensor pipe only once
  // descriptors of the operands at their first stage; a sweep step adds its stage's offset (one add per MMA:
  // the issuing thread's own instruction stream is on every step's critical path)
  const SmemDescBase dk_k = make_smem_desc_base(sK, 16, 1024), dv_k = make_smem_desc_base(sV, 16, 1024);
  const SmemDescBase dq_k = make_smem_desc_base(sQ0, 16, 1024), ddo_k = make_smem_desc_base(sdO0, 16, 1024);
  const SmemDescBase dq_mn = make_smem_desc_base(sQ0, TK * 128, 1024), ddo_mn = make_smem_desc_base(sdO0, TK * 128, 1024);
  auto issue_s = [&](int j) {
    const int it = j - q0, st = it % NST;
    if (!mbar_wait(bar_q0 + 8 * st, (uint32_t)(it / NST) & 1u, abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
    const uint32_t so = (uint32_t)(st * C::BLK_BYTES);
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
      const uint32_t off_a = (ks >> 2) * (TQ * 128) + (ks & 3) * 32;
      const uint32_t off_b = so + (ks >> 2) * (TK * 128) + (ks & 3) * 32;
      umma_bf16(tmem_base, desc_at(dk_k, off_a), desc_at(dq_k, off_b), idesc_s, ks ? 1u : 0u);
      if (PART != 1) umma_bf16(tmem_base + 64, desc_at(dv_k, off_a), desc_at(ddo_k, off_b), idesc_s, ks ? 1u : 0u);
    }
    umma_commit(bar_s);
  };
  if (tid == 0 && q0 < nq) {
    if (!mbar_wait(bar_kv, 0, abortp)) { fail = 1; abort_flag = 1; }
    if (C::AHEAD) issue_s(q0);
  }

  for (int j = q0; j < nq; ++j) {
    const int it = j - q0;
    const int st = it % NST;
    if (j + 1 < nq) put_vec(j + 1, vec_next);      // visible after this step's barrier
    vec_next = fetch_vec(j + 2);
    if (!C::AHEAD) {
      // single stage: the previous step's products must have retired before its tiles are replaced and the
      // new scores overwrite the packed columns; only then are this step's scores issued
      if (it > 0) {
        if (!mbar_wait(bar_acc, (uint32_t)(it - 1) & 1u, abortp)) { fail = 1; abort_flag = 1; }
        if (tid == 0) load_q(j);
      }
      if (tid == 0) issue_s(j);
    }
    if (!mbar_wait(bar_s, (uint32_t)it & 1u, abortp)) { fail = 1; abort_flag = 1; }
    // the previous step's dV/dK products were issued before these scores, so they have landed too: the packed
    // P^T / dS^T columns and that step's Q/dO stage are free
    // (the tensor pipe retires in order: bar_s covers them, only the last step's products are committed on their own)
    if (C::AHEAD && it > 0) {
      if (tid == 0 && j - 1 + NST < nq) load_q(j - 1 + NST);
    }
    tc_fence_after();
    {
      float p[32], ds[32];
      uint32_t r0[32], r1[32];
      tmem_ld_32x32(t_lane + 32 * hf, r0);
      if (PART != 1) tmem_ld_32x32(t_lane + 64 + 32 * hf, r1);
      tmem_ld_wait();
      const float4* lv = reinterpret_cast<const float4*>(s_lse + (j & 1) * 64 + 32 * hf);
      const float4* dv_ = reinterpret_cast<const float4*>(s_del + (j & 1) * 64 + 32 * hf);
      const bool diag = (j * TK < kb * TQ + TQ);   // some queries of this block precede some keys of this CTA
      const bool tail = (j * TK + TK > T);
      const int qbase = j * TK + 32 * hf;
#pragma unroll
      for (int i4 = 0; i4 < 8; ++i4) {
        const float4 l4 = lv[i4], d4 = dv_[i4];
        const float ll[4] = {l4.x, l4.y, l4.z, l4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = 4 * i4 + e;
          p[i] = ex2_fast(fmaf(__uint_as_float(r0[i]), c2, -ll[e]));
          ds[i] = PART != 1 ? __uint_as_float(r1[i]) - dd[e] : 0.f;
        }
      }
      if (diag || tail) {                          // uniform: only blocks on the diagonal or past the sequence end
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (qbase + i < key || qbase + i >= T) p[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) ds[i] *= p[i];
      uint32_t pw[16], dw[16];
      if (PART != 2) {
        pack_row32(p, pw);
        tmem_st_32x16(t_lane + 32 * hf, pw);       // P^T over the first half of the S^T columns this thread read
      }
      if (PART != 1) {
        pack_row32(ds, dw);
        tmem_st_32x16(t_lane + 64 + 32 * hf, dw);  // dS^T likewise over dP^T
      }
      tmem_st_wait();
    }
    tc_fence_before();
    if (__syncthreads_or(fail)) { fail = 1; break; }
    if (tid == 0) {
      tc_fence_after();
      const uint32_t so = (uint32_t)(st * C::BLK_BYTES);
#pragma unroll
      for (int ks = 0; ks < TK / 16; ++ks) {
        const uint32_t off_b = so + ks * 2048;                                              // MN-major: 16 queries
        if (PART != 2)
          umma_bf16_ts(tmem_base + 128, tmem_base + packed_col(ks), desc_at(ddo_mn, off_b), idesc_g, (it | ks) ? 1u : 0u);
        if (PART != 1)
          umma_bf16_ts(tmem_base + 128 + (PART == 0 ? DH : 0), tmem_base + 64 + packed_col(ks), desc_at(dq_mn, off_b), idesc_g,
                       (it | ks) ? 1u : 0u);
      }
      // every thread has read S^T / dP^T of this step (barrier above); the tensor pipe runs the products just
      // issued, which read the packed columns, before it overwrites them with the next scores
      if (C::AHEAD && j + 1 < nq) issue_s(j + 1);
      else umma_commit(bar_acc);
    }
  }
  const int nit = nq - q0;
  if (!fail && nit > 0) {
    if (!mbar_wait(bar_acc, C::AHEAD ? 0u : ((uint32_t)(nit - 1) & 1u), abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
  }
  fail = __syncthreads_or(fail);
  if (!fail) {
    bf16* rowp = dqkv + ((size_t)nb * T + key) * (3 * d) + h * DH;
    {
      // one launch for both: the first half of the threads writes dV, the second half dK; a launch that holds
      // one of them splits its columns between the two halves
      const int which = PART == 0 ? hf : PART - 1;
      const uint32_t tcol = t_lane + 128 + (PART == 0 ? which * DH : 0);
      bf16* dst = rowp + (which == 0 ? 2 * d : d);
      const float f = which == 0 ? 1.0f : scale;
      const int cbeg = PART == 0 ? 0 : hf * (DH / 2), cend = PART == 0 ? DH : cbeg + DH / 2;
#pragma unroll
      for (int c0 = cbeg; c0 < cend; c0 += 32) {
        float v[32];
        if (c0 + 32 <= DH) {
          uint32_t rr[32];
          tmem_ld_32x32(tcol + c0, rr);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = nit > 0 ? __uint_as_float(rr[i]) * f : 0.f;
        } else {
          uint32_t rr[16];
          tmem_ld_32x16(tcol + c0, rr);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = nit > 0 ? __uint_as_float(rr[i]) * f : 0.f;
        }
        if (key < T) {
#pragma unroll
          for (int i = 0; i < 32 && c0 + i < DH; i += 8) {
            uint4 pk;
            pk.x = pack_bf16x2(v[i], v[i + 1]);
            pk.y = pack_bf16x2(v[i + 2], v[i + 3]);
            pk.z = pack_bf16x2(v[i + 4], v[i + 5]);
            pk.w = pack_bf16x2(v[i + 6], v[i + 7]);
            *reinterpret_cast<uint4*>(dst + c0 + i) = pk;
          }
        }
      }
    }
  }
  if (tid == 0) {
    if (fail && err) atomicExch(err, DEV_TIMEOUT_MMA);
    umma_commit(bar_drain);
    int never = 0;
    mbar_wait(bar_drain, 0, &never);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TCOLS_KV);
  }
}

template <int DH>
__global__ void __launch_bounds__(256) attn_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmRow,    // qkv, 128-row box
                                                             const __grid_constant__ CUtensorMap tmBlk,    // qkv, 64-row box
                                                             const __grid_constant__ CUtensorMap tmdO,     // dout, 128-row box
                                                             const float* __restrict__ lse, const float* __restrict__ delta,
                                                             bf16* __restrict__ dqkv, int B, int T, int H, float scale,
                                                             unsigned* err) {
  using C = BwdCfg<DH>;
  constexpr int NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_smem;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base, sdO = sQ + C::ROW_BYTES;
  const uint32_t sK0 = sdO + C::ROW_BYTES, sV0 = sK0 + NST * C::BLK_BYTES;
  const uint32_t bars = sV0 + NST * C::BLK_BYTES;
  const uint32_t bar_q = bars, bar_s = bars + 8, bar_acc = bars + 16, bar_drain = bars + 24, bar_kv0 = bars + 32;

  // 256 threads: thread (r, hf) owns row r = tid % 128 and columns [32 hf, 32 hf + 32) of each 64-wide block
  const int tid = threadIdx.x, warp = tid >> 5, r = tid & 127, hf = tid >> 7;
  const int qb = gridDim.x - 1 - blockIdx.x;
  const int nb = blockIdx.y / H, h = blockIdx.y % H;
  const int bs = nb % B;
  const int d = H * DH;
  const int row = qb * TQ + r;
  int nkv = (qb * TQ + TQ + TK - 1) / TK;
  const int nkv_all = (T + TK - 1) / TK;
  if (nkv > nkv_all) nkv = nkv_all;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_q, 1);
    for (int s = 0; s < NST; ++s) mbar_init(bar_kv0 + 8 * s, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_acc, 1);
    mbar_init(bar_drain, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmRow);
    tma_prefetch_desc(&tmBlk);
    tma_prefetch_desc(&tmdO);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_base_smem), C::TCOLS_Q);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  grid_dep_sync();
  const uint32_t tmem_base = tmem_base_smem;     // S [0,64), dP [64,128) (later in part the packed dS), dQ [128,128+dh)
  const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  volatile int* abortp = &abort_flag;
  constexpr uint32_t idesc_s = make_idesc_bf16(TQ, TK, 0, 0);
  constexpr uint32_t idesc_g = make_idesc_bf16(TQ, DH, 0, 1);
  int fail = 0;

  auto load_kv = [&](int j) {
    const int st = j % NST;
    mbar_expect_tx(bar_kv0 + 8 * st, 2 * C::BLK_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) {
      tma_load_4d(sK0 + st * C::BLK_BYTES + c * (TK * 128), &tmBlk, c * 64, H + h, j * TK, bs, bar_kv0 + 8 * st);
      tma_load_4d(sV0 + st * C::BLK_BYTES + c * (TK * 128), &tmBlk, c * 64, 2 * H + h, j * TK, bs, bar_kv0 + 8 * st);
    }
  };
  if (tid == 0) {
    mbar_expect_tx(bar_q, 2 * C::ROW_BYTES);
#pragma unroll
    for (int c = 0; c < C::NCH; ++c) {
      tma_load_4d(sQ + c * (TQ * 128), &tmRow, c * 64, h, qb * TQ, bs, bar_q);
      tma_load_4d(sdO + c * (TQ * 128), &tmdO, c * 64, h, qb * TQ, nb, bar_q);
    }
    for (int i = 0; i < NST; ++i)
      if (i < nkv) load_kv(i);
  }
  const float c2 = scale * IL_LOG2E;
  const float lse2 = row < T ? lse[((size_t)bs * H + h) * T + row] * IL_LOG2E : 0.f;
  const float del = row < T ? delta[((size_t)nb * H + h) * T + row] : 0.f;

  // S and dP of key block j; issued by thread 0 one step ahead (right after the previous block's dQ product)
  // descriptors at the first stage; a sweep step adds its stage's offset (one add per MMA)
  const SmemDescBase dq_k = make_smem_desc_base(sQ, 16, 1024), ddo_k = make_smem_desc_base(sdO, 16, 1024);
  const SmemDescBase dk_k = make_smem_desc_base(sK0, 16, 1024), dv_k = make_smem_desc_base(sV0, 16, 1024);
  const SmemDescBase dk_mn = make_smem_desc_base(sK0, TK * 128, 1024);
  auto issue_s = [&](int j) {
    const int st = j % NST;
    if (!mbar_wait(bar_kv0 + 8 * st, (uint32_t)(j / NST) & 1u, abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
    const uint32_t so = (uint32_t)(st * C::BLK_BYTES);
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
      const uint32_t off_a = (ks >> 2) * (TQ * 128) + (ks & 3) * 32;
      const uint32_t off_b = so + (ks >> 2) * (TK * 128) + (ks & 3) * 32;
      umma_bf16(tmem_base, desc_at(dq_k, off_a), desc_at(dk_k, off_b), idesc_s, ks ? 1u : 0u);
      umma_bf16(tmem_base + 64, desc_at(ddo_k, off_a), desc_at(dv_k, off_b), idesc_s, ks ? 1u : 0u);
    }
    umma_commit(bar_s);
  };
  if (tid == 0 && nkv > 0) {
    if (!mbar_wait(bar_q, 0, abortp)) { fail = 1; abort_flag = 1; }
    if (C::AHEAD) issue_s(0);
  }

  for (int j = 0; j < nkv; ++j) {
    const int st = j % NST;
    if (!C::AHEAD) {      // single stage: retire the previous step's product, replace its tiles, then issue these scores
      if (j > 0) {
        if (!mbar_wait(bar_acc, (uint32_t)(j - 1) & 1u, abortp)) { fail = 1; abort_flag = 1; }
        if (tid == 0) load_kv(j);
      }
      if (tid == 0) issue_s(j);
    }
    if (!mbar_wait(bar_s, (uint32_t)j & 1u, abortp)) { fail = 1; abort_flag = 1; }
    if (C::AHEAD && j > 0) {                         // issued before these scores: landed (bar_s covers it), the packed dS and that step's K/V stage are free
      if (tid == 0 && j - 1 + NST < nkv) load_kv(j - 1 + NST);
    }
    tc_fence_after();
    {
      float ds[32];
      uint32_t r0[32], r1[32];
      tmem_ld_32x32(t_lane + 32 * hf, r0);
      tmem_ld_32x32(t_lane + 64 + 32 * hf, r1);
      tmem_ld_wait();
      const bool diag = (j * TK + TK - 1 > qb * TQ);
      const int kbase = j * TK + 32 * hf;
#pragma unroll
      for (int i = 0; i < 32; ++i) ds[i] = ex2_fast(fmaf(__uint_as_float(r0[i]), c2, -lse2));
      if (diag) {                                  // uniform: only blocks on the diagonal
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (kbase + i > row) ds[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) ds[i] *= (__uint_as_float(r1[i]) - del);
      uint32_t dw[16];
      pack_row32(ds, dw);
      tmem_st_32x16(t_lane + 64 + 32 * hf, dw);      // dS over the first half of the dP columns this thread read
      tmem_st_wait();
    }
    tc_fence_before();
    if (__syncthreads_or(fail)) { fail = 1; break; }
    if (tid == 0) {
      tc_fence_after();
      const uint32_t so = (uint32_t)(st * C::BLK_BYTES);
#pragma unroll
      for (int ks = 0; ks < TK / 16; ++ks)
        umma_bf16_ts(tmem_base + 128, tmem_base + 64 + packed_col(ks), desc_at(dk_mn, so + ks * 2048), idesc_g,
                     (j | ks) ? 1u : 0u);
      if (C::AHEAD && j + 1 < nkv) issue_s(j + 1);
      else umma_commit(bar_acc);
    }
  }
  if (!fail && nkv > 0) {
    if (!mbar_wait(bar_acc, C::AHEAD ? 0u : ((uint32_t)(nkv - 1) & 1u), abortp)) { fail = 1; abort_flag = 1; }
    tc_fence_after();
  }
  fail = __syncthreads_or(fail);
  if (!fail) {
    bf16* dst = dqkv + ((size_t)nb * T + row) * (3 * d) + h * DH;
#pragma unroll
    for (int u = 0; u < DH / 16; ++u) {              // 16-column units, alternating between the two halves
      if ((u & 1) != hf) continue;
      const int c0 = u * 16;
      float v[16];
      {
        uint32_t rr[16];
        tmem_ld_32x16(t_lane + 128 + c0, rr);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(rr[i]) * scale;
      }
      if (row < T) {
#pragma unroll
        for (int i = 0; i < 16; i += 8) {
          uint4 pk;
          pk.x = pack_bf16x2(v[i], v[i + 1]);
          pk.y = pack_bf16x2(v[i + 2], v[i + 3]);
          pk.z = pack_bf16x2(v[i + 4], v[i + 5]);
          pk.w = pack_bf16x2(v[i + 6], v[i + 7]);
          *reinterpret_cast<uint4*>(dst + c0 + i) = pk;
        }
      }
    }
  }
  if (tid == 0) {
    if (fail && err) atomicExch(err, DEV_TIMEOUT_MMA);
    umma_commit(bar_drain);
    int never = 0;
    mbar_wait(bar_drain, 0, &never);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TCOLS_Q);
  }
}

// ------------------------------------------------------------------------------------------------
// Backward in one sweep (head dimensions up to 64).  The two-kernel form above recomputes the scores twice (seven
// products for five); here a CTA owns 128 keys, sweeps the queries in blocks of 128 and produces dV, dK and its
// share of dQ from one recomputation of S^T and dP^T:
//   S^T, dP^T   tcgen05.mma M128 (keys) N64 per 64-query half -> TMEM, two halves per step
//   P^T, dS^T   threads (four per key row, 16 columns of a half each) recompute the probabilities from the saved
//               log-sum-exp, round to bf16 and store the packed pairs back over the score columns
//   dV += P^T dO, dK += dS^T Q      A operand read from those TMEM columns, accumulated over the whole sweep
//   dQ_blk = dS K                   needs dS with the queries as rows: the same threads also write their dS values
//                                   to shared memory in the layout of an MN-major A operand (swizzled 128-byte
//                                   rows, one row per key); the product lands in one of two TMEM buffers and is
//                                   added to an fp32 [rows, d] accumulator in global memory with red.add (every
//                                   key tile of a (sequence, head) contributes to the same query rows)
// Roles: warps 0-15 recompute and convert (four threads per key row), warps 16-19 add finished dQ blocks to the
// global accumulator and store an item's dV / dK, warps 20 and 21 issue the MMAs (scores and dQ / dV and dK: a
// single thread issues small MMAs no faster than one per ~54 cycles), warp 22 feeds the Q / dO ring by TMA and the
// per-query lse / delta vectors by plain loads.  The halves
// give the pipeline its overlap: while the threads work on one half of the step, the tensor pipe runs the other
// half's products and the next step's scores for the half just finished.  One CTA per SM (all 512 TMEM columns,
// ~195 KB of shared memory), persistent: a CTA walks a list of (key tile, sequence, head) items, and the loads and
// scores of an item start while the previous item's dV / dK are still being written out.
// The sum over key tiles in dQ is made by floating-point atomics: its order, and with it the last bit of dQ,
// depends on scheduling.  Every wait is bounded.
// ------------------------------------------------------------------------------------------------
template <int DH>
struct FusedCfg {
  static constexpr int NST = 3;                          // Q / dO ring depth
  static constexpr int ROW_BYTES = TQ * 128;             // a 128-row operand (one 64-column chunk)
  static constexpr int DS_BYTES = 2 * TQ * 128;          // dS of one step: two 64-query chunks x 128 key rows x 128 B
  static constexpr int VEC_BYTES = 2 * TQ * 4;           // lse (log2 units) and delta of the step's 128 queries
  static constexpr int SMEM = 2 * ROW_BYTES + NST * (2 * ROW_BYTES + VEC_BYTES) + 2 * DS_BYTES + 256 + 1024;
  // TMEM columns: S^T [0,128) (two halves), dP^T [128,256), dV [256,256+DH), dK [320,320+DH), dQ [384,384+DH) / [448,448+DH)
  static constexpr int C_S = 0, C_DP = 128, C_DV = 256, C_DK = 320, C_DQ = 384;
};

constexpr int FUSED_THREADS = 768;   // warps 0-15 recompute, 16-19 flush dQ and store dV / dK, 20-22 issue MMAs, 23 loads
constexpr int FUSED_RW = 16;         // recompute warps: four threads per key row, 16 query columns of a half each

// Work item = (key tile, gradient sequence, head).  Items are numbered key tile first, so the long sweeps (key tile
// 0 sees every query block) come first; CTA c takes items c, c + gridDim.x, ...  Every role walks the same list and
// counts the same global step number g, from which ring stages and barrier parities follow.
struct FusedItem { int kb, nb, h, bs, nit; };
__device__ __forceinline__ FusedItem fused_item(int item, int nbh, int H, int B, int nq) {
  FusedItem w;
  w.kb = item / nbh;
  const int r = item - w.kb * nbh;
  w.nb = r / H;
  w.h = r - w.nb * H;
  w.bs = w.nb % B;
  w.nit = nq - w.kb;                    // query blocks kb .. nq-1 see these keys
  return w;
}

template <int DH>
__global__ void __launch_bounds__(FUSED_THREADS, 1) attn_bwd_fused_kernel(const __grid_constant__ CUtensorMap tmRow,     // qkv, 128-row box
                                                                          const __grid_constant__ CUtensorMap tmdO,      // dout, 128-row box
                                                                          const __grid_constant__ CUtensorMap tmAcc,     // dQ accumulator (fp32), 32 x 128 box
                                                                          const float* __restrict__ lse, const float* __restrict__ delta,
                                                                          bf16* __restrict__ dqkv, int NB,
                                                                          int B, int T, int H, float scale, unsigned* err) {
  using C = FusedCfg<DH>;
  constexpr int NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ volatile int flush_fail;
  __shared__ uint32_t tmem_base_smem;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = base, sV = sK + C::ROW_BYTES;
  const uint32_t sQ0 = sV + C::ROW_BYTES;                                  // stage st: Q at sQ0 + st * STAGE, dO after it
  constexpr uint32_t STAGE = 2 * C::ROW_BYTES;
  const uint32_t sDS = sQ0 + NST * STAGE;                                  // two dS buffers
  const uint32_t sVec = sDS + 2 * C::DS_BYTES;                             // NST x (lse2[128], delta[128])
  const uint32_t bars = sVec + NST * C::VEC_BYTES;
  // barriers (8 bytes each)
  const uint32_t bar_kv = bars, bar_kvfree = bars + 8, bar_acc = bars + 16, bar_accfree = bars + 24, bar_ds = bars + 32, bar_init = bars + 40;
  auto bar_drain = [&](int t) { return bars + 48 + 8 * t; };                   // one per issuing thread
  auto bar_full = [&](int st) { return bars + 72 + 8 * st; };
  auto bar_empty = [&](int st) { return bars + 72 + 8 * (NST + st); };
  auto bar_s = [&](int x) { return bars + 72 + 8 * (2 * NST + x); };           // scores of half x ready
  auto bar_p = [&](int x) { return bars + 72 + 8 * (2 * NST + 2 + x); };       // P^T / dS^T of half x in tensor memory
  auto bar_dq = [&](int b) { return bars + 72 + 8 * (2 * NST + 4 + b); };      // dQ buffer b complete
  auto bar_dqfree = [&](int b) { return bars + 72 + 8 * (2 * NST + 6 + b); };  // dQ buffer b flushed
  auto bar_vec = [&](int st) { return bars + 72 + 8 * (2 * NST + 8 + st); };   // lse / delta vectors of stage st written
  auto bar_dsfree = [&](int b) { return bars + 72 + 8 * (3 * NST + 8 + b); };  // dS buffer b (also the staging of its dQ block) free again
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  float* s_vec = reinterpret_cast<float*>(gen + (sVec - base));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = H * DH;
  const int nq = (T + TQ - 1) / TQ;
  const int nbh = NB * H;
  const int nitems = nq * nbh;
  volatile int* abortp = &abort_flag;

  if (tid == 0) {
    abort_flag = 0;
    flush_fail = 0;
    mbar_init(bar_kv, 1);
    mbar_init(bar_kvfree, 3);            // the three issuing threads
    mbar_init(bar_acc, 2);               // the two half threads
    mbar_init(bar_init, 1);
    mbar_init(bar_accfree, 4);           // one arrival per flush warp
    mbar_init(bar_ds, FUSED_RW);         // one arrival per recompute warp
    mbar_init(bar_drain(0), 1);
    mbar_init(bar_drain(1), 1);
    mbar_init(bar_drain(2), 1);
    for (int st = 0; st < NST; ++st) { mbar_init(bar_full(st), 1); mbar_init(bar_empty(st), 2); mbar_init(bar_vec(st), 1); }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar_s(x), 1);
      mbar_init(bar_p(x), FUSED_RW);
      mbar_init(bar_dq(x), 1);
      mbar_init(bar_dqfree(x), 4);       // one arrival per flush warp
      mbar_init(bar_dsfree(x), 1);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tmRow);
    tma_prefetch_desc(&tmdO);
    tma_prefetch_desc(&tmAcc);
  }
  if (warp == 20) {
    tmem_alloc(smem_u32(&tmem_base_smem), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  grid_dep_sync();
  const uint32_t tmem_base = tmem_base_smem;
  const float c2 = scale * IL_LOG2E;
  int fail = 0;

  if (warp == 23) {
    // ---------------------------------------------------------------- loads
    int g = 0, n_item = 0;
    for (int item = blockIdx.x; item < nitems && !fail; item += gridDim.x, ++n_item) {
      const FusedItem w = fused_item(item, nbh, H, B, nq);
      const float* lse_b = lse + ((size_t)w.bs * H + w.h) * T;
      const float* del_b = delta + ((size_t)w.nb * H + w.h) * T;
      for (int it = 0; it < w.nit; ++it) {
        const int gs = g + it, st = gs % NST, j = w.kb + it;
        int ok = 1;
        if (lane == 0 && gs >= NST) ok = mbar_wait(bar_empty(st), (uint32_t)(gs / NST - 1) & 1u, abortp) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { fail = 1; abort_flag = 1; break; }
        // the tiles first (their latency is the longer one), then the step's lse / delta vectors by plain loads,
        // published on a barrier of their own
        if (lane == 0) {
          mbar_expect_tx(bar_full(st), 2 * C::ROW_BYTES);
          tma_load_4d(sQ0 + st * STAGE, &tmRow, 0, w.h, j * TQ, w.bs, bar_full(st));
          tma_load_4d(sQ0 + st * STAGE + C::ROW_BYTES, &tmdO, 0, w.h, j * TQ, w.nb, bar_full(st));
        }
        float* vec = s_vec + st * (2 * TQ);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int q = j * TQ + q4 * 32 + lane;
          vec[q4 * 32 + lane] = q < T ? lse_b[q] * IL_LOG2E : 0.f;
          vec[TQ + q4 * 32 + lane] = q < T ? del_b[q] : 0.f;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_vec(st));                   // its release publishes the warp's stores
        if (it == 0) {
          // the item's K and V (after its first query block, which does not depend on the previous item): their
          // buffers are free once the previous item's last products that read them have retired
          int ok2 = 1;
          if (lane == 0 && n_item > 0) ok2 = mbar_wait(bar_kvfree, (uint32_t)(n_item - 1) & 1u, abortp) ? 1 : 0;
          ok2 = __shfl_sync(0xffffffffu, ok2, 0);
          if (!ok2) { fail = 1; abort_flag = 1; break; }
          if (lane == 0) {
            mbar_expect_tx(bar_kv, 2 * C::ROW_BYTES);
            tma_load_4d(sK, &tmRow, 0, H + w.h, w.kb * TQ, w.bs, bar_kv);
            tma_load_4d(sV, &tmRow, 0, 2 * H + w.h, w.kb * TQ, w.bs, bar_kv);
          }
        }
      }
      g += w.nit;
    }
  } else if (warp == 20 || warp == 21) {
    // ---------------------------------------------------------------- MMA issue, one thread per half x of the query block
    // A thread issues small MMAs no faster than one per ~54 cycles, and every hand-over between threads costs a
    // commit / barrier round trip of several hundred cycles.  So each half has its own issuing thread that does, in
    // program order (the tensor pipe keeps one thread's MMAs in order), dV += P^T(x) dO(x), dK += dS^T(x) Q(x) and
    // then the next step's S^T(x), dP^T(x) into the score columns those products have just read.  Both threads add
    // into the same dV / dK accumulators (the pipe executes one MMA at a time; the order in which the two halves are
    // added is not fixed).
    if (lane == 0) {
      const int x = warp - 20;
      constexpr uint32_t idesc_s = make_idesc_bf16(TQ, TK, 0, 0);          // S^T / dP^T half: M128 N64, both K-major
      constexpr uint32_t idesc_g = make_idesc_bf16(TQ, DH, 0, 1);          // dV / dK: A from TMEM, B MN-major
      const SmemDescBase dk_k = make_smem_desc_base(sK, 16, 1024), dv_k = make_smem_desc_base(sV, 16, 1024);
      const SmemDescBase dq_k = make_smem_desc_base(sQ0, 16, 1024), ddo_k = make_smem_desc_base(sQ0 + C::ROW_BYTES, 16, 1024);
      const SmemDescBase dq_mn = make_smem_desc_base(sQ0, TQ * 128, 1024), ddo_mn = make_smem_desc_base(sQ0 + C::ROW_BYTES, TQ * 128, 1024);
      bool ok = true;
      // scores of this half of the step held in stage st: rows 64x .. 64x+63 of the Q / dO tiles (8 KB further)
      auto issue_scores = [&](int st) {
        const uint32_t so = (uint32_t)st * STAGE + (uint32_t)x * (TK * 128);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          umma_bf16(tmem_base + C::C_S + 64 * x, desc_at(dk_k, ks * 32), desc_at(dq_k, so + ks * 32), idesc_s, ks ? 1u : 0u);
          umma_bf16(tmem_base + C::C_DP + 64 * x, desc_at(dv_k, ks * 32), desc_at(ddo_k, so + ks * 32), idesc_s, ks ? 1u : 0u);
        }
        umma_commit(bar_s(x));
      };
      int g = 0, n_item = 0;
      for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++n_item) {
        const FusedItem w = fused_item(item, nbh, H, B, nq);
        // first step of the item: its scores need the item's K / V and the step's Q / dO (the score columns are free:
        // this thread's own last products of the previous item come before them in the pipe)
        if (!mbar_wait(bar_kv, (uint32_t)n_item & 1u, abortp)) { ok = false; break; }
        if (!mbar_wait(bar_full(g % NST), (uint32_t)(g / NST) & 1u, abortp)) { ok = false; break; }
        tc_fence_after();
        issue_scores(g % NST);
        // the accumulators still hold the previous item's dV / dK until they have been stored; the half-1 thread also
        // lets the half-0 thread's first products (which overwrite instead of adding) go first
        if (n_item > 0 && !mbar_wait(bar_accfree, (uint32_t)(n_item - 1) & 1u, abortp)) { ok = false; break; }
        if (x == 1 && !mbar_wait(bar_init, (uint32_t)n_item & 1u, abortp)) { ok = false; break; }
        for (int it = 0; it < w.nit && ok; ++it) {
          const int gs = g + it, st = gs % NST, st1 = (gs + 1) % NST;
          const uint32_t ph = (uint32_t)gs & 1u;
          const bool more = it + 1 < w.nit;
          if (!mbar_wait(bar_p(x), ph, abortp)) { ok = false; break; }
          tc_fence_after();
          // dV += P^T(x) dO(x), dK += dS^T(x) Q(x): contraction over the half's 64 queries (MN-major B: 16 queries = 2048 B)
          const uint32_t so = (uint32_t)st * STAGE + (uint32_t)x * (TK * 128);
#pragma unroll
          for (int ks = 0; ks < TK / 16; ++ks) {
            const uint32_t acc = (it | x | ks) ? 1u : 0u;
            umma_bf16_ts(tmem_base + C::C_DV, tmem_base + C::C_S + 64 * x + 16 * ks, desc_at(ddo_mn, so + ks * 2048), idesc_g, acc);
            umma_bf16_ts(tmem_base + C::C_DK, tmem_base + C::C_DP + 64 * x + 16 * ks, desc_at(dq_mn, so + ks * 2048), idesc_g, acc);
          }
          if (x == 0 && it == 0) umma_commit(bar_init);
          umma_commit(bar_empty(st));                       // (one of two arrivals) the stage's tiles have been read by this half
          if (more) {
            if (!mbar_wait(bar_full(st1), (uint32_t)((gs + 1) / NST) & 1u, abortp)) { ok = false; break; }
            tc_fence_after();
            issue_scores(st1);
          } else {
            umma_commit(bar_kvfree);                        // (one of three) nothing of this item reads K / V from this thread any more
            umma_commit(bar_acc);                           // (one of two) this half's share of dV / dK is complete
          }
        }
        g += w.nit;
      }
      if (!ok) { fail = 1; abort_flag = 1; }
      umma_commit(bar_drain(x));                   // every MMA this thread issued has retired before TMEM goes
      int never = 0;
      mbar_wait(bar_drain(x), 0, &never);
    }
  } else if (warp == 22) {
    // ---------------------------------------------------------------- MMA issue, third thread: dQ
    if (lane == 0) {
      constexpr uint32_t idesc_q = make_idesc_bf16(TQ, DH, 1, 1);          // A = dS (MN-major), B = K (MN-major)
      const SmemDescBase dk_mn = make_smem_desc_base(sK, TQ * 128, 1024);
      const SmemDescBase dds_mn = make_smem_desc_base(sDS, TQ * 128, 1024);
      bool ok = true;
      int g = 0, n_item = 0;
      for (int item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++n_item) {
        const FusedItem w = fused_item(item, nbh, H, B, nq);
        if (!mbar_wait(bar_kv, (uint32_t)n_item & 1u, abortp)) { ok = false; break; }     // this item's K is in place
        for (int it = 0; it < w.nit && ok; ++it) {
          const int gs = g + it, b = gs & 1;
          // dQ(step) = dS K over this tile's 128 keys: both halves of dS are in shared memory (bar_ds; the item's K
          // arrived before the scores that dS came from), buffer b of the accumulator is free once the flush of
          // step gs-2 is done
          if (!mbar_wait(bar_ds, (uint32_t)gs & 1u, abortp)) { ok = false; break; }
          if (gs >= 2 && !mbar_wait(bar_dqfree(b), (uint32_t)((gs >> 1) - 1) & 1u, abortp)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < TQ / 16; ++ks)
            umma_bf16(tmem_base + C::C_DQ + 64 * b, desc_at(dds_mn, (uint32_t)b * C::DS_BYTES + ks * 2048), desc_at(dk_mn, ks * 2048),
                      idesc_q, ks ? 1u : 0u);
          umma_commit(bar_dq(b));
          if (it + 1 == w.nit) umma_commit(bar_kvfree);      // (one of three)
        }
        g += w.nit;
      }
      if (!ok) { fail = 1; abort_flag = 1; }
      umma_commit(bar_drain(2));
      int never = 0;
      mbar_wait(bar_drain(2), 0, &never);
    }
  } else if (warp >= 16 && warp < 20) {
    // ---------------------------------------------------------------- dQ flush and dV / dK store (warps 16-19: thread = row)
    const int r = tid - 512;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    // The four flush warps meet at a named barrier inside every step, so they must leave the loops together: the
    // outcome of a wait is agreed on (through a shared flag and that barrier) before anyone acts on it.
    auto all_ok = [&](int got) -> bool {
      if (!got) flush_fail = 1;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      return flush_fail == 0;
    };
    int g = 0, n_item = 0;
    for (int item = blockIdx.x; item < nitems && !fail; item += gridDim.x, ++n_item) {
      const FusedItem w = fused_item(item, nbh, H, B, nq);
      for (int it = 0; it < w.nit; ++it) {
        const int gs = g + it, b = gs & 1;
        int got = 1;
        if (lane == 0) got = mbar_wait(bar_dq(b), (uint32_t)(gs >> 1) & 1u, abortp) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        if (!all_ok(got)) { fail = 1; abort_flag = 1; break; }
        tc_fence_after();
        // The block goes to the global accumulator as one bulk reduction per 32 columns: the rows are staged in the
        // dS buffer of this step (its dQ product, the only reader, has retired) in the 128-byte-swizzled layout of
        // the tensor map, and one thread issues cp.reduce.async.bulk.tensor (rows past the sequence end are dropped
        // by the map's bounds).
        const uint32_t stage = sDS + (uint32_t)b * C::DS_BYTES;
#pragma unroll
        for (int c0 = 0; c0 < DH; c0 += 32) {
          uint32_t rr[32];
          tmem_ld_32x32(t_lane + C::C_DQ + 64 * b + c0, rr);
          tmem_ld_wait();
          const uint32_t rowaddr = stage + (uint32_t)(c0 / 32) * (TQ * 128) + (uint32_t)r * 128;
#pragma unroll
          for (int t = 0; t < 8; ++t)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rowaddr + (((uint32_t)t ^ (uint32_t)(r & 7)) * 16)), "r"(rr[4 * t]),
                         "r"(rr[4 * t + 1]), "r"(rr[4 * t + 2]), "r"(rr[4 * t + 3])
                         : "memory");
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_dqfree(b));               // the TMEM buffer has been read
        fence_proxy_async();
        asm volatile("bar.sync 1, 128;" ::: "memory");           // the four flush warps: the block is staged
        if (r == 0) {
#pragma unroll
          for (int c0 = 0; c0 < DH; c0 += 32)
            tma_reduce_add_3d(&tmAcc, stage + (uint32_t)(c0 / 32) * (TQ * 128), w.h * DH + c0, (w.kb + it) * TQ, w.nb);
          bulk_commit_group();
          bulk_wait_group_read0();                               // the staging has been read: the buffer may be rewritten
          mbar_arrive(bar_dsfree(b));
        }
      }
      if (fail) break;
      g += w.nit;
      // the item's dV and dK: this thread's key row, scaled and rounded to bf16
      {
        int got = 1;
        if (lane == 0) got = mbar_wait(bar_acc, (uint32_t)n_item & 1u, abortp) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        if (!all_ok(got)) { fail = 1; abort_flag = 1; break; }
      }
      tc_fence_after();
      const int key = w.kb * TQ + r;
      bf16* rowp = dqkv + ((size_t)w.nb * T + key) * (3 * d) + w.h * DH;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        bf16* dst = rowp + (which == 0 ? 2 * d : d);
        const float f = which == 0 ? 1.0f : scale;
        const uint32_t tcol = t_lane + (which == 0 ? C::C_DV : C::C_DK);
#pragma unroll
        for (int c0 = 0; c0 < DH; c0 += 32) {
          uint32_t rr[32];
          tmem_ld_32x32(tcol + c0, rr);
          tmem_ld_wait();
          if (key < T) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 pk;
              pk.x = pack_bf16x2(__uint_as_float(rr[i]) * f, __uint_as_float(rr[i + 1]) * f);
              pk.y = pack_bf16x2(__uint_as_float(rr[i + 2]) * f, __uint_as_float(rr[i + 3]) * f);
              pk.z = pack_bf16x2(__uint_as_float(rr[i + 4]) * f, __uint_as_float(rr[i + 5]) * f);
              pk.w = pack_bf16x2(__uint_as_float(rr[i + 6]) * f, __uint_as_float(rr[i + 7]) * f);
              *reinterpret_cast<uint4*>(dst + c0 + i) = pk;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_accfree);               // the accumulators may be overwritten by the next item
    }
    if (r == 0) bulk_wait_group0();                            // every reduction this thread issued has reached memory
  } else if (warp < FUSED_RW) {
    // ---------------------------------------------------------------- recompute and convert (warps 0-15)
    // thread (r, sub): key row r, query columns [16 sub, 16 sub + 16) of each 64-column half
    const int r = tid & 127, sub = tid >> 7;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    auto wait = [&](uint32_t bar, uint32_t parity) -> bool {     // lane 0 polls, the warp learns the outcome
      int got = 1;
      if (lane == 0) got = mbar_wait(bar, parity, abortp) ? 1 : 0;
      return __shfl_sync(0xffffffffu, got, 0) != 0;
    };
    int g = 0;
    for (int item = blockIdx.x; item < nitems && !fail; item += gridDim.x) {
      const FusedItem w = fused_item(item, nbh, H, B, nq);
      const int key = w.kb * TQ + r;
      for (int it = 0; it < w.nit && !fail; ++it) {
        const int gs = g + it, st = gs % NST, b = gs & 1, j = w.kb + it;
        const uint32_t ph = (uint32_t)gs & 1u;
        const float* vec = s_vec + st * (2 * TQ);
        // the stage's lse / delta vectors have their own barrier; the dS buffer of this step is free once the dQ
        // block of step gs-2, staged in it after its product, has been handed to the bulk reduction
        if (!wait(bar_vec(st), (uint32_t)(gs / NST) & 1u)) { fail = 1; abort_flag = 1; break; }
        if (gs >= 2 && !wait(bar_dsfree(b), (uint32_t)((gs >> 1) - 1) & 1u)) { fail = 1; abort_flag = 1; break; }
        const bool diag = (it == 0);                       // some queries of this block precede some keys of this tile
        const bool tail = (j * TQ + TQ > T);
        for (int x = 0; x < 2; ++x) {
          if (!wait(bar_s(x), ph)) { fail = 1; abort_flag = 1; break; }
          tc_fence_after();
          uint32_t r0[16], r1[16];
          tmem_ld_32x16(t_lane + C::C_S + 64 * x + 16 * sub, r0);
          tmem_ld_32x16(t_lane + C::C_DP + 64 * x + 16 * sub, r1);
          tmem_ld_wait();
          float p[16], ds[16];
          const float4* lv = reinterpret_cast<const float4*>(vec + 64 * x + 16 * sub);
          const float4* dv_ = reinterpret_cast<const float4*>(vec + TQ + 64 * x + 16 * sub);
          const int qbase = j * TQ + 64 * x + 16 * sub;
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            const float4 l4 = lv[i4], d4 = dv_[i4];
            const float ll[4] = {l4.x, l4.y, l4.z, l4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int i = 4 * i4 + e;
              p[i] = ex2_fast(fmaf(__uint_as_float(r0[i]), c2, -ll[e]));
              ds[i] = __uint_as_float(r1[i]) - dd[e];
            }
          }
          if (diag || tail) {                              // uniform across the CTA
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (qbase + i < key || qbase + i >= T) p[i] = 0.f;
          }
          uint32_t pw[8], dw[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            pw[i] = pack_bf16x2(p[2 * i], p[2 * i + 1]);
            dw[i] = pack_bf16x2(ds[2 * i] * p[2 * i], ds[2 * i + 1] * p[2 * i + 1]);
          }
          tmem_st_32x8(t_lane + C::C_S + 64 * x + 16 * sub, pw);      // P^T over the first half of the columns this thread read
          tmem_st_32x8(t_lane + C::C_DP + 64 * x + 16 * sub, dw);     // dS^T likewise
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p(x));                       // dV / dK of this half can go
          // dS as the A operand of dQ = dS K: row = key, 64 queries of half x = one swizzled 128-byte row of chunk x
          {
            const uint32_t rowaddr = sDS + (uint32_t)b * C::DS_BYTES + (uint32_t)x * (TQ * 128) + (uint32_t)r * 128;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              const uint32_t unit = (uint32_t)(2 * sub + t) ^ (uint32_t)(r & 7);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rowaddr + unit * 16), "r"(dw[4 * t]), "r"(dw[4 * t + 1]),
                           "r"(dw[4 * t + 2]), "r"(dw[4 * t + 3])
                           : "memory");
            }
          }
          if (x == 1) {
            fence_proxy_async();                             // both halves' dS rows are read by the tensor pipe (async proxy)
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ds);
          }
        }
      }
      if (fail) break;
      g += w.nit;
    }
  }
  fail = __syncthreads_or(fail);
  if (tid == 0 && fail && err) atomicExch(err, DEV_TIMEOUT_MMA);
  tc_fence_before();
  __syncthreads();
  if (warp == 20) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// dqkv[row, h*dh + c] (the Q third) = bf16(scale * dq_acc[row, h*dh + c]): the accumulated dQ leaves fp32 here.
__global__ void __launch_bounds__(256) attn_dq_convert_kernel(const float* __restrict__ acc, bf16* __restrict__ dqkv, size_t rows,
                                                              int d, float scale) {
  grid_dep_sync();
  const int d8 = d >> 3;
  const size_t total = rows * (size_t)d8;
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (size_t)gridDim.x * 256) {
    const size_t row = i / d8;
    const int c = (int)(i % d8) * 8;
    const float4 a = *reinterpret_cast<const float4*>(acc + row * d + c);
    const float4 b = *reinterpret_cast<const float4*>(acc + row * d + c + 4);
    uint4 o;
    o.x = pack_bf16x2(a.x * scale, a.y * scale);
    o.y = pack_bf16x2(a.z * scale, a.w * scale);
    o.z = pack_bf16x2(b.x * scale, b.y * scale);
    o.w = pack_bf16x2(b.z * scale, b.w * scale);
    *reinterpret_cast<uint4*>(dqkv + row * (size_t)(3 * d) + c) = o;
  }
}

// delta[nb, h, t] = sum_c dO[nb*T+t, h*dh+c] * O[(nb%B)*T+t, h*dh+c].  A thread takes 8 consecutive columns
// (16 bytes of each operand); the dh/8 threads of a (row, head) sit in one warp and combine by shuffles.
// With dq_zero != NULL the same threads also clear their 8 columns of the fp32 dQ accumulator [NB*T, H*dh] that the
// one-sweep backward adds into.
template <int DH>
__global__ void __launch_bounds__(256) attn_delta_tc_kernel(const bf16* __restrict__ dout, const bf16* __restrict__ o,
                                                            float* __restrict__ delta, float* __restrict__ dq_zero, int NB,
                                                            int B, int T, int H) {
  grid_dep_sync();
  constexpr int TPR = (DH == 80) ? 16 : DH / 8;      // threads per (row, head): a power of two (dh 80: 10 of 16 active)
  const long long gid = (long long)blockIdx.x * 256 + threadIdx.x;
  const long long item = gid / TPR;                  // (row, head) index
  const int part = (int)(gid % TPR);
  const long long total = (long long)NB * T * H;
  float s = 0.f;
  int h = 0;
  long long row = 0;
  if (item < total) {
    h = (int)(item % H);
    row = item / H;
    const int nb = (int)(row / T), t = (int)(row % T);
    if (part * 8 < DH) {
      const int d = H * DH;
      if (dq_zero) {
        float4* z = reinterpret_cast<float4*>(dq_zero + (size_t)row * d + h * DH + part * 8);
        z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      const uint4 a = *reinterpret_cast<const uint4*>(dout + (size_t)row * d + h * DH + part * 8);
      const uint4 c = *reinterpret_cast<const uint4*>(o + ((size_t)(nb % B) * T + t) * d + h * DH + part * 8);
      const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* c2 = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 x = __bfloat1622float2(a2[i]), y = __bfloat1622float2(c2[i]);
        s += x.x * y.x + x.y * y.y;
      }
    }
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (item < total && part == 0) {
    const int nb = (int)(row / T), t = (int)(row % T);
    delta[((size_t)nb * H + h) * T + t] = s;
  }
}

template <int DH>
cudaError_t bwd_tc_launch(const bf16* qkv, const bf16* o, const float* lse, const bf16* dout, bf16* dqkv, float* delta, int NB,
                          int B, int T, int H, unsigned* err, cudaStream_t s) {
  using C = BwdCfg<DH>;
  const unsigned long long d3 = 3ull * H * DH, d1 = (unsigned long long)H * DH;
  const unsigned long long dims[4] = {(unsigned long long)DH, 3ull * H, (unsigned long long)T, (unsigned long long)B};
  const unsigned long long strides[3] = {(unsigned long long)DH * 2, d3 * 2, (unsigned long long)T * d3 * 2};
  const unsigned long long ddims[4] = {(unsigned long long)DH, (unsigned long long)H, (unsigned long long)T, (unsigned long long)NB};
  const unsigned long long dstrides[3] = {(unsigned long long)DH * 2, d1 * 2, (unsigned long long)T * d1 * 2};
  const unsigned box128[4] = {64, 1, TQ, 1}, box64[4] = {64, 1, TK, 1};
  CUtensorMap tmRow, tmBlk, tmdO64, tmdO128;
  if (!tma_encode_bf16(&tmRow, qkv, 4, dims, strides, box128) || !tma_encode_bf16(&tmBlk, qkv, 4, dims, strides, box64) ||
      !tma_encode_bf16(&tmdO64, dout, 4, ddims, dstrides, box64) || !tma_encode_bf16(&tmdO128, dout, 4, ddims, dstrides, box128))
    return cudaErrorInvalidValue;
  constexpr bool SPLIT = 128 + 2 * DH > 512;      // dV and dK accumulators do not fit TMEM together: one launch each
  cudaError_t e = cudaSuccess;
  if constexpr (SPLIT) {
    e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel<DH, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_KV);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel<DH, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_KV);
  } else {
    e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel<DH, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_KV);
  }
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_bwd_dq_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_Q);
  if (e != cudaSuccess) return e;
  constexpr int TPR = (DH == 80) ? 16 : DH / 8;
  const long long nthreads = (long long)NB * T * H * TPR;
  launch_dep(attn_delta_tc_kernel<DH>, dim3((unsigned)((nthreads + 255) / 256)), dim3(256), 0, s, dout, o, delta, nullptr, NB, B, T, H);
  dim3 grid((T + TQ - 1) / TQ, NB * H);
  const float scale = rsqrtf((float)DH);
  if constexpr (SPLIT) {
    launch_dep(attn_bwd_dkv_tc_kernel<DH, 1>, dim3(grid), dim3(256), C::SMEM_KV, s, tmRow, tmBlk, tmdO64, lse, delta, dqkv, B, T, H, scale, err);
    launch_dep(attn_bwd_dkv_tc_kernel<DH, 2>, dim3(grid), dim3(256), C::SMEM_KV, s, tmRow, tmBlk, tmdO64, lse, delta, dqkv, B, T, H, scale, err);
  } else {
    launch_dep(attn_bwd_dkv_tc_kernel<DH, 0>, dim3(grid), dim3(256), C::SMEM_KV, s, tmRow, tmBlk, tmdO64, lse, delta, dqkv, B, T, H, scale, err);
  }
  launch_dep(attn_bwd_dq_tc_kernel<DH>, dim3(grid), dim3(256), C::SMEM_Q, s, tmRow, tmBlk, tmdO128, lse, delta, dqkv, B, T, H, scale, err);
  return cudaGetLastError();
}

// One-sweep backward: delta (+ clearing the accumulator), the sweep, then dQ from fp32 to bf16.
template <int DH>
cudaError_t bwd_fused_launch(const bf16* qkv, const bf16* o, const float* lse, const bf16* dout, bf16* dqkv, float* delta,
                             float* dq_acc, int NB, int B, int T, int H, unsigned* err, cudaStream_t s) {
  using C = FusedCfg<DH>;
  const unsigned long long d3 = 3ull * H * DH, d1 = (unsigned long long)H * DH;
  const unsigned long long dims[4] = {(unsigned long long)DH, 3ull * H, (unsigned long long)T, (unsigned long long)B};
  const unsigned long long strides[3] = {(unsigned long long)DH * 2, d3 * 2, (unsigned long long)T * d3 * 2};
  const unsigned long long ddims[4] = {(unsigned long long)DH, (unsigned long long)H, (unsigned long long)T, (unsigned long long)NB};
  const unsigned long long dstrides[3] = {(unsigned long long)DH * 2, d1 * 2, (unsigned long long)T * d1 * 2};
  const unsigned box128[4] = {64, 1, TQ, 1};
  CUtensorMap tmRow, tmdO, tmAcc;
  if (!tma_encode_bf16(&tmRow, qkv, 4, dims, strides, box128) || !tma_encode_bf16(&tmdO, dout, 4, ddims, dstrides, box128))
    return cudaErrorInvalidValue;
  // the fp32 dQ accumulator [NB, T, d] as the target of the bulk reductions: boxes of 32 columns x 128 rows of one sequence
  const unsigned long long adims[3] = {d1, (unsigned long long)T, (unsigned long long)NB};
  const unsigned long long astrides[2] = {d1 * 4, (unsigned long long)T * d1 * 4};
  const unsigned abox[3] = {32, TQ, 1};
  if (!tma_encode_f32(&tmAcc, dq_acc, 3, adims, astrides, abox)) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_fused_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return e;
  constexpr int TPR = DH / 8;
  const long long nthreads = (long long)NB * T * H * TPR;
  launch_dep(attn_delta_tc_kernel<DH>, dim3((unsigned)((nthreads + 255) / 256)), dim3(256), 0, s, dout, o, delta, dq_acc, NB, B, T, H);
  // persistent CTAs, one per SM, each walking its share of the (key tile, sequence, head) items
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const long long nitems = (long long)((T + TQ - 1) / TQ) * NB * H;
  const int grid = (int)(nitems < sms ? nitems : sms);
  const float scale = rsqrtf((float)DH);
  launch_dep(attn_bwd_fused_kernel<DH>, dim3(grid), dim3(FUSED_THREADS), C::SMEM, s, tmRow, tmdO, tmAcc, lse, delta, dqkv, NB, B, T, H, scale, err);
  const size_t rows = (size_t)NB * T;
  size_t blocks = (rows * (size_t)(H * DH / 8) + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  launch_dep(attn_dq_convert_kernel, dim3((unsigned)blocks), dim3(256), 0, s, dq_acc, dqkv, rows, H * DH, scale);
  return cudaGetLastError();
}

}  // namespace

cudaError_t attention_fwd(const bf16* qkv, bf16* o, float* lse, int B, int T, int H, int dh, unsigned* err,
                          cudaStream_t s) {
  if (((uintptr_t)qkv % 16) || ((uintptr_t)o % 16) || ((uintptr_t)lse % 4)) return cudaErrorInvalidValue;
  switch (dh) {
    case 32: return fwd_tc_launch<32>(qkv, o, lse, B, T, H, err, s);
    case 64: return fwd_tc_launch<64>(qkv, o, lse, B, T, H, err, s);
    case 80: return fwd_tc_launch<80>(qkv, o, lse, B, T, H, err, s);
    case 128: return fwd_tc_launch<128>(qkv, o, lse, B, T, H, err, s);
    case 256: return fwd_tc_launch<256>(qkv, o, lse, B, T, H, err, s);
  }
  return cudaErrorInvalidValue;
}

cudaError_t attention_bwd(const bf16* qkv, const bf16* o, const float* lse, const bf16* dout, bf16* dqkv, float* delta,
                          float* dq_acc, int NB, int B, int T, int H, int dh, unsigned* err, cudaStream_t s) {
  // o is read with 16-byte loads by the delta kernel, qkv / dout / dqkv by TMA and 16-byte stores
  if (((uintptr_t)qkv % 16) || ((uintptr_t)o % 16) || ((uintptr_t)dout % 16) || ((uintptr_t)dqkv % 16) ||
      ((uintptr_t)lse % 4) || ((uintptr_t)delta % 4))
    return cudaErrorInvalidValue;
  if (dq_acc && (dh == 32 || dh == 64)) {        // one sweep, dQ summed over key tiles in the fp32 accumulator
    if ((uintptr_t)dq_acc % 16) return cudaErrorInvalidValue;
    return dh == 32 ? bwd_fused_launch<32>(qkv, o, lse, dout, dqkv, delta, dq_acc, NB, B, T, H, err, s)
                    : bwd_fused_launch<64>(qkv, o, lse, dout, dqkv, delta, dq_acc, NB, B, T, H, err, s);
  }
  switch (dh) {
    case 32: return bwd_tc_launch<32>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, err, s);
    case 64: return bwd_tc_launch<64>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, err, s);
    case 80: return bwd_tc_launch<80>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, err, s);
    case 128: return bwd_tc_launch<128>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, err, s);
    case 256: return bwd_tc_launch<256>(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, err, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace il

