// C ABI and host runtime of the n-wise training step: parameter registry, activation arena, one CUDA
// stream per component with event dependencies, and the bookkeeping of the gradient streams of the
// n-wise rule (Sec. 3, Fig. 2 of the paper).
//
// Gradient streams.  Head h (0-based) back-propagates through components h, h-1, ..., term(h) with
// term(h) = max(h-n+1, 0) and is dropped at the input of component term(h).  Back-propagation is linear
// in the incoming gradient, so component k does not carry one tensor per head but one per distinct
// termination level among the heads crossing it, as cumulative sums
//     U_j = sum of the gradients of heads h crossing k with term(h) <= t_j,   t_0 > t_1 > ...
// U_0 is the sum over all crossing heads: the parameter gradients of component k come from U_0 alone (one
// wgrad per matrix), and the U_j are stacked along the token axis so that each dgrad GEMM / attention
// backward / LayerNorm backward of the component runs once on s_k * Ntok rows.  At the boundary below,
// the stream that terminates is dropped, the own head's gradient is added to every remaining stream.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <new>
#include <cstdio>
#include <cstring>
#include <string>
#include <utility>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/il.h"
#include "../../include/il_ops.h"
#include "common.cuh"
#include "gemm.h"
#include "kernels.h"

using namespace il;

namespace {


struct TensorRec {
  std::string name;
  int component, is_head, rank;
  long long shape[2];
  size_t off, count;
};

struct LayerOff { size_t ln1g, ln1b, wqkv, bqkv, wo, bo, ln2g, ln2b, w1, b1, w2, b2; };
struct HeadOff { size_t lng, lnb, w; };

struct LayerActs {
  bf16 *ln1, *qkv, *attn_o, *ln2, *hgrad, *hact;   // hgrad = gelu'(FC1 pre-activation)
  float *mean1, *rstd1, *lse, *x_mid, *mean2, *rstd2, *x_out;
};

struct CompScratch {     // backward scratch of one component, rows = s_cap * ntok_max
  float* dx; bf16* dxb; bf16* dbig; bf16* dln; bf16* dattn; bf16* dqkv; float* delta;
};
struct HeadScratch {
  bf16* u; float *mean, *rstd, *pmax, *psum, *tgt_logit, *lse, *nll, *du, *ghead;
  bf16* z;   // stored mode: [Ntok, ldz] exp(logits) kept by the loss pass, the backward patches the target column in
             // place; recompute mode: [Ntok, chunk] dZ of one vocabulary chunk
  bf16* us;  // [Ntok, d]: rows of u scaled by exp(-lse) / Ntok (stored mode)
  float* rs; // [Ntok]: exp(-lse) / Ntok (stored mode)
};

struct ProfRec { cudaEvent_t a, b; double flops; };

// Named range on the host timeline of a profiler (NVTX; costs nothing when no tool is attached): one per call of
// the step and, inside the backward, one per component, so that a trace shows which launches belong to which
// component and phase.
struct Range {
  explicit Range(const char* fmt, int k = -1) {
    char buf[64];
    snprintf(buf, sizeof buf, fmt, k);
    nvtxRangePushA(buf);
  }
  ~Range() { nvtxRangePop(); }
};

}  // namespace

struct il_model {
  int K, Lc, d, H, F, V, n, dh;
  int Lh;                             // Transformer blocks inside every auxiliary head (0 = LayerNorm + linear)
  int micro, micro_done;              // micro-batches per update, backward passes since the last update
  int rule;                           // IL_RULE_*: which heads update a component's parameters
  int head_mode;                      // IL_HEAD_STORED / IL_HEAD_RECOMPUTE
  int attn_bwd;                       // IL_ATTN_BWD_ONE_SWEEP / IL_ATTN_BWD_TWO_KERNELS
  int placement;                      // IL_PLACE_SINGLE / IL_PLACE_PIPELINE
  std::vector<int> dev;               // device of component k (all equal to `device` unless placed as a pipeline)
  std::vector<int> dev_list;          // the distinct devices in use
  std::vector<int> sms;               // SM count of component k's device
  int device, num_sms;
  int max_batch, max_seq, ntok_max;
  float ln_eps;
  il_options opt;
  bool own_streams;
  std::vector<cudaStream_t> streams;
  std::vector<cudaEvent_t> ev_fwd, ev_bwd, ev_join;
  // The vocabulary matrix of head k is final as soon as the head's own backward is: its optimiser update runs on a
  // side stream that waits for that point only (ev_head), beside the component's backward.
  std::vector<cudaStream_t> side;
  std::vector<cudaEvent_t> ev_head, ev_side;
  cudaEvent_t ev_batch;
  // parameters
  std::vector<TensorRec> tensors;
  std::vector<LayerOff> layer_off;   // K*Lc main layers, then K*Lh head layers (head k's at K*Lc + k*Lh)
  std::vector<HeadOff> head_off;     // K
  size_t off_wte, off_wpe;
  std::vector<size_t> comp_begin, comp_mat_end, comp_end;   // flat ranges per component
  size_t total;
  // Per-component views of the parameter, gradient, Adam and bf16-shadow storage, biased so that view[k] + off is
  // the element at flat offset `off` for every off in [comp_begin[k], comp_end[k]).  One flat buffer on a single
  // device (all views equal); one buffer per component, on that component's device, in the pipeline placement.
  std::vector<float*> P, G, M1, M2;
  std::vector<bf16*> Pb;
  long long step;
  int adamw_issued;                   // il_adamw_step calls since the last il_sync
  // activations
  std::vector<float*> a;             // K+1 boundaries; a[k+1] aliases the last layer's x_out
  std::vector<LayerActs> acts;       // same indexing as layer_off
  std::vector<CompScratch> cs;
  std::vector<HeadScratch> hs;
  int s_cap;
  std::vector<int*> tokens, targets;  // per component: the batch on that component's device (shared on one device)
  std::vector<float*> losses;         // per component: device [K] array holding losses[k] at index k
  // Error words, per component (shared on one device): word 0 = DEV_* code of the first failure, words 1..K =
  // number of AdamW updates component k-1 applied since the last il_sync (an update is skipped while word 0 is set).
  std::vector<unsigned*> err_word;
  // pipeline placement: receive buffers owned by the component's device
  std::vector<float*> a_in;           // a_{k}: input of component k (k >= 1), copied from component k-1's output
  std::vector<float*> g_in;           // [s_cap, Ntok, d]: gradient streams passed down from component k+1
  std::vector<cudaEvent_t> ev_copy;   // per component: last copy into its receive buffers
  std::vector<int> xfer_log;          // pipeline placement: (direction, boundary, id) of every copy of the current step
  std::vector<unsigned*> sort_keys;   // [0]: scratch of the deterministic embedding backward on component 0's device
  int part_ld;
  int ldz;                            // stored mode: row stride of exp(logits) (vocabulary rounded up to 64)
  int head_chunk;                     // recompute mode: columns per vocabulary chunk = row stride of the dZ chunk
  // step state
  int B, T, ntok;
  bool batch_set, bwd_done;
  std::vector<char> fwd_done, loss_done;
  // allocations
  std::vector<std::pair<void*, int>> allocs;   // (pointer, device it was obtained on)
  std::vector<size_t> alloc_bytes;
  long long bytes, launches;
  // profiling
  int prof;                           // 0 off, 1 events around each GEMM, 2 the same with the GEMM alone on the GPU
  std::vector<ProfRec> prof_recs;
  std::vector<cudaEvent_t> prof_pool;
  std::string err;
};

namespace {

il_status fail(il_model* m, il_status s, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (m) m->err = buf;
  return s;
}

#define IL_CUDA(m, call)                                                                            \
  do {                                                                                              \
    cudaError_t e__ = (call);                                                                       \
    if (e__ != cudaSuccess)                                                                         \
      return fail(m, IL_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e__), __FILE__, __LINE__); \
  } while (0)
#define IL_TRY(call)                      \
  do {                                    \
    il_status s__ = (call);               \
    if (s__ != IL_OK) return s__;         \
  } while (0)

// Nothing may throw across the C boundary: every exported function runs its body through this.  Host containers
// (the tensor registry, stream bookkeeping, the error string) can raise std::bad_alloc.
template <class F>
il_status guarded(F&& body) noexcept {
  try {
    return body();
  } catch (const std::bad_alloc&) {
    return IL_ERR_OOM;
  } catch (...) {
    return IL_ERR_CUDA;
  }
}

il_status dev_alloc(il_model* m, void** out, size_t bytes) {
  bytes = (bytes + 255) & ~size_t(255);
  if (bytes == 0) bytes = 256;
  void* p = nullptr;
  if (m->opt.alloc) {
    p = m->opt.alloc(bytes, m->opt.alloc_ctx);
  } else {
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); p = nullptr; }
  }
  if (!p) return fail(m, IL_ERR_OOM, "device allocation of %zu bytes failed", bytes);
  if ((uintptr_t)p % 256) return fail(m, IL_ERR_INVALID_ARG, "allocator returned a pointer that is not 256-byte aligned");
  int cur = 0;
  cudaGetDevice(&cur);
  m->allocs.push_back(std::make_pair(p, cur));
  m->alloc_bytes.push_back(bytes);
  m->bytes += (long long)bytes;
  *out = p;
  return IL_OK;
}
// Hand one allocation back (the device it came from is made current for the hook).
void dev_free(il_model* m, void* p) {
  if (!p) return;
  for (size_t i = 0; i < m->allocs.size(); ++i)
    if (m->allocs[i].first == p) {
      cudaSetDevice(m->allocs[i].second);
      if (m->opt.free_) m->opt.free_(p, m->opt.alloc_ctx);
      else cudaFree(p);
      m->bytes -= (long long)m->alloc_bytes[i];
      m->allocs.erase(m->allocs.begin() + i);
      m->alloc_bytes.erase(m->alloc_bytes.begin() + i);
      return;
    }
}
template <typename T>
il_status dev_alloc_t(il_model* m, T** out, size_t count) {
  void* p;
  IL_TRY(dev_alloc(m, &p, count * sizeof(T)));
  *out = reinterpret_cast<T*>(p);
  return IL_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Vocabulary columns per chunk of the recompute head mode (a multiple of the 256-column output tile).
constexpr int HEAD_CHUNK = 8192;

// termination level of head h under the n-wise rule
inline int term_of(int h, int n) { return h - n + 1 > 0 ? h - n + 1 : 0; }
// distinct termination levels of the heads crossing component k, descending
std::vector<int> terms_of(int k, int K, int n) {
  std::vector<int> t;
  const int hi = k + n - 1 < K - 1 ? k + n - 1 : K - 1;
  for (int h = hi; h >= k; --h) {
    const int th = term_of(h, n);
    if (t.empty() || t.back() != th) t.push_back(th);
  }
  return t;
}
int s_cap_for(int K, int n) {
  size_t s = 1;
  for (int k = 0; k < K; ++k) s = std::max(s, terms_of(k, K, n).size());
  return (int)s;
}

// weight of head h's gradient in the parameter update of component k (k <= h <= min(k+n-1, K-1))
float rule_weight(int rule, int k, int h, int n, int K) {
  const int far = k + n - 1 < K - 1 ? k + n - 1 : K - 1;
  if (rule == IL_RULE_FAR) return h == far ? 1.0f : 0.0f;
  if (rule == IL_RULE_MEAN) return 0.5f * (h == k) + 0.5f * (h == far);
  return 1.0f;
}

il_status gemm(il_model* m, int k, const GemmArgs& g) {
  cudaStream_t st = m->streams[k];
  ProfRec rec{};
  if (m->prof) {
    for (int i = 0; i < 2; ++i) {
      cudaEvent_t e;
      // (events belong to the device they were created on: the pool is only drawn from on a single device)
      if (!m->prof_pool.empty() && m->dev_list.size() == 1) { e = m->prof_pool.back(); m->prof_pool.pop_back(); }
      else IL_CUDA(m, cudaEventCreate(&e));
      (i == 0 ? rec.a : rec.b) = e;
    }
    rec.flops = 2.0 * g.M * g.N * (double)g.K;
    if (m->prof == 2) {
      // exclusive timing: nothing else of this model runs while the GEMM does, so the event pair measures the
      // kernel and not its wait for SMs held by other components' streams
      for (int j = 0; j < m->K; ++j)
        if (j != k) {
          IL_CUDA(m, cudaEventRecord(m->ev_join[j], m->streams[j]));
          IL_CUDA(m, cudaStreamWaitEvent(st, m->ev_join[j], 0));
        }
    }
    IL_CUDA(m, cudaEventRecord(rec.a, st));
  }
  cudaError_t e = gemm_launch(g, m->err_word[k], m->sms[k], st);
  if (e != cudaSuccess)
    return fail(m, e == cudaErrorInvalidValue ? IL_ERR_INVALID_ARG : IL_ERR_CUDA, "gemm launch (M=%d N=%d K=%d epi=%d): %s",
                g.M, g.N, g.K, g.epilogue, cudaGetErrorString(e));
  if (m->prof) {
    IL_CUDA(m, cudaEventRecord(rec.b, st));
    if (m->prof == 2)
      for (int j = 0; j < m->K; ++j)
        if (j != k) IL_CUDA(m, cudaStreamWaitEvent(m->streams[j], rec.b, 0));
    m->prof_recs.push_back(rec);
  }
  m->launches++;
  return IL_OK;
}

GemmArgs gemm_args(int M, int N, int K, const void* A, int lda, int a_mn, const void* B, int ldb, int b_mn, int epi,
                   void* C, int ldc) {
  GemmArgs g;
  memset(&g, 0, sizeof g);
  g.M = M; g.N = N; g.K = K;
  g.A = {A, lda, a_mn};
  g.B = {B, ldb, b_mn};
  g.epilogue = epi;
  g.C = C; g.ldc = ldc;
  return g;
}

#define IL_K(m, call)                                                                                   \
  do {                                                                                                  \
    cudaError_t e__ = (call);                                                                           \
    if (e__ != cudaSuccess) return fail(m, IL_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__));      \
    (m)->launches++;                                                                                    \
  } while (0)

// Weight-gradient GEMM dW[M,N] = dY^T X over K tokens.  The output has few tiles compared with the number of CTA
// pairs, so the tile width (256 or 512 columns) and the number of work units per tile the token axis is split
// into (partial sums are added atomically into the zeroed gradient) are chosen together, by a small model of
// the kernel: waves of units over the pairs, times the k-slabs of a unit (a 512-wide slab costs 1.72 of a
// 256-wide one) plus the unit's exposed prologue / epilogue.
il_status wgrad(il_model* m, int k, int M, int N, int K, const bf16* dY, int ld_dy, const bf16* X, int ld_x, float* dW,
                bool acc) {
  const int pairs = m->sms[k] / 2;
  const int slabs = (K + 63) / 64;
  int best_nt = 1, best_s = 1;
  double best_cost = 1e300;
  for (int nt = 1; nt <= 2; ++nt) {
    if (nt == 2 && N <= 256) break;
    const int tiles = ((M + 255) / 256) * ((N + 256 * nt - 1) / (256 * nt));
    const double slab_cost = nt == 1 ? 1.0 : 1.72, unit_cost = nt == 1 ? 2.0 : 10.0;
    for (int s = 1; s <= 8; ++s) {
      if (s > 1 && slabs / s < 16) break;
      const int per = (slabs + s - 1) / s;
      const int waves = (tiles * s + pairs - 1) / pairs;
      const double cost = waves * (per * slab_cost + unit_cost) + (s > 1 ? 4.0 : 0.0);   // + zeroing the output
      if (cost < best_cost * 0.97) { best_cost = cost; best_nt = nt; best_s = s; }
    }
  }
  GemmArgs g = gemm_args(M, N, K, dY, ld_dy, 1, X, ld_x, 1, EPI_F32, dW, N);
  g.tile_blocks = best_nt;
  if (best_s > 1) {
    // split units add their partial sums into the output: zero it first, unless this pass adds to the last one's
    if (!acc) IL_CUDA(m, cudaMemsetAsync(dW, 0, (size_t)M * N * sizeof(float), m->streams[k]));
    g.split_k = best_s;
  } else {
    g.accumulate = acc ? 1 : 0;
  }
  return gemm(m, k, g);
}

il_status alloc_scratch(il_model* m, int s_cap) {
  // Backward scratch for s_cap stacked gradient streams per component.  It only grows; a superseded set is handed
  // back before the larger one is obtained (the callers have synchronised the devices).
  if (s_cap <= m->s_cap) return IL_OK;
  const size_t R = (size_t)s_cap * m->ntok_max;
  const int d = m->d, F = m->F;
  for (auto& c : m->cs) {
    dev_free(m, c.dx); dev_free(m, c.dxb); dev_free(m, c.dbig); dev_free(m, c.dln); dev_free(m, c.dattn);
    dev_free(m, c.dqkv); dev_free(m, c.delta);
  }
  for (float* g : m->g_in) dev_free(m, g);
  m->cs.assign(m->K, CompScratch{});
  m->g_in.assign(m->K, nullptr);
  m->s_cap = 0;
  for (int k = 0; k < m->K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    CompScratch& c = m->cs[k];
    IL_TRY(dev_alloc_t(m, &c.dx, R * d));
    IL_TRY(dev_alloc_t(m, &c.dxb, R * d));
    IL_TRY(dev_alloc_t(m, &c.dbig, R * F));
    IL_TRY(dev_alloc_t(m, &c.dln, R * d));
    IL_TRY(dev_alloc_t(m, &c.dattn, R * d));
    IL_TRY(dev_alloc_t(m, &c.dqkv, R * 3 * d));
    IL_TRY(dev_alloc_t(m, &c.delta, R * m->H));
    // pipeline placement: the gradient streams component k+1 passes down land here, in memory of k's device
    if (m->placement == IL_PLACE_PIPELINE && k + 1 < m->K) IL_TRY(dev_alloc_t(m, &m->g_in[k], R * d));
  }
  m->s_cap = s_cap;
  return IL_OK;
}

il_status join_all(il_model* m) {
  // stream 0 waits for every other stream, then everyone waits for stream 0
  for (int k = 1; k < m->K; ++k) {
    IL_CUDA(m, cudaEventRecord(m->ev_join[k], m->streams[k]));
    IL_CUDA(m, cudaStreamWaitEvent(m->streams[0], m->ev_join[k], 0));
  }
  return IL_OK;
}

// input of head k's LayerNorm: the component's output, or the output of the head's own blocks
const float* head_input(const il_model* m, int k) {
  if (m->Lh == 0) return m->a[k + 1];
  return m->acts[(size_t)m->K * m->Lc + (size_t)k * m->Lh + m->Lh - 1].x_out;
}

il_status check_model(const il_model* m) { return m ? IL_OK : IL_ERR_INVALID_ARG; }

// Stream-ordered copy on component k's stream followed by a wait: the data is in place when this returns.
il_status copy_sync(il_model* m, int k, void* dst, const void* src, size_t bytes, cudaMemcpyKind kind) {
  IL_CUDA(m, cudaSetDevice(m->dev[k]));
  IL_CUDA(m, cudaMemcpyAsync(dst, src, bytes, kind, m->streams[k]));
  IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));
  return IL_OK;
}

// Wait for everything enqueued on every device the model uses.
il_status sync_devices(il_model* m) {
  for (int dv : m->dev_list) {
    IL_CUDA(m, cudaSetDevice(dv));
    IL_CUDA(m, cudaDeviceSynchronize());
  }
  return IL_OK;
}

// input of component k: the embeddings (k = 0), the output of component k-1 read in place (single device), or
// this device's copy of it (pipeline placement)
const float* comp_input(const il_model* m, int k) {
  return (m->placement == IL_PLACE_PIPELINE && k > 0) ? m->a_in[k] : m->a[k];
}

}  // namespace

// =================================================================================================
// creation / destruction
// =================================================================================================
extern "C" il_status il_create(int K, int Lc, int d, int H, int F, int V, int n, const il_options* opt, il_model** out) {
  return guarded([&]() -> il_status {
  if (!out) return IL_ERR_INVALID_ARG;
  *out = nullptr;
  if (!opt || K < 1 || K > 64 || Lc < 1 || d < 8 || H < 1 || F < 8 || V < 2 || n < 1 || n > K) return IL_ERR_INVALID_ARG;
  if (opt->head_layers < 0 || opt->head_layers > 64) return IL_ERR_INVALID_ARG;
  if (d % H || d % 8 || F % 8 || opt->max_batch < 1 || opt->max_seq < 1) return IL_ERR_INVALID_ARG;
  const int dh = d / H;
  if (!(dh == 32 || dh == 64 || dh == 80 || dh == 128 || dh == 256)) return IL_ERR_INVALID_ARG;
  if (opt->streams && opt->n_streams < K) return IL_ERR_INVALID_ARG;
  if ((opt->alloc == nullptr) != (opt->free_ == nullptr)) return IL_ERR_INVALID_ARG;
  if (opt->use_bias != 1) return IL_ERR_INVALID_ARG;             // only the GPT-2 form with biases is built
  if (opt->head_mode != IL_HEAD_STORED && opt->head_mode != IL_HEAD_RECOMPUTE) return IL_ERR_INVALID_ARG;
  if (opt->placement != IL_PLACE_SINGLE && opt->placement != IL_PLACE_PIPELINE) return IL_ERR_INVALID_ARG;
  if (opt->attn_bwd != IL_ATTN_BWD_ONE_SWEEP && opt->attn_bwd != IL_ATTN_BWD_TWO_KERNELS) return IL_ERR_INVALID_ARG;
  if (opt->devices && (opt->placement != IL_PLACE_PIPELINE || opt->n_devices != K)) return IL_ERR_INVALID_ARG;

  il_model* m = new (std::nothrow) il_model();
  if (!m) return IL_ERR_OOM;
  m->K = K; m->Lc = Lc; m->d = d; m->H = H; m->F = F; m->V = V; m->n = n; m->dh = dh;
  m->Lh = opt->head_layers; m->micro = 1; m->micro_done = 0;
  m->opt = *opt;
  m->opt.devices = nullptr;            // the caller's array is not kept
  m->device = opt->device;
  m->head_mode = opt->head_mode; m->placement = opt->placement; m->attn_bwd = opt->attn_bwd;
  m->max_batch = opt->max_batch; m->max_seq = opt->max_seq;
  m->ntok_max = opt->max_batch * opt->max_seq;
  m->ln_eps = opt->ln_eps > 0 ? opt->ln_eps : 1e-5f;
  m->rule = IL_RULE_SUM; m->step = 0; m->adamw_issued = 0; m->bytes = 0; m->launches = 0; m->s_cap = 0;
  m->prof = 0; m->batch_set = false; m->bwd_done = false;
  m->B = m->T = m->ntok = 0;
  m->ev_batch = nullptr;
  *out = m;   // returned even on failure below so that il_last_error/il_destroy work

  auto bail = [&](il_status s) { return s; };
  m->dev.assign(K, opt->device);
  if (opt->devices)
    for (int k = 0; k < K; ++k) m->dev[k] = opt->devices[k];
  m->sms.assign(K, 0);
  for (int k = 0; k < K; ++k) {
    if (std::find(m->dev_list.begin(), m->dev_list.end(), m->dev[k]) == m->dev_list.end()) m->dev_list.push_back(m->dev[k]);
    cudaError_t e = cudaSetDevice(m->dev[k]);
    if (e != cudaSuccess) return bail(fail(m, IL_ERR_CUDA, "cudaSetDevice(%d): %s", m->dev[k], cudaGetErrorString(e)));
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, m->dev[k]);
    if (e != cudaSuccess) return bail(fail(m, IL_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(e)));
    if (prop.major != 10) return bail(fail(m, IL_ERR_CUDA, "device %d is sm_%d%d; this library is built for sm_100a only", m->dev[k], prop.major, prop.minor));
    m->sms[k] = prop.multiProcessorCount;
    e = gemm_init();
    if (e != cudaSuccess) return bail(fail(m, IL_ERR_CUDA, "gemm_init: %s", cudaGetErrorString(e)));
  }
  m->num_sms = m->sms[0];
  // Neighbouring devices of the pipeline exchange boundary tensors with cudaMemcpyPeerAsync; with peer access
  // enabled those copies go over NVLink directly instead of through host memory.  Failure to enable it is not an
  // error (the copies still work).
  for (int k = 0; k + 1 < K; ++k)
    if (m->dev[k] != m->dev[k + 1])
      for (int dir = 0; dir < 2; ++dir) {
        const int a = m->dev[k + dir], b = m->dev[k + 1 - dir];
        int can = 0;
        if (cudaDeviceCanAccessPeer(&can, a, b) == cudaSuccess && can) {
          cudaSetDevice(a);
          cudaDeviceEnablePeerAccess(b, 0);
          cudaGetLastError();            // "already enabled" is fine
        }
      }

  // ---- parameter registry and flat layout (per component: matrices first, then vectors)
  auto add = [&](const std::string& name, int comp, int is_head, int rank, long long s0, long long s1) {
    TensorRec t;
    t.name = name; t.component = comp; t.is_head = is_head; t.rank = rank;
    t.shape[0] = s0; t.shape[1] = rank == 2 ? s1 : 1;
    t.count = (size_t)s0 * (rank == 2 ? s1 : 1);
    t.off = 0;
    m->tensors.push_back(t);
    return (int)m->tensors.size() - 1;
  };
  add("wte", 0, 0, 2, V, d);
  add("wpe", 0, 0, 2, m->max_seq, d);
  const char* lnames[12] = {"ln1.g", "ln1.b", "attn.wqkv", "attn.bqkv", "attn.wo", "attn.bo",
                            "ln2.g", "ln2.b", "mlp.w1", "mlp.b1", "mlp.w2", "mlp.b2"};
  const long long ls0[12] = {d, d, 3LL * d, 3LL * d, d, d, d, d, F, F, d, d};
  const long long ls1[12] = {0, 0, d, 0, d, 0, 0, 0, d, 0, F, 0};
  const int Lh = m->Lh;
  for (int k = 0; k < K; ++k)
    for (int l = 0; l < Lc; ++l) {
      char pre[64];
      snprintf(pre, sizeof pre, "c%d.l%d.", k, l);
      for (int i = 0; i < 12; ++i) add(std::string(pre) + lnames[i], k, 0, ls1[i] ? 2 : 1, ls0[i], ls1[i]);
    }
  for (int k = 0; k < K; ++k) {
    char pre[64];
    for (int l = 0; l < Lh; ++l) {       // the auxiliary network's own blocks (App. B.3), same shape as the main ones
      snprintf(pre, sizeof pre, "head%d.l%d.", k, l);
      for (int i = 0; i < 12; ++i) add(std::string(pre) + lnames[i], k, 1, ls1[i] ? 2 : 1, ls0[i], ls1[i]);
    }
    snprintf(pre, sizeof pre, "head%d.", k);
    add(std::string(pre) + "ln.g", k, 1, 1, d, 0);
    add(std::string(pre) + "ln.b", k, 1, 1, d, 0);
    add(std::string(pre) + "w", k, 1, 2, V, d);
  }
  size_t cur = 0;
  m->comp_begin.resize(K); m->comp_mat_end.resize(K); m->comp_end.resize(K);
  for (int k = 0; k < K; ++k) {
    m->comp_begin[k] = cur;
    for (int pass = 0; pass < 2; ++pass) {       // pass 0: rank-2 (decayed), pass 1: rank-1
      for (auto& t : m->tensors)
        if (t.component == k && (t.rank == 2) == (pass == 0)) {
          t.off = cur;
          cur = align_up(cur + t.count, 64);
        }
      if (pass == 0) m->comp_mat_end[k] = cur;
    }
    m->comp_end[k] = cur;
  }
  m->total = cur;
  m->layer_off.resize((size_t)K * (Lc + Lh));
  m->head_off.resize(K);
  {
    size_t i = 0;
    m->off_wte = m->tensors[i++].off;
    m->off_wpe = m->tensors[i++].off;
    auto take_layer = [&](LayerOff& o) {
      o.ln1g = m->tensors[i++].off; o.ln1b = m->tensors[i++].off; o.wqkv = m->tensors[i++].off;
      o.bqkv = m->tensors[i++].off; o.wo = m->tensors[i++].off; o.bo = m->tensors[i++].off;
      o.ln2g = m->tensors[i++].off; o.ln2b = m->tensors[i++].off; o.w1 = m->tensors[i++].off;
      o.b1 = m->tensors[i++].off; o.w2 = m->tensors[i++].off; o.b2 = m->tensors[i++].off;
    };
    for (int kl = 0; kl < K * Lc; ++kl) take_layer(m->layer_off[kl]);
    for (int k = 0; k < K; ++k) {
      for (int l = 0; l < Lh; ++l) take_layer(m->layer_off[(size_t)K * Lc + (size_t)k * Lh + l]);
      HeadOff& o = m->head_off[k];
      o.lng = m->tensors[i++].off; o.lnb = m->tensors[i++].off; o.w = m->tensors[i++].off;
    }
  }

  // ---- streams and events (each on its component's device)
  m->own_streams = (opt->streams == nullptr);
  m->streams.resize(K);
  for (int k = 0; k < K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    if (m->own_streams) {
      cudaError_t e = cudaStreamCreateWithFlags(&m->streams[k], cudaStreamNonBlocking);
      if (e != cudaSuccess) { m->streams.resize(k); return bail(fail(m, IL_ERR_CUDA, "cudaStreamCreate: %s", cudaGetErrorString(e))); }
    } else {
      m->streams[k] = reinterpret_cast<cudaStream_t>(opt->streams[k]);
    }
  }
  auto mk_events = [&](std::vector<cudaEvent_t>& v) -> il_status {
    v.resize(K);
    for (int k = 0; k < K; ++k) {
      IL_CUDA(m, cudaSetDevice(m->dev[k]));
      cudaError_t e = cudaEventCreateWithFlags(&v[k], cudaEventDisableTiming);
      if (e != cudaSuccess) { v.resize(k); return fail(m, IL_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(e)); }
    }
    return IL_OK;
  };
  IL_TRY(mk_events(m->ev_fwd));
  IL_TRY(mk_events(m->ev_bwd));
  IL_TRY(mk_events(m->ev_join));
  IL_TRY(mk_events(m->ev_copy));
  IL_TRY(mk_events(m->ev_head));
  IL_TRY(mk_events(m->ev_side));
  m->side.resize(K);
  for (int k = 0; k < K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    cudaError_t e = cudaStreamCreateWithFlags(&m->side[k], cudaStreamNonBlocking);
    if (e != cudaSuccess) { m->side.resize(k); return bail(fail(m, IL_ERR_CUDA, "cudaStreamCreate: %s", cudaGetErrorString(e))); }
  }
  IL_CUDA(m, cudaSetDevice(m->dev[0]));
  IL_CUDA(m, cudaEventCreateWithFlags(&m->ev_batch, cudaEventDisableTiming));

  // ---- parameter, gradient and optimiser storage
  // All host<->device copies of the library are stream-ordered on the owning component's stream (a synchronous
  // cudaMemcpy from pageable memory may return before its DMA has landed, and the legacy stream does not order
  // against the non-blocking streams used here).
  const bool pipe = m->placement == IL_PLACE_PIPELINE;
  m->P.assign(K, nullptr); m->G.assign(K, nullptr); m->M1.assign(K, nullptr); m->M2.assign(K, nullptr);
  m->Pb.assign(K, nullptr);
  for (int k = 0; k < K; ++k) {
    if (!pipe && k > 0) {   // one flat buffer: every component's view is the same pointer
      m->P[k] = m->P[0]; m->G[k] = m->G[0]; m->M1[k] = m->M1[0]; m->M2[k] = m->M2[0]; m->Pb[k] = m->Pb[0];
      continue;
    }
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    const size_t lo = pipe ? m->comp_begin[k] : 0, cnt = pipe ? m->comp_end[k] - m->comp_begin[k] : m->total;
    float* f[4];
    for (int i = 0; i < 4; ++i) {
      IL_TRY(dev_alloc_t(m, &f[i], cnt));
      IL_CUDA(m, cudaMemsetAsync(f[i], 0, cnt * 4, m->streams[k]));
    }
    bf16* pb;
    IL_TRY(dev_alloc_t(m, &pb, cnt));
    IL_CUDA(m, cudaMemsetAsync(pb, 0, cnt * 2, m->streams[k]));
    m->P[k] = f[0] - lo; m->G[k] = f[1] - lo; m->M1[k] = f[2] - lo; m->M2[k] = f[3] - lo; m->Pb[k] = pb - lo;
  }
  {  // LayerNorm gains start at one
    std::vector<float> ones(d, 1.0f);
    for (auto& t : m->tensors)
      if (t.name.size() >= 2 && t.name.compare(t.name.size() - 2, 2, ".g") == 0) {
        const int k = t.component;
        IL_CUDA(m, cudaSetDevice(m->dev[k]));
        IL_CUDA(m, cudaMemcpyAsync(m->P[k] + t.off, ones.data(), d * 4, cudaMemcpyHostToDevice, m->streams[k]));
        IL_K(m, f32_to_bf16(m->P[k] + t.off, m->Pb[k] + t.off, d, m->streams[k]));
        IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));   // `ones` is pageable host memory
      }
  }

  // ---- activations, on the device of the component that produces them
  const size_t N = m->ntok_max;
  m->a.assign(K + 1, nullptr);
  m->a_in.assign(K, nullptr);
  IL_CUDA(m, cudaSetDevice(m->dev[0]));
  IL_TRY(dev_alloc_t(m, &m->a[0], N * d));
  m->acts.resize((size_t)K * (Lc + Lh));
  for (int k = 0; k < K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    if (pipe && k > 0) IL_TRY(dev_alloc_t(m, &m->a_in[k], N * d));
    for (int l = 0; l < Lc + Lh; ++l) {
      LayerActs& A = l < Lc ? m->acts[(size_t)k * Lc + l] : m->acts[(size_t)K * Lc + (size_t)k * Lh + (l - Lc)];
      IL_TRY(dev_alloc_t(m, &A.ln1, N * d));
      IL_TRY(dev_alloc_t(m, &A.qkv, N * 3 * d));
      IL_TRY(dev_alloc_t(m, &A.attn_o, N * d));
      IL_TRY(dev_alloc_t(m, &A.ln2, N * d));
      IL_TRY(dev_alloc_t(m, &A.hgrad, N * F));
      IL_TRY(dev_alloc_t(m, &A.hact, N * F));
      IL_TRY(dev_alloc_t(m, &A.mean1, N));
      IL_TRY(dev_alloc_t(m, &A.rstd1, N));
      IL_TRY(dev_alloc_t(m, &A.mean2, N));
      IL_TRY(dev_alloc_t(m, &A.rstd2, N));
      IL_TRY(dev_alloc_t(m, &A.lse, N * H));
      IL_TRY(dev_alloc_t(m, &A.x_mid, N * d));
      IL_TRY(dev_alloc_t(m, &A.x_out, N * d));
      if (l == Lc - 1) m->a[k + 1] = A.x_out;   // the component's output; head blocks (l >= Lc) follow it
    }
  }
  m->part_ld = (V + 127) / 128;
  // stored mode: row stride of exp(logits) = the vocabulary rounded up to 64; recompute mode: the width of one
  // vocabulary chunk of dZ (a multiple of the 256-column tile)
  m->ldz = m->head_mode == IL_HEAD_STORED ? (V + 63) / 64 * 64 : std::min(HEAD_CHUNK, (V + 255) / 256 * 256);
  // A stored-mode model can fall back to recomputation (il_sync, after a row left the representable range): its
  // [Ntok, ldz] buffer then serves as the chunk buffer, so the chunk is the largest multiple of 256 it holds
  // (the whole vocabulary in one chunk when it is narrower than that).
  m->head_chunk = m->head_mode != IL_HEAD_STORED ? m->ldz : (m->ldz >= 256 ? std::min(HEAD_CHUNK, m->ldz / 256 * 256) : m->ldz);
  m->hs.assign(K, HeadScratch{});
  for (int k = 0; k < K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    HeadScratch& h = m->hs[k];
    IL_TRY(dev_alloc_t(m, &h.u, N * d));
    IL_TRY(dev_alloc_t(m, &h.mean, N));
    IL_TRY(dev_alloc_t(m, &h.rstd, N));
    IL_TRY(dev_alloc_t(m, &h.pmax, N * m->part_ld));
    IL_TRY(dev_alloc_t(m, &h.psum, N * m->part_ld));
    IL_TRY(dev_alloc_t(m, &h.tgt_logit, N));
    IL_TRY(dev_alloc_t(m, &h.lse, N));
    IL_TRY(dev_alloc_t(m, &h.nll, N));
    IL_TRY(dev_alloc_t(m, &h.du, N * d));
    IL_TRY(dev_alloc_t(m, &h.ghead, N * d));
    IL_TRY(dev_alloc_t(m, &h.z, N * (size_t)m->ldz));
    if (m->head_mode == IL_HEAD_STORED) {
      IL_TRY(dev_alloc_t(m, &h.us, N * d));
      IL_TRY(dev_alloc_t(m, &h.rs, N));
    }
  }
  IL_TRY(alloc_scratch(m, s_cap_for(K, n)));
  // batch, losses and error words: one set shared by all components on a single device, one per component otherwise
  m->tokens.assign(K, nullptr); m->targets.assign(K, nullptr); m->losses.assign(K, nullptr);
  m->err_word.assign(K, nullptr); m->sort_keys.assign(K, nullptr);
  for (int k = 0; k < K; ++k) {
    if (!pipe && k > 0) {
      m->tokens[k] = m->tokens[0]; m->targets[k] = m->targets[0]; m->losses[k] = m->losses[0];
      m->err_word[k] = m->err_word[0];
      continue;
    }
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    IL_TRY(dev_alloc_t(m, &m->tokens[k], N));
    IL_TRY(dev_alloc_t(m, &m->targets[k], N));
    IL_TRY(dev_alloc_t(m, &m->losses[k], (size_t)K));
    IL_TRY(dev_alloc_t(m, &m->err_word[k], (size_t)(1 + K)));
    IL_CUDA(m, cudaMemsetAsync(m->err_word[k], 0, 4 * (1 + K), m->streams[k]));
    IL_CUDA(m, cudaMemsetAsync(m->losses[k], 0, K * 4, m->streams[k]));
  }
  IL_CUDA(m, cudaSetDevice(m->dev[0]));
  IL_TRY(dev_alloc_t(m, &m->sort_keys[0], (N + 8191) / 8192 * 8192));     // embedding backward: sorted (token, position) keys
  m->fwd_done.assign(K, 0);
  m->loss_done.assign(K, 0);
  for (int dv : m->dev_list) {
    IL_CUDA(m, cudaSetDevice(dv));
    IL_CUDA(m, cudaDeviceSynchronize());
  }
  return IL_OK;
  });
}

extern "C" il_status il_destroy(il_model* m) {
  return guarded([&]() -> il_status {
  if (!m) return IL_ERR_INVALID_ARG;
  for (int dv : m->dev_list) {
    cudaSetDevice(dv);
    cudaDeviceSynchronize();
  }
  for (auto& pr : m->allocs) {
    cudaSetDevice(pr.second);
    if (m->opt.free_) m->opt.free_(pr.first, m->opt.alloc_ctx);
    else cudaFree(pr.first);
  }
  for (auto e : m->ev_fwd) cudaEventDestroy(e);
  for (auto e : m->ev_bwd) cudaEventDestroy(e);
  for (auto e : m->ev_join) cudaEventDestroy(e);
  for (auto e : m->ev_copy) cudaEventDestroy(e);
  for (auto e : m->ev_head) cudaEventDestroy(e);
  for (auto e : m->ev_side) cudaEventDestroy(e);
  for (auto st : m->side) cudaStreamDestroy(st);
  if (m->ev_batch) cudaEventDestroy(m->ev_batch);
  for (auto e : m->prof_pool) cudaEventDestroy(e);
  for (auto& r : m->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  if (m->own_streams)
    for (auto s : m->streams) cudaStreamDestroy(s);
  delete m;
  return IL_OK;
  });
}

extern "C" il_status il_set_n(il_model* m, int n) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (n < 1 || n > m->K) return fail(m, IL_ERR_INVALID_ARG, "n=%d outside [1, %d]", n, m->K);
  IL_TRY(sync_devices(m));
  IL_TRY(alloc_scratch(m, m->rule == IL_RULE_SUM ? s_cap_for(m->K, n) : n));
  m->n = n;
  return IL_OK;
  });
}

extern "C" il_status il_set_rule(il_model* m, int rule) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (rule != IL_RULE_SUM && rule != IL_RULE_FAR && rule != IL_RULE_MEAN) return fail(m, IL_ERR_INVALID_ARG, "unknown rule %d", rule);
  if (m->n > 8 && rule != IL_RULE_SUM) return fail(m, IL_ERR_INVALID_ARG, "weighted rules support n <= 8");
  IL_TRY(sync_devices(m));
  IL_TRY(alloc_scratch(m, rule == IL_RULE_SUM ? s_cap_for(m->K, m->n) : m->n));
  m->rule = rule;
  return IL_OK;
  });
}

// =================================================================================================
// registry
// =================================================================================================
extern "C" int il_num_tensors(const il_model* m) { return m ? (int)m->tensors.size() : -1; }

extern "C" il_status il_tensor_info(const il_model* m, int idx, const char** name, int* component, int* is_head, int* rank,
                                    long long shape[2]) {
  return guarded([&]() -> il_status {
  if (!m || idx < 0 || idx >= (int)m->tensors.size()) return IL_ERR_INVALID_ARG;
  const TensorRec& t = m->tensors[idx];
  if (name) *name = t.name.c_str();
  if (component) *component = t.component;
  if (is_head) *is_head = t.is_head;
  if (rank) *rank = t.rank;
  if (shape) { shape[0] = t.shape[0]; shape[1] = t.shape[1]; }
  return IL_OK;
  });
}

static il_status tensor_io(il_model* m, int idx, size_t count, const TensorRec** t) {
  IL_TRY(check_model(m));
  if (idx < 0 || idx >= (int)m->tensors.size()) return fail(m, IL_ERR_INVALID_ARG, "tensor index %d out of range", idx);
  *t = &m->tensors[idx];
  if (count != (*t)->count) return fail(m, IL_ERR_INVALID_ARG, "tensor %s has %zu elements, got %zu", (*t)->name.c_str(), (*t)->count, count);
  IL_TRY(sync_devices(m));
  return IL_OK;
}

extern "C" il_status il_set_param(il_model* m, int idx, const float* host, size_t count) {
  return guarded([&]() -> il_status {
  const TensorRec* t;
  if (!host) return IL_ERR_INVALID_ARG;
  IL_TRY(tensor_io(m, idx, count, &t));
  const int k = t->component;
  IL_CUDA(m, cudaSetDevice(m->dev[k]));
  IL_CUDA(m, cudaMemcpyAsync(m->P[k] + t->off, host, count * 4, cudaMemcpyHostToDevice, m->streams[k]));
  IL_K(m, f32_to_bf16(m->P[k] + t->off, m->Pb[k] + t->off, align_up(count, 4), m->streams[k]));
  IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));
  return IL_OK;
  });
}
extern "C" il_status il_get_param(il_model* m, int idx, float* host, size_t count) {
  return guarded([&]() -> il_status {
  const TensorRec* t;
  if (!host) return IL_ERR_INVALID_ARG;
  IL_TRY(tensor_io(m, idx, count, &t));
  IL_TRY(copy_sync(m, t->component, host, m->P[t->component] + t->off, count * 4, cudaMemcpyDeviceToHost));
  return IL_OK;
  });
}
extern "C" il_status il_get_grad(il_model* m, int idx, float* host, size_t count) {
  return guarded([&]() -> il_status {
  const TensorRec* t;
  if (!host) return IL_ERR_INVALID_ARG;
  IL_TRY(tensor_io(m, idx, count, &t));
  if (!m->bwd_done) return fail(m, IL_ERR_STATE, "il_get_grad before il_backward_nwise");
  IL_TRY(copy_sync(m, t->component, host, m->G[t->component] + t->off, count * 4, cudaMemcpyDeviceToHost));
  return IL_OK;
  });
}
extern "C" il_status il_get_opt_state(il_model* m, int idx, float* mh, float* vh, long long* step) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (idx < 0 || idx >= (int)m->tensors.size()) return fail(m, IL_ERR_INVALID_ARG, "tensor index %d out of range", idx);
  const TensorRec* t;
  IL_TRY(tensor_io(m, idx, m->tensors[idx].count, &t));
  const int k = t->component;
  if (mh) IL_TRY(copy_sync(m, k, mh, m->M1[k] + t->off, t->count * 4, cudaMemcpyDeviceToHost));
  if (vh) IL_TRY(copy_sync(m, k, vh, m->M2[k] + t->off, t->count * 4, cudaMemcpyDeviceToHost));
  if (step) *step = m->step;
  return IL_OK;
  });
}
extern "C" il_status il_set_opt_state(il_model* m, int idx, const float* mh, const float* vh, long long step) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (idx < 0 || idx >= (int)m->tensors.size()) return fail(m, IL_ERR_INVALID_ARG, "tensor index %d out of range", idx);
  if (step < 0) return fail(m, IL_ERR_INVALID_ARG, "negative step");
  const TensorRec* t;
  IL_TRY(tensor_io(m, idx, m->tensors[idx].count, &t));
  const int k = t->component;
  if (mh) IL_TRY(copy_sync(m, k, m->M1[k] + t->off, mh, t->count * 4, cudaMemcpyHostToDevice));
  if (vh) IL_TRY(copy_sync(m, k, m->M2[k] + t->off, vh, t->count * 4, cudaMemcpyHostToDevice));
  m->step = step;
  return IL_OK;
  });
}

// =================================================================================================
// the step
// =================================================================================================
extern "C" il_status il_set_batch(il_model* m, const int* tokens, const int* targets, int B, int T, int on_device) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  Range range("il_set_batch");
  if (!tokens || !targets) return fail(m, IL_ERR_INVALID_ARG, "NULL tokens/targets");
  if (B < 1 || T < 1 || B > m->max_batch || T > m->max_seq || (size_t)B * T > (size_t)m->ntok_max)
    return fail(m, IL_ERR_INVALID_ARG, "batch %dx%d exceeds max_batch=%d, max_seq=%d", B, T, m->max_batch, m->max_seq);
  IL_CUDA(m, cudaSetDevice(m->dev[0]));
  // every stream's previous work must be finished before buffers of the last step are overwritten
  IL_TRY(join_all(m));
  cudaStream_t s0 = m->streams[0];
  const size_t bytes = (size_t)B * T * sizeof(int);
  const cudaMemcpyKind kind = on_device ? cudaMemcpyDefault : cudaMemcpyHostToDevice;
  IL_CUDA(m, cudaEventRecord(m->ev_batch, s0));
  for (int k = 0; k < m->K; ++k) {
    if (k > 0) IL_CUDA(m, cudaStreamWaitEvent(m->streams[k], m->ev_batch, 0));
    if (k > 0 && m->tokens[k] == m->tokens[0]) continue;       // one shared copy on a single device
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    IL_CUDA(m, cudaMemcpyAsync(m->tokens[k], tokens, bytes, kind, m->streams[k]));
    IL_CUDA(m, cudaMemcpyAsync(m->targets[k], targets, bytes, kind, m->streams[k]));
  }
  IL_CUDA(m, cudaSetDevice(m->dev[0]));
  // (token, position) keys in sorted order for the embedding backward: known as soon as the batch is
  IL_K(m, embed_sort(m->tokens[0], m->sort_keys[0], B * T, m->V, s0));
  if (m->tokens[1 % m->K] == m->tokens[0]) {     // shared buffers: the other streams start after the copies
    IL_CUDA(m, cudaEventRecord(m->ev_batch, s0));
    for (int k = 1; k < m->K; ++k) IL_CUDA(m, cudaStreamWaitEvent(m->streams[k], m->ev_batch, 0));
  }
  m->B = B; m->T = T; m->ntok = B * T;
  m->xfer_log.clear();
  m->batch_set = true;
  m->bwd_done = false;
  std::fill(m->fwd_done.begin(), m->fwd_done.end(), 0);
  std::fill(m->loss_done.begin(), m->loss_done.end(), 0);
  return IL_OK;
  });
}

namespace {

// `count` consecutive pre-LN blocks (layer records base .. base+count-1) applied to x_in on stream k.
il_status layers_forward(il_model* m, int k, size_t base, int count, const float* x_in) {
  cudaStream_t st = m->streams[k];
  const int N = m->ntok, d = m->d, F = m->F;
  for (int l = 0; l < count; ++l) {
    const LayerOff& o = m->layer_off[base + l];
    LayerActs& A = m->acts[base + l];
    IL_K(m, layernorm_fwd(x_in, m->P[k] + o.ln1g, m->P[k] + o.ln1b, A.ln1, A.mean1, A.rstd1, N, d, m->ln_eps, st));
    {
      GemmArgs g = gemm_args(N, 3 * d, d, A.ln1, d, 0, m->Pb[k] + o.wqkv, d, 0, EPI_BF16, A.qkv, 3 * d);
      g.bias = m->P[k] + o.bqkv;
      IL_TRY(gemm(m, k, g));
    }
    IL_K(m, attention_fwd(A.qkv, A.attn_o, A.lse, m->B, m->T, m->H, m->dh, m->err_word[k], st));
    {
      GemmArgs g = gemm_args(N, d, d, A.attn_o, d, 0, m->Pb[k] + o.wo, d, 0, EPI_F32_RESID, A.x_mid, d);
      g.bias = m->P[k] + o.bo;
      g.resid = x_in;
      IL_TRY(gemm(m, k, g));
    }
    IL_K(m, layernorm_fwd(A.x_mid, m->P[k] + o.ln2g, m->P[k] + o.ln2b, A.ln2, A.mean2, A.rstd2, N, d, m->ln_eps, st));
    {
      GemmArgs g = gemm_args(N, F, d, A.ln2, d, 0, m->Pb[k] + o.w1, d, 0, EPI_BF16_GELU, A.hgrad, F);
      g.C2 = A.hact;
      g.bias = m->P[k] + o.b1;
      IL_TRY(gemm(m, k, g));
    }
    {
      GemmArgs g = gemm_args(N, d, F, A.hact, F, 0, m->Pb[k] + o.w2, F, 0, EPI_F32_RESID, A.x_out, d);
      g.bias = m->P[k] + o.b2;
      g.resid = A.x_mid;
      IL_TRY(gemm(m, k, g));
    }
    x_in = A.x_out;
  }
  return IL_OK;
}

}  // namespace

extern "C" il_status il_forward_component(il_model* m, int k) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  Range range("il_forward_component %d", k);
  if (k < 0 || k >= m->K) return fail(m, IL_ERR_INVALID_ARG, "component %d out of range", k);
  if (!m->batch_set) return fail(m, IL_ERR_STATE, "il_forward_component before il_set_batch");
  if (k > 0 && !m->fwd_done[k - 1]) return fail(m, IL_ERR_STATE, "component %d forward needs component %d first", k, k - 1);
  if (m->fwd_done[k]) return fail(m, IL_ERR_STATE, "component %d already forwarded in this step", k);
  IL_CUDA(m, cudaSetDevice(m->dev[k]));
  cudaStream_t st = m->streams[k];
  const int N = m->ntok, d = m->d;
  if (k == 0) {
    IL_K(m, embed_fwd(m->tokens[k], m->P[k] + m->off_wte, m->P[k] + m->off_wpe, m->a[0], N, m->T, d, m->V, st));
  } else {
    IL_CUDA(m, cudaStreamWaitEvent(st, m->ev_fwd[k - 1], 0));
    // pipeline placement (Sec. 3: the module's output is sent to the next accelerator): a_k is copied into a
    // buffer this component's device owns; every kernel of the component then reads local memory only
    if (m->placement == IL_PLACE_PIPELINE) {
      IL_CUDA(m, cudaMemcpyPeerAsync(m->a_in[k], m->dev[k], m->a[k], m->dev[k - 1], (size_t)N * d * sizeof(float), st));
      m->xfer_log.push_back(0); m->xfer_log.push_back(k - 1); m->xfer_log.push_back(-1);
    }
  }
  IL_TRY(layers_forward(m, k, (size_t)k * m->Lc, m->Lc, comp_input(m, k)));
  IL_CUDA(m, cudaEventRecord(m->ev_fwd[k], st));
  m->fwd_done[k] = 1;
  return IL_OK;
  });
}

extern "C" il_status il_aux_head_loss(il_model* m, int k, float* loss_host) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  Range range("il_aux_head_loss %d", k);
  if (k < 0 || k >= m->K) return fail(m, IL_ERR_INVALID_ARG, "head %d out of range", k);
  if (!m->batch_set || !m->fwd_done[k]) return fail(m, IL_ERR_STATE, "il_aux_head_loss(%d) needs il_forward_component(%d)", k, k);
  IL_CUDA(m, cudaSetDevice(m->dev[k]));
  cudaStream_t st = m->streams[k];
  if (!m->loss_done[k]) {
    const int N = m->ntok, d = m->d, V = m->V;
    const HeadOff& o = m->head_off[k];
    HeadScratch& h = m->hs[k];
    const size_t hbase = (size_t)m->K * m->Lc + (size_t)k * m->Lh;
    if (m->Lh > 0) IL_TRY(layers_forward(m, k, hbase, m->Lh, m->a[k + 1]));
    const float* hx = head_input(m, k);
    IL_K(m, layernorm_fwd(hx, m->P[k] + o.lng, m->P[k] + o.lnb, h.u, h.mean, h.rstd, N, d, m->ln_eps, st));
    // One GEMM over the whole vocabulary whose epilogue keeps per-(row, 128-column block) softmax partials and the
    // target logit.  Stored mode: it also writes exp(logit) in bf16 for the backward.  Recompute mode: nothing of
    // the [Ntok, V] matrix is written; the backward forms it again chunk by chunk.
    const bool stored = m->head_mode == IL_HEAD_STORED;
    GemmArgs g = gemm_args(N, V, d, h.u, d, 0, m->Pb[k] + o.w, d, 0, EPI_LSE, stored ? h.z : nullptr, stored ? m->ldz : 0);
    g.targets = m->targets[k];
    g.part_max = h.pmax; g.part_sum = h.psum; g.part_ld = m->part_ld;
    g.tgt_logit = h.tgt_logit;
    g.col0 = 0;
    g.store_exp = stored ? 1 : 0;
    IL_TRY(gemm(m, k, g));
    // per-row log-sum-exp and negative log-likelihood, then the mean of the latter in a fixed summation order
    IL_K(m, lse_finalize(h.pmax, h.psum, m->part_ld, m->part_ld, h.tgt_logit, h.lse, h.nll, N, st));
    IL_K(m, mean_f32(h.nll, N, m->losses[k] + k, st));
    m->loss_done[k] = 1;
  }
  if (loss_host) {
    IL_CUDA(m, cudaMemcpyAsync(loss_host, m->losses[k] + k, sizeof(float), cudaMemcpyDeviceToHost, st));
    IL_CUDA(m, cudaStreamSynchronize(st));
  }
  return IL_OK;
  });
}

extern "C" il_status il_get_token_losses(il_model* m, int k, float* host, size_t count) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (k < 0 || k >= m->K || !host) return fail(m, IL_ERR_INVALID_ARG, "head %d out of range or NULL output", k);
  if (!m->batch_set || !m->loss_done[k]) return fail(m, IL_ERR_STATE, "head %d has no loss in this step", k);
  if (count != (size_t)m->ntok) return fail(m, IL_ERR_INVALID_ARG, "expected %d values, got %zu", m->ntok, count);
  IL_TRY(copy_sync(m, k, host, m->hs[k].nll, count * 4, cudaMemcpyDeviceToHost));
  return IL_OK;
  });
}

extern "C" il_status il_get_losses(il_model* m, float* losses_host) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (!losses_host) return fail(m, IL_ERR_INVALID_ARG, "NULL output");
  for (int k = 0; k < m->K; ++k)
    if (!m->loss_done[k]) return fail(m, IL_ERR_STATE, "head %d has no loss in this step", k);
  if (m->losses[m->K - 1] == m->losses[0]) {        // one shared array
    IL_CUDA(m, cudaSetDevice(m->dev[0]));
    for (int k = 1; k < m->K; ++k) IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));
    IL_TRY(copy_sync(m, 0, losses_host, m->losses[0], m->K * sizeof(float), cudaMemcpyDeviceToHost));
  } else {
    for (int k = 0; k < m->K; ++k) IL_TRY(copy_sync(m, k, losses_host + k, m->losses[k] + k, sizeof(float), cudaMemcpyDeviceToHost));
  }
  return IL_OK;
  });
}

namespace {

// Backward on stream k through `count` consecutive blocks (layer records base .. base+count-1, whose first block
// read x_first) for s stacked gradient streams already placed in cs[k].dx / dxb; the result is left there.
// acc: parameter gradients are added to what the buffers hold (a later micro-batch) instead of replacing it.
il_status layers_backward(il_model* m, int k, int s, size_t base, int count, const float* x_first, bool acc) {
  cudaStream_t st = m->streams[k];
  const int N = m->ntok, d = m->d, F = m->F;
  const int R = s * N;
  CompScratch& c = m->cs[k];
  const bool fused_ln = d % 128 == 0 && d <= 1024;     // widths the one-pass LayerNorm backward covers
  for (int l = count - 1; l >= 0; --l) {
    const LayerOff& o = m->layer_off[base + l];
    LayerActs& A = m->acts[base + l];
    const float* x_in = (l == 0) ? x_first : m->acts[base + l - 1].x_out;
    // ---- MLP: x_out = x_mid + W2 gelu(W1 ln2 + b1) + b2
    // bias gradient of FC2: column sums of the incoming gradient (first stream).  Below the top block they come
    // out of the LayerNorm backward that produced this gradient.
    if (l == count - 1 || !fused_ln) IL_K(m, colsum_f32(c.dx, d, m->G[k] + o.b2, N, d, st));
    IL_TRY(wgrad(m, k, d, F, N, c.dxb, d, A.hact, F, m->G[k] + o.w2, acc));
    {
      GemmArgs g = gemm_args(R, F, d, c.dxb, d, 0, m->Pb[k] + o.w2, F, 1, EPI_BF16_DGELU, c.dbig, F);
      g.aux = A.hgrad; g.ld_aux = F; g.aux_rows = N;
      g.colsum = m->G[k] + o.b1;                 // FC1 bias gradient: column sums of the first gradient stream
      IL_TRY(gemm(m, k, g));
    }
    IL_TRY(wgrad(m, k, F, d, N, c.dbig, F, A.ln2, d, m->G[k] + o.w1, acc));
    IL_TRY(gemm(m, k, gemm_args(R, d, F, c.dbig, F, 0, m->Pb[k] + o.w1, d, 1, EPI_BF16, c.dln, d)));
    if (fused_ln) {   // LayerNorm backward with its parameter gradients and the bias gradient of Wo in one pass
      IL_K(m, layernorm_bwd_fused(c.dln, A.x_mid, A.mean2, A.rstd2, m->P[k] + o.ln2g, c.dx, c.dx, c.dxb, m->G[k] + o.ln2g,
                                  m->G[k] + o.ln2b, m->G[k] + o.bo, R, N, d, st));
    } else {
      IL_K(m, layernorm_bwd_params(c.dln, 0, A.x_mid, A.mean2, A.rstd2, m->G[k] + o.ln2g, m->G[k] + o.ln2b, N, d, st));
      IL_K(m, layernorm_bwd_rows(c.dln, 0, A.x_mid, A.mean2, A.rstd2, m->P[k] + o.ln2g, c.dx, c.dx, c.dxb, R, N, d, st));
      // ---- attention: x_mid = x_in + Wo attn(Wqkv ln1 + bqkv) + bo
      IL_K(m, colsum_f32(c.dx, d, m->G[k] + o.bo, N, d, st));
    }
    IL_TRY(wgrad(m, k, d, d, N, c.dxb, d, A.attn_o, d, m->G[k] + o.wo, acc));
    IL_TRY(gemm(m, k, gemm_args(R, d, d, c.dxb, d, 0, m->Pb[k] + o.wo, d, 1, EPI_BF16, c.dattn, d)));
    // dQ accumulator of the one-sweep attention backward: the FC1 gradient buffer (bf16 [R, F], at least the
    // [R, d] fp32 needed whenever F >= 2 d) is free between the MLP's and the attention's backward
    float* dq_acc = (m->attn_bwd == IL_ATTN_BWD_ONE_SWEEP && F >= 2 * d) ? reinterpret_cast<float*>(c.dbig) : nullptr;
    IL_K(m, attention_bwd(A.qkv, A.attn_o, A.lse, c.dattn, c.dqkv, c.delta, dq_acc, s * m->B, m->B, m->T, m->H, m->dh,
                          m->err_word[k], st));
    m->launches += 2;
    IL_K(m, colsum_bf16(c.dqkv, 3 * d, m->G[k] + o.bqkv, N, 3 * d, st));
    IL_TRY(wgrad(m, k, 3 * d, d, N, c.dqkv, 3 * d, A.ln1, d, m->G[k] + o.wqkv, acc));
    IL_TRY(gemm(m, k, gemm_args(R, d, 3 * d, c.dqkv, 3 * d, 0, m->Pb[k] + o.wqkv, d, 1, EPI_BF16, c.dln, d)));
    if (fused_ln) {   // ... and the FC2 bias gradient of the block below
      float* b2_below = l > 0 ? m->G[k] + m->layer_off[base + l - 1].b2 : nullptr;
      IL_K(m, layernorm_bwd_fused(c.dln, x_in, A.mean1, A.rstd1, m->P[k] + o.ln1g, c.dx, c.dx, c.dxb, m->G[k] + o.ln1g,
                                  m->G[k] + o.ln1b, b2_below, R, N, d, st));
    } else {
      IL_K(m, layernorm_bwd_params(c.dln, 0, x_in, A.mean1, A.rstd1, m->G[k] + o.ln1g, m->G[k] + o.ln1b, N, d, st));
      IL_K(m, layernorm_bwd_rows(c.dln, 0, x_in, A.mean1, A.rstd1, m->P[k] + o.ln1g, c.dx, c.dx, c.dxb, R, N, d, st));
    }
  }
  return IL_OK;
}

// Head k backward on stream k.  The loss pass kept E = exp(logits); dZ = (softmax - onehot) / Ntok equals
// diag(s) E' with s = exp(-lse) / Ntok and E' = E with exp(lse) subtracted at the target, so after a per-row
// set-up kernel dU = diag(s) (E' W) and dW_h = E'^T (diag(s) U) run straight on E' — no pass over the
// [Ntok, V] matrix other than the two GEMMs.  LayerNorm backward -> ghead.
// With blocks inside the head (App. B.3) the gradient then runs through them, in the component's backward
// scratch (free at this point of stream k), and ghead is the gradient at the component's output either way.
// acc / scale: this pass adds scale * gradient to the buffers (micro-batch 2.. of an update) or overwrites them.
il_status head_backward(il_model* m, int k, bool acc, float scale) {
  cudaStream_t st = m->streams[k];
  const int N = m->ntok, d = m->d, V = m->V;
  const HeadOff& o = m->head_off[k];
  HeadScratch& h = m->hs[k];
  if (m->head_mode == IL_HEAD_STORED) {
    IL_K(m, head_backward_prepare(h.z, m->ldz, h.lse, m->targets[k], h.u, h.us, h.rs, N, d, scale, m->err_word[k], st));
    {  // dU = diag(s) (E' W).  Not split over the contraction: atomically added partial sums would make dU, and
       // with it every gradient below this head, depend on the order the work units finish in.
      GemmArgs g = gemm_args(N, d, V, h.z, m->ldz, 0, m->Pb[k] + o.w, d, 1, EPI_F32, h.du, d);
      g.rowscale = h.rs;
      IL_TRY(gemm(m, k, g));
    }
    {  // dW = E'^T (diag(s) U)
      GemmArgs g = gemm_args(V, d, N, h.z, m->ldz, 1, h.us, d, 1, EPI_F32, m->G[k] + o.w, d);
      g.accumulate = acc ? 1 : 0;
      IL_TRY(gemm(m, k, g));
    }
  } else {
    // Recompute mode: nothing of the [Ntok, V] matrix was kept.  The vocabulary is walked in chunks of HEAD_CHUNK
    // columns; per chunk the logits are formed again and turned into dZ = (softmax - onehot) * scale / Ntok in the
    // GEMM's epilogue (bf16, [Ntok, chunk]), then dU += dZ W_chunk and dW_chunk = dZ^T U.  The chunks follow each
    // other on this head's stream, so dU is summed in a fixed order.
    const int chunk = m->head_chunk;
    for (int c0 = 0; c0 < V; c0 += chunk) {
      const int w = std::min(chunk, V - c0);
      {
        GemmArgs g = gemm_args(N, w, d, h.u, d, 0, m->Pb[k] + o.w + (size_t)c0 * d, d, 0, EPI_DZ, h.z, chunk);
        g.targets = m->targets[k];
        g.lse = h.lse;
        g.scale = scale / (float)N;
        g.col0 = c0;
        IL_TRY(gemm(m, k, g));
      }
      {
        GemmArgs g = gemm_args(N, d, w, h.z, chunk, 0, m->Pb[k] + o.w + (size_t)c0 * d, d, 1, EPI_F32, h.du, d);
        g.accumulate = c0 > 0 ? 1 : 0;
        IL_TRY(gemm(m, k, g));
      }
      {
        GemmArgs g = gemm_args(w, d, N, h.z, chunk, 1, h.u, d, 1, EPI_F32, m->G[k] + o.w + (size_t)c0 * d, d);
        g.accumulate = acc ? 1 : 0;
        IL_TRY(gemm(m, k, g));
      }
    }
  }
  const float* hx = head_input(m, k);
  IL_K(m, layernorm_bwd_params(h.du, 1, hx, h.mean, h.rstd, m->G[k] + o.lng, m->G[k] + o.lnb, N, d, st));
  if (m->Lh == 0) {
    IL_K(m, layernorm_bwd_rows(h.du, 1, hx, h.mean, h.rstd, m->P[k] + o.lng, nullptr, h.ghead, nullptr, N, N, d, st));
    return IL_OK;
  }
  CompScratch& c = m->cs[k];
  IL_K(m, layernorm_bwd_rows(h.du, 1, hx, h.mean, h.rstd, m->P[k] + o.lng, nullptr, c.dx, c.dxb, N, N, d, st));
  IL_TRY(layers_backward(m, k, 1, (size_t)m->K * m->Lc + (size_t)k * m->Lh, m->Lh, m->a[k + 1], acc));
  IL_CUDA(m, cudaMemcpyAsync(h.ghead, c.dx, (size_t)N * d * sizeof(float), cudaMemcpyDeviceToDevice, st));
  return IL_OK;
}

il_status component_backward(il_model* m, int k, int s, bool acc) {
  return layers_backward(m, k, s, (size_t)k * m->Lc, m->Lc, comp_input(m, k), acc);
}

}  // namespace

extern "C" il_status il_backward_nwise(il_model* m) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  Range range("il_backward_nwise");
  if (!m->batch_set) return fail(m, IL_ERR_STATE, "il_backward_nwise before il_set_batch");
  for (int k = 0; k < m->K; ++k)
    if (!m->fwd_done[k] || !m->loss_done[k])
      return fail(m, IL_ERR_STATE, "il_backward_nwise needs all %d forwards and head losses (component %d missing)", m->K, k);
  if (m->bwd_done) return fail(m, IL_ERR_STATE, "il_backward_nwise already called in this step");
  if (m->micro > 1 && m->micro_done >= m->micro)
    return fail(m, IL_ERR_STATE, "all %d micro-batches of this update have been back-propagated; call il_adamw_step", m->micro);
  const int K = m->K, n = m->n, N = m->ntok, d = m->d;
  const size_t slice = (size_t)N * d;
  // Gradient stream `slot` of component k+1 as component k reads it: in place on a single device; in the pipeline
  // placement (Sec. 3: gradients are sent back to the previous accelerator) copied, once, on stream k into the
  // receive buffer that k's device owns.  Stream k has already waited for component k+1's backward.
  std::vector<char> fetched;
  cudaError_t fetch_err = cudaSuccess;
  auto from_above = [&](int k, int slot, int id) -> const float* {
    const float* src = m->cs[k + 1].dx + (size_t)slot * slice;
    if (m->placement != IL_PLACE_PIPELINE) return src;
    float* dst = m->g_in[k] + (size_t)slot * slice;
    if (!fetched[slot]) {
      cudaError_t e = cudaMemcpyPeerAsync(dst, m->dev[k], src, m->dev[k + 1], slice * sizeof(float), m->streams[k]);
      if (e != cudaSuccess) fetch_err = e;
      fetched[slot] = 1;
      m->xfer_log.push_back(1); m->xfer_log.push_back(k); m->xfer_log.push_back(id);
    }
    return dst;
  };
  // Micro-batching (Sec. 3.1): the first backward pass of an update overwrites the gradients, the later ones add
  // to them; each pass is scaled by 1 / micro-batches so that the buffers end up holding the mini-batch mean.
  const bool acc = m->micro > 1 && m->micro_done > 0;
  const float gscale = 1.0f / (float)m->micro;

  // every head's own backward is independent of the others: enqueue all of them first
  for (int k = 0; k < K; ++k) {
    cudaStream_t st = m->streams[k];
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    if (!acc) {   // vectors are summed into atomically; embedding rows no token selects must read zero
      IL_CUDA(m, cudaMemsetAsync(m->G[k] + m->comp_mat_end[k], 0, (m->comp_end[k] - m->comp_mat_end[k]) * 4, st));
      if (k == 0) {
        const size_t emb = (size_t)m->V * d;
        IL_CUDA(m, cudaMemsetAsync(m->G[k] + m->off_wte, 0, emb * 4, st));
        IL_CUDA(m, cudaMemsetAsync(m->G[k] + m->off_wpe, 0, (size_t)m->max_seq * d * 4, st));
      }
    }
    {
      Range r2("head backward %d", k);
      IL_TRY(head_backward(m, k, acc, gscale));
    }
    IL_CUDA(m, cudaEventRecord(m->ev_head[k], st));      // head k's parameter gradients are final from here on
  }
  if (m->rule == IL_RULE_SUM) {
    // components from the top down; component k needs the pass-down of component k+1 when any stream crosses
    std::vector<int> above;   // termination levels of the streams of component k+1
    for (int k = K - 1; k >= 0; --k) {
      cudaStream_t st = m->streams[k];
      IL_CUDA(m, cudaSetDevice(m->dev[k]));
      fetched.assign((size_t)m->s_cap + 1, 0);
      const std::vector<int> terms = terms_of(k, K, n);
      const int s = (int)terms.size();
      bool needs_above = false;
      for (int j = 0; j < s; ++j) {
        int src = -1;
        for (size_t q = 0; q < above.size(); ++q)
          if (above[q] == terms[j]) src = (int)q;
        if (src >= 0 && !needs_above) {
          IL_CUDA(m, cudaStreamWaitEvent(st, m->ev_bwd[k + 1], 0));
          needs_above = true;
        }
        const float* passed = src >= 0 ? from_above(k, src, terms[j]) : nullptr;
        if (fetch_err != cudaSuccess) return fail(m, IL_ERR_CUDA, "cudaMemcpyPeerAsync: %s", cudaGetErrorString(fetch_err));
        IL_K(m, add_convert(m->hs[k].ghead, passed, m->cs[k].dx + (size_t)j * slice, m->cs[k].dxb + (size_t)j * slice, slice, st));
      }
      {
        Range r2("component backward %d", k);
        IL_TRY(component_backward(m, k, s, acc));
      }
      if (k == 0) {
        IL_K(m, embed_bwd(m->tokens[k], m->sort_keys[0], m->cs[0].dx, m->G[k] + m->off_wte, m->G[k] + m->off_wpe, N, m->T, d, m->V, acc ? 1 : 0, st));
        m->launches++;
      }
      IL_CUDA(m, cudaEventRecord(m->ev_bwd[k], st));
      above = terms;
    }
  } else {
    // Weighted rules: component k carries slot 0 = sum_h W(k,h) g^(h) (drives every parameter gradient) and one
    // slot per head that continues below k (all crossing heads but the one with h = k+n-1); the pass-down of a
    // head is taken from its own slot of component k+1.  When the combination is a single head with weight one that
    // also continues below (the top component under the mean rule), slot 0 serves as that head's slot too.
    std::vector<int> above_heads;     // heads carried by component k+1 ...
    std::vector<int> above_slots;     // ... and the slot each of them occupies there
    for (int k = K - 1; k >= 0; --k) {
      cudaStream_t st = m->streams[k];
      IL_CUDA(m, cudaSetDevice(m->dev[k]));
      fetched.assign((size_t)m->s_cap + 1, 0);
      const int hi = k + n - 1 < K - 1 ? k + n - 1 : K - 1;
      auto grad_of = [&](int h) -> const float* {      // gradient of head h at the output of component k
        if (h == k) return m->hs[k].ghead;
        for (size_t q = 0; q < above_heads.size(); ++q)
          if (above_heads[q] == h) return from_above(k, above_slots[q], h);
        return nullptr;
      };
      if (hi > k) IL_CUDA(m, cudaStreamWaitEvent(st, m->ev_bwd[k + 1], 0));
      // slot 0: the weighted combination
      int single = -1;                  // the head slot 0 equals exactly, if any
      {
        const float* xs[8];
        float ws[8];
        int cnt = 0;
        for (int h = k; h <= hi; ++h) {
          const float wgt = rule_weight(m->rule, k, h, n, K);
          if (wgt == 0.0f) continue;
          xs[cnt] = grad_of(h);
          if (!xs[cnt]) return fail(m, IL_ERR_STATE, "internal: gradient stream of head %d missing at component %d", h, k);
          single = (cnt == 0 && wgt == 1.0f) ? h : -1;
          ws[cnt++] = wgt;
        }
        for (int c0 = 0; c0 < cnt; c0 += 4) {
          const int c = cnt - c0 < 4 ? cnt - c0 : 4;
          IL_K(m, lincomb_convert(xs + c0, ws + c0, c, c0 > 0, m->cs[k].dx, c0 + 4 >= cnt ? m->cs[k].dxb : nullptr, slice, st));
        }
      }
      // slots 1..: heads that continue below this component
      std::vector<int> mine, mine_slots;
      int used = 1;
      if (k > 0)
        for (int h = k; h <= hi; ++h)
          if (h < k + n - 1) {
            mine.push_back(h);
            if (h == single) { mine_slots.push_back(0); continue; }
            const float* src = grad_of(h);
            if (!src) return fail(m, IL_ERR_STATE, "internal: gradient stream of head %d missing at component %d", h, k);
            IL_K(m, add_convert(src, nullptr, m->cs[k].dx + (size_t)used * slice, m->cs[k].dxb + (size_t)used * slice, slice, st));
            mine_slots.push_back(used++);
          }
      if (fetch_err != cudaSuccess) return fail(m, IL_ERR_CUDA, "cudaMemcpyPeerAsync: %s", cudaGetErrorString(fetch_err));
      {
        Range r2("component backward %d", k);
        IL_TRY(component_backward(m, k, used, acc));
      }
      if (k == 0) {
        IL_K(m, embed_bwd(m->tokens[k], m->sort_keys[0], m->cs[0].dx, m->G[k] + m->off_wte, m->G[k] + m->off_wpe, N, m->T, d, m->V, acc ? 1 : 0, st));
        m->launches++;
      }
      IL_CUDA(m, cudaEventRecord(m->ev_bwd[k], st));
      above_heads = mine;
      above_slots = mine_slots;
    }
  }
  m->bwd_done = true;
  m->micro_done = m->micro > 1 ? m->micro_done + 1 : 1;
  return IL_OK;
  });
}

extern "C" il_status il_set_micro_batches(il_model* m, int micro_batches) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (micro_batches < 1) return fail(m, IL_ERR_INVALID_ARG, "micro_batches must be >= 1");
  m->micro = micro_batches;
  m->micro_done = 0;      // gradients accumulated so far are abandoned: the next backward pass overwrites them
  return IL_OK;
  });
}

extern "C" il_status il_lr_schedule(long long step, int d_model, int warmup_steps, double* lr) {
  return guarded([&]() -> il_status {
  if (step < 1 || d_model < 1 || warmup_steps < 1 || !lr) return IL_ERR_INVALID_ARG;
  const double s = (double)step, w = (double)warmup_steps;
  const double a = 1.0 / sqrt(s), b = s / (w * sqrt(w));
  *lr = (a < b ? a : b) / sqrt((double)d_model);
  return IL_OK;
  });
}

extern "C" il_status il_adamw_step(il_model* m, float lr, float beta1, float beta2, float eps, float wd) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  Range range("il_adamw_step");
  if (!m->bwd_done || !m->batch_set) return fail(m, IL_ERR_STATE, "il_adamw_step needs il_backward_nwise of the current step");
  if (m->micro_done != m->micro)
    return fail(m, IL_ERR_STATE, "il_adamw_step after %d of %d micro-batches", m->micro_done, m->micro);
  if (!(beta1 >= 0 && beta1 < 1 && beta2 >= 0 && beta2 < 1 && eps >= 0)) return fail(m, IL_ERR_INVALID_ARG, "bad AdamW hyper-parameters");
  m->step += 1;
  m->adamw_issued += 1;
  const double bc1 = 1.0 - pow((double)beta1, (double)m->step);
  const double bc2 = 1.0 - pow((double)beta2, (double)m->step);
  // Parameters, gradients and bf16 shadows of component k (its head and, for k = 0, the embeddings included)
  // are read and written by stream k only, so each component updates on its own stream as soon as its
  // gradients are final (the last backward pass through a module triggers its update, App. C).
  for (int k = 0; k < m->K; ++k) {
    const size_t b = m->comp_begin[k], e = m->comp_end[k], me = m->comp_mat_end[k];
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    // The kernels leave everything untouched while the error word is set (the gradients of a failed step are not
    // applied); the main launch counts the update in word 1 + k.  The head's vocabulary matrix (the last matrix of
    // the component's range, more than half of its parameters) is updated on the side stream as soon as the head's
    // own backward is done, so that this HBM-bound pass runs beside the component's tensor-bound backward.
    const size_t hw0 = m->head_off[k].w, hw1 = me;
    const bool aside = m->prof != 2;        // (the exclusive GEMM timing mode keeps everything on the component streams)
    cudaStream_t hs = aside ? m->side[k] : m->streams[k];
    if (aside) IL_CUDA(m, cudaStreamWaitEvent(hs, m->ev_head[k], 0));
    IL_K(m, adamw(m->P[k] + hw0, m->M1[k] + hw0, m->M2[k] + hw0, m->G[k] + hw0, m->Pb[k] + hw0, hw1 - hw0, hw1 - hw0, lr, beta1, beta2,
                  eps, wd, (float)bc1, (float)bc2, m->err_word[k], nullptr, 0, 0, hs));
    if (aside) IL_CUDA(m, cudaEventRecord(m->ev_side[k], hs));
    IL_K(m, adamw(m->P[k] + b, m->M1[k] + b, m->M2[k] + b, m->G[k] + b, m->Pb[k] + b, e - b, me - b, lr, beta1, beta2, eps, wd,
                  (float)bc1, (float)bc2, m->err_word[k], m->err_word[k] + 1 + k, hw0 - b, hw1 - b, m->streams[k]));
    if (aside) IL_CUDA(m, cudaStreamWaitEvent(m->streams[k], m->ev_side[k], 0));   // stream k's tail covers the side stream
  }
  m->batch_set = false;   // a new batch is required for the next step
  m->micro_done = 0;
  return IL_OK;
  });
}

extern "C" il_status il_sync(il_model* m) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  for (int k = 0; k < m->K; ++k) {
    IL_CUDA(m, cudaSetDevice(m->dev[k]));
    IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));
  }
  // error word and per-component update counters of every distinct buffer
  unsigned first = 0;
  int applied_min = m->adamw_issued, applied_max = 0;
  unsigned words[1 + 64];                 // K <= 64 (il_create)
  const bool shared = m->err_word[m->K - 1] == m->err_word[0];
  for (int k = 0; k < m->K; ++k) {
    if (shared && k > 0) break;
    IL_TRY(copy_sync(m, k, words, m->err_word[k], 4 * (size_t)(1 + m->K), cudaMemcpyDeviceToHost));
    if (words[0] && !first) first = words[0];
    for (int j = shared ? 0 : k; j <= (shared ? m->K - 1 : k); ++j) {
      applied_min = std::min(applied_min, (int)words[1 + j]);
      applied_max = std::max(applied_max, (int)words[1 + j]);
    }
    IL_CUDA(m, cudaMemsetAsync(m->err_word[k], 0, 4 * (size_t)(1 + m->K), m->streams[k]));
    IL_CUDA(m, cudaStreamSynchronize(m->streams[k]));
  }
  const int issued = m->adamw_issued;
  m->adamw_issued = 0;
  if (first) {
    // Updates enqueued after the failure were skipped on the device: the step counter goes back to the number of
    // updates that were applied.  A component whose update ran before another component raised the error keeps it.
    m->step -= (issued - applied_max);
    const char* partial = applied_min != applied_max ? "; some components applied an update that others skipped" : "";
    if (first == DEV_LOGIT_RANGE) {
      // Only the stored-exp(logit) head has this limit.  From here on the model recomputes the logits in the head
      // backward instead (the stored matrix's memory becomes the chunk buffer); the caller repeats the step.
      m->head_mode = IL_HEAD_RECOMPUTE;
      return fail(m, IL_ERR_NONFINITE, "a head's log-sum-exp left [-80, 80]: exp(logit) is not representable; "
                  "%d of %d optimiser updates since the last il_sync were applied%s; the model has switched to "
                  "IL_HEAD_RECOMPUTE (no range limit): repeat the step", applied_max, issued, partial);
    }
    return fail(m, IL_ERR_TIMEOUT, "a bounded device-side wait expired (code %u); %d of %d optimiser updates since the "
                "last il_sync were applied%s", first, applied_max, issued, partial);
  }
  return IL_OK;
  });
}

extern "C" il_status il_get_boundary(il_model* m, int k, float* host, size_t count) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (k < 0 || k > m->K || !host) return fail(m, IL_ERR_INVALID_ARG, "boundary %d out of range", k);
  if (!m->batch_set || (k > 0 && !m->fwd_done[k - 1]) || (k == 0 && !m->fwd_done[0])) return fail(m, IL_ERR_STATE, "boundary %d not computed in this step", k);
  if (count != (size_t)m->ntok * m->d) return fail(m, IL_ERR_INVALID_ARG, "boundary has %zu elements, got %zu", (size_t)m->ntok * m->d, count);
  IL_TRY(sync_devices(m));
  IL_TRY(copy_sync(m, k > 0 ? k - 1 : 0, host, m->a[k], count * 4, cudaMemcpyDeviceToHost));
  return IL_OK;
  });
}

extern "C" int il_head_mode(const il_model* m) { return m ? m->head_mode : -1; }

extern "C" il_status il_stats(const il_model* m, long long* device_bytes, long long* kernel_launches) {
  return guarded([&]() -> il_status {
  if (!m) return IL_ERR_INVALID_ARG;
  if (device_bytes) *device_bytes = m->bytes;
  if (kernel_launches) *kernel_launches = m->launches;
  return IL_OK;
  });
}

extern "C" il_status il_profile(il_model* m, int enable) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  IL_TRY(sync_devices(m));
  for (auto& r : m->prof_recs) { m->prof_pool.push_back(r.a); m->prof_pool.push_back(r.b); }
  m->prof_recs.clear();
  m->prof = enable == 2 ? 2 : (enable != 0 ? 1 : 0);
  return IL_OK;
  });
}

extern "C" il_status il_profile_read(il_model* m, double* gemm_ms, long long* gemm_launches, double* gemm_flops) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  IL_TRY(sync_devices(m));
  double ms = 0, fl = 0;
  for (auto& r : m->prof_recs) {
    float t = 0;
    IL_CUDA(m, cudaEventElapsedTime(&t, r.a, r.b));
    ms += t;
    fl += r.flops;
  }
  if (gemm_ms) *gemm_ms = ms;
  if (gemm_launches) *gemm_launches = (long long)m->prof_recs.size();
  if (gemm_flops) *gemm_flops = fl;
  for (auto& r : m->prof_recs) { m->prof_pool.push_back(r.a); m->prof_pool.push_back(r.b); }
  m->prof_recs.clear();
  return IL_OK;
  });
}

extern "C" il_status il_nwise_streams(int K, int n, int k, int* terms, int* count) {
  return guarded([&]() -> il_status {
  if (K < 1 || n < 1 || n > K || k < 0 || k >= K || !count) return IL_ERR_INVALID_ARG;
  const std::vector<int> t = terms_of(k, K, n);
  *count = (int)t.size();
  if (terms)
    for (size_t i = 0; i < t.size(); ++i) terms[i] = t[i];
  return IL_OK;
  });
}

// The tensors that cross component boundaries in one step, in the order the step issues them.
static void plan_transfers(int K, int n, int rule, std::vector<int>& out) {
  for (int b = 0; b + 1 < K; ++b) { out.push_back(0); out.push_back(b); out.push_back(-1); }
  for (int k = K - 2; k >= 0; --k) {
    if (rule == IL_RULE_SUM) {
      // stream j of component k continues the stream of component k+1 with the same termination level
      const std::vector<int> mine = terms_of(k, K, n), above = terms_of(k + 1, K, n);
      for (int t : mine)
        if (std::find(above.begin(), above.end(), t) != above.end()) { out.push_back(1); out.push_back(k); out.push_back(t); }
    } else {
      // one tensor per head above k that component k uses: the farthest head of its window (the one that updates
      // its parameters) and, unless k is the lowest component, the heads it relays further down
      const int hi = k + n - 1 < K - 1 ? k + n - 1 : K - 1;
      if (hi > k) { out.push_back(1); out.push_back(k); out.push_back(hi); }
      if (k > 0)
        for (int h = k + 1; h <= hi; ++h)
          if (h != hi && h < k + n - 1) { out.push_back(1); out.push_back(k); out.push_back(h); }
    }
  }
}

extern "C" il_status il_pipeline_transfers(int K, int n, int rule, int* records, int capacity, int* count) {
  return guarded([&]() -> il_status {
  if (K < 1 || n < 1 || n > K || !count || capacity < 0) return IL_ERR_INVALID_ARG;
  if (rule != IL_RULE_SUM && rule != IL_RULE_FAR && rule != IL_RULE_MEAN) return IL_ERR_INVALID_ARG;
  std::vector<int> plan;
  plan_transfers(K, n, rule, plan);
  *count = (int)plan.size() / 3;
  if (records)
    for (int i = 0; i < *count && i < capacity; ++i)
      for (int j = 0; j < 3; ++j) records[3 * i + j] = plan[3 * i + j];
  return IL_OK;
  });
}

extern "C" il_status il_pipeline_last_transfers(il_model* m, int* records, int capacity, int* count) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (!count || capacity < 0) return fail(m, IL_ERR_INVALID_ARG, "NULL count");
  *count = (int)m->xfer_log.size() / 3;
  if (records)
    for (int i = 0; i < *count && i < capacity; ++i)
      for (int j = 0; j < 3; ++j) records[3 * i + j] = m->xfer_log[3 * i + j];
  return IL_OK;
  });
}

extern "C" il_status il_error_word(il_model* m, int k, void** device_ptr) {
  return guarded([&]() -> il_status {
  IL_TRY(check_model(m));
  if (k < 0 || k >= m->K || !device_ptr) return fail(m, IL_ERR_INVALID_ARG, "component %d out of range or NULL output", k);
  *device_ptr = m->err_word[k];
  return IL_OK;
  });
}

extern "C" const char* il_last_error(const il_model* m) { return m ? m->err.c_str() : "null model"; }

extern "C" const char* il_status_string(il_status s) {
  switch (s) {
    case IL_OK: return "IL_OK";
    case IL_ERR_INVALID_ARG: return "IL_ERR_INVALID_ARG";
    case IL_ERR_STATE: return "IL_ERR_STATE";
    case IL_ERR_OOM: return "IL_ERR_OOM";
    case IL_ERR_CUDA: return "IL_ERR_CUDA";
    case IL_ERR_TIMEOUT: return "IL_ERR_TIMEOUT";
    case IL_ERR_NONFINITE: return "IL_ERR_NONFINITE";
  }
  return "unknown";
}

// =================================================================================================
// operator-level entry points
// =================================================================================================
static il_status op_status(cudaError_t e) {
  if (e == cudaSuccess) return IL_OK;
  return e == cudaErrorInvalidValue ? IL_ERR_INVALID_ARG : IL_ERR_CUDA;
}

extern "C" il_status il_op_gemm(const il_gemm_desc* q, unsigned* err_word, void* stream) {
  return guarded([&]() -> il_status {
  if (!q || !err_word) return IL_ERR_INVALID_ARG;
  GemmArgs g = gemm_args(q->M, q->N, q->K, q->A, q->lda, q->a_mn_major, q->B, q->ldb, q->b_mn_major, q->epilogue, q->C, q->ldc);
  g.C2 = q->C2; g.bias = q->bias; g.resid = q->resid; g.aux = q->aux; g.ld_aux = q->ld_aux; g.aux_rows = q->aux_rows; g.colsum = q->colsum;
  g.accumulate = q->accumulate; g.split_k = q->split_k; g.targets = q->targets; g.part_max = q->part_max; g.part_sum = q->part_sum;
  g.part_ld = q->part_ld; g.tgt_logit = q->tgt_logit; g.lse = q->lse; g.scale = q->scale; g.col0 = q->col0;
  g.tile_blocks = q->tile_blocks; g.rowscale = q->rowscale; g.store_exp = q->store_exp;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return IL_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return IL_ERR_CUDA;
  return op_status(gemm_launch(g, err_word, sms, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_attention_fwd(const void* qkv, void* o, float* lse, int B, int T, int H, int dh, void* stream) {
  return guarded([&]() -> il_status {
  if (!qkv || !o || !lse || B < 1 || T < 1 || H < 1) return IL_ERR_INVALID_ARG;
  return op_status(attention_fwd((const bf16*)qkv, (bf16*)o, lse, B, T, H, dh, nullptr, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_attention_bwd(const void* qkv, const void* o, const float* lse, const void* dout, void* dqkv,
                                         float* delta, int NB, int B, int T, int H, int dh, void* stream) {
  return guarded([&]() -> il_status {
  if (!qkv || !o || !lse || !dout || !dqkv || !delta || B < 1 || NB < 1 || T < 1 || H < 1) return IL_ERR_INVALID_ARG;
  return op_status(attention_bwd((const bf16*)qkv, (const bf16*)o, lse, (const bf16*)dout, (bf16*)dqkv, delta, nullptr, NB, B, T,
                                 H, dh, nullptr, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_attention_bwd_one_sweep(const void* qkv, const void* o, const float* lse, const void* dout,
                                                   void* dqkv, float* delta, float* dq_acc, int NB, int B, int T, int H,
                                                   int dh, unsigned* err_word, void* stream) {
  return guarded([&]() -> il_status {
  if (!qkv || !o || !lse || !dout || !dqkv || !delta || !dq_acc || B < 1 || NB < 1 || T < 1 || H < 1) return IL_ERR_INVALID_ARG;
  if (dh != 32 && dh != 64) return IL_ERR_INVALID_ARG;
  return op_status(attention_bwd((const bf16*)qkv, (const bf16*)o, lse, (const bf16*)dout, (bf16*)dqkv, delta, dq_acc, NB, B, T,
                                 H, dh, err_word, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_wait_probe(unsigned* err_word, unsigned limit_us, void* stream) {
  return guarded([&]() -> il_status {
  if (!err_word || limit_us < 1 || limit_us > 1000000u) return IL_ERR_INVALID_ARG;
  return op_status(wait_probe(err_word, 1000ull * limit_us, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_layernorm_fwd(const float* x, const float* gamma, const float* beta, void* y, float* mean,
                                         float* rstd, int rows, int d, float eps, void* stream) {
  return guarded([&]() -> il_status {
  if (!x || !gamma || !beta || !y || !mean || !rstd || rows < 1 || d < 8 || d % 8) return IL_ERR_INVALID_ARG;
  return op_status(layernorm_fwd(x, gamma, beta, (bf16*)y, mean, rstd, rows, d, eps, reinterpret_cast<cudaStream_t>(stream)));
  });
}

extern "C" il_status il_op_layernorm_bwd(const void* dy, int dy_is_f32, const float* x, const float* mean, const float* rstd,
                                         const float* gamma, const float* resid, float* dx, void* dx_bf16, float* dgamma,
                                         float* dbeta, int rows, int x_rows, int d, void* stream) {
  return guarded([&]() -> il_status {
  if (!dy || !x || !mean || !rstd || !gamma || !dx || rows < 1 || x_rows < 1 || d < 8 || d % 8) return IL_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dgamma && dbeta) {
    cudaError_t e = layernorm_bwd_params(dy, dy_is_f32, x, mean, rstd, dgamma, dbeta, x_rows < rows ? x_rows : rows, d, st);
    if (e != cudaSuccess) return op_status(e);
  }
  return op_status(layernorm_bwd_rows(dy, dy_is_f32, x, mean, rstd, gamma, resid, dx, (bf16*)dx_bf16, rows, x_rows, d, st));
  });
}

extern "C" il_status il_op_layernorm_bwd_fused(const void* dy, const float* x, const float* mean, const float* rstd,
                                               const float* gamma, const float* resid, float* dx, void* dx_bf16,
                                               float* dgamma, float* dbeta, float* colsum, int rows, int x_rows, int d,
                                               void* stream) {
  return guarded([&]() -> il_status {
  if (!dy || !x || !mean || !rstd || !gamma || !dx || !dgamma || !dbeta || rows < 1 || x_rows < 1) return IL_ERR_INVALID_ARG;
  if (d < 128 || d > 1024 || d % 128) return IL_ERR_INVALID_ARG;
  return op_status(layernorm_bwd_fused((const bf16*)dy, x, mean, rstd, gamma, resid, dx, (bf16*)dx_bf16, dgamma, dbeta, colsum,
                                       rows, x_rows, d, reinterpret_cast<cudaStream_t>(stream)));
  });
}
