/*
 * il.h — C ABI of the interlocking-backpropagation training-step library (CUDA, sm_100a).
 *
 * One il_model is a decoder-only Transformer language model cut into K contiguous
 * components ("modules", Sec. 3 of the paper: f = f_cK o ... o f_c1), each of
 * `layers_per_component` pre-LN blocks, with an auxiliary LM head h_ck (LayerNorm + untied
 * linear map to the vocabulary) after every component and the local loss
 *     L_ck(x, y) = L(h_ck(f_ck o ... o f_c1 (x)), y)            (Sec. 3, unnumbered equations)
 * with L the mean next-token cross-entropy.  One training step is
 *     il_set_batch -> il_forward_component(0..K-1) -> il_aux_head_loss(0..K-1)
 *                  -> il_backward_nwise -> il_adamw_step
 * where il_backward_nwise applies the n-wise rule (Sec. 3, Fig. 2): the gradient of head h
 * flows through component h and across n-1 component boundaries and then stops; the
 * contributions of all heads crossing a component are summed.  n = 1 is local learning,
 * n = K is ordinary backpropagation of the sum of the K head losses.
 *
 * Conventions
 *  - Every call returns il_status.  Nothing throws, aborts or exits across this boundary.
 *    On an error other than IL_ERR_CUDA the model stays usable and outputs are untouched.
 *  - The library owns all device memory it obtains (through il_options.alloc when given,
 *    cudaMalloc otherwise) and every string it returns.  The caller owns every buffer it
 *    passes; "host" pointers are ordinary host memory, "device" pointers are CUDA device
 *    memory on the model's device.  Inputs are copied before the call returns unless the
 *    call is documented as asynchronous on device pointers.
 *  - Components, heads and tensors are 0-based.  Matrices are row-major [out, in].
 *  - Work is issued on K CUDA streams (component k on stream k); calls return once the
 *    work is enqueued unless stated otherwise.  One host thread per model.
 *  - Kernels are launched with programmatic stream serialization: a kernel may become
 *    resident while its predecessor in the stream drains, and waits (griddepcontrol.wait)
 *    before it touches global memory.  Stream order as seen by the caller is unchanged.
 *    IL_NO_DEPENDENT_LAUNCH=1 in the environment (read once) launches the ordinary way.
 *  - Arithmetic: bf16 tensor-core operands, fp32 accumulation, fp32 residual stream,
 *    fp32 master weights, gradients and optimiser state.
 */
#ifndef IL_H_
#define IL_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct il_model il_model;

typedef enum {
  IL_OK = 0,
  IL_ERR_INVALID_ARG = 1, /* bad shape, NULL pointer, index out of range, n outside [1,K]          */
  IL_ERR_STATE = 2,       /* call order violated (e.g. backward before all K forwards + losses)     */
  IL_ERR_OOM = 3,         /* the allocator returned NULL                                            */
  IL_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; see il_last_error                   */
  IL_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (kernel returned early)             */
  IL_ERR_NONFINITE = 6    /* a head's log-sum-exp left [-80, 80] (the backward keeps exp(logit) in bf16)  */
} il_status;

typedef struct {
  int device;                       /* CUDA device ordinal                                           */
  int max_batch, max_seq;           /* activation arena is sized for max_batch*max_seq tokens;       */
                                    /* wpe has max_seq rows                                          */
  void* (*alloc)(size_t bytes, void* ctx);  /* device allocator hook (256-byte aligned); NULL => cudaMalloc */
  void (*free_)(void* p, void* ctx);
  void* alloc_ctx;
  void** streams;                   /* K cudaStream_t owned by the caller; NULL => library-created   */
  int n_streams;
  int use_bias;                     /* must be 1 (GPT-2 style biases on every projection); anything else is refused  */
  float ln_eps;                     /* <= 0 => 1e-5                                                  */
  int head_layers;                  /* Transformer blocks inside every auxiliary head, 0..64.  0: the  */
                                    /* head is LayerNorm + linear.  2 is the auxiliary network of the  */
                                    /* paper's Transformer runs (App. B.3: main network output ->      */
                                    /* 2 Transformer blocks -> embedding matrix -> logits); the blocks */
                                    /* have the main network's shape, the head's LayerNorm follows them */
  int head_mode;                    /* IL_HEAD_STORED (0, default) or IL_HEAD_RECOMPUTE (1): see il_aux_head_loss     */
  int placement;                    /* IL_PLACE_SINGLE (0, default): all components on `device`, component k+1 reads   */
                                    /* component k's output in place.  IL_PLACE_PIPELINE (1): the paper's placement,   */
                                    /* one module per accelerator (Sec. 3): component k lives on devices[k] with its   */
                                    /* parameters, optimiser state and activations; a_k travels forward and at most    */
                                    /* n-1 gradient tensors travel backward per boundary, each copied into a buffer    */
                                    /* the receiving device owns (see il_pipeline_transfers)                           */
  int attn_bwd;                     /* IL_ATTN_BWD_ONE_SWEEP (0, default): attention backward in one sweep that         */
                                    /* recomputes the scores once; dQ is summed over key tiles with fp32 atomics, so    */
                                    /* its last bit (and that of everything computed from it) may differ between runs.  */
                                    /* IL_ATTN_BWD_TWO_KERNELS (1): dK/dV and dQ in two kernels that each recompute the */
                                    /* scores; slower, every sum in a fixed order.  Head dims other than 32 / 64 always */
                                    /* take the two-kernel form                                                         */
  const int* devices;               /* IL_PLACE_PIPELINE: K device ordinals (n_devices == K), or NULL: every component */
  int n_devices;                    /* on `device`, still exchanged through the copy path.  Caller-owned streams[k]    */
                                    /* must belong to devices[k]; the alloc hook is called with that device current    */
} il_options;

enum { IL_HEAD_STORED = 0, IL_HEAD_RECOMPUTE = 1 };
enum { IL_PLACE_SINGLE = 0, IL_PLACE_PIPELINE = 1 };
enum { IL_ATTN_BWD_ONE_SWEEP = 0, IL_ATTN_BWD_TWO_KERNELS = 1 };

/* Build a model: K components x layers_per_component blocks, d_model, n_heads, d_ff, vocab, and the
 * n of the n-wise rule (Sec. 3: N in [1, number of modules]).  Requires d_model % n_heads == 0,
 * head dim in {32, 64, 80, 128, 256}, d_model % 8 == 0, d_ff % 8 == 0.  opt must be non-NULL with
 * max_batch, max_seq > 0.  Parameters start at zero (LayerNorm gains at one); set them with
 * il_set_param. */
il_status il_create(int K, int layers_per_component, int d_model, int n_heads, int d_ff, int vocab,
                    int n, const il_options* opt, il_model** out);
il_status il_destroy(il_model* m);
/* Change n (1..K) between steps. */
il_status il_set_n(il_model* m, int n);

/* Which heads update the parameters of component k (Sec. 3).  Every rule uses the same windows (head h reaches
 * components h .. h-n+1); they differ in the weight of head h in component k's parameter gradient:
 *   IL_RULE_SUM  (default) every head whose window covers k, weight 1 (n = K: backprop of the summed losses);
 *   IL_RULE_FAR  the paper's main-text rule: head min(k+n-1, K-1) alone (n = K: end-to-end on the last loss);
 *   IL_RULE_MEAN the variant of the paper's Transformer experiments: mean of heads k and min(k+n-1, K-1).
 * Head parameters always get their own loss's gradient.  Weighted rules need n <= 8. */
enum { IL_RULE_SUM = 0, IL_RULE_FAR = 1, IL_RULE_MEAN = 2 };
il_status il_set_rule(il_model* m, int rule);

/* Parameter registry.  Order and names: "wte" [V,d], "wpe" [max_seq,d] (component 0: the first
 * module holds the input projection, App. B.3), then per component k and layer l
 * "c{k}.l{l}.{ln1.g,ln1.b,attn.wqkv,attn.bqkv,attn.wo,attn.bo,ln2.g,ln2.b,mlp.w1,mlp.b1,mlp.w2,mlp.b2}",
 * then per head k its blocks "head{k}.l{j}.{the same twelve names}" (j < head_layers) followed by
 * "head{k}.{ln.g,ln.b,w}".  Everything named head{k}.* is a parameter of the auxiliary network of
 * component k and is updated from L_ck alone (Sec. 3).  Host fp32 buffers; `count` must equal the tensor size.
 * These calls synchronise the device. */
int il_num_tensors(const il_model* m);
il_status il_tensor_info(const il_model* m, int idx, const char** name, int* component, int* is_head,
                         int* rank, long long shape[2]);
il_status il_set_param(il_model* m, int idx, const float* host, size_t count);
il_status il_get_param(il_model* m, int idx, float* host, size_t count);
il_status il_get_grad(il_model* m, int idx, float* host, size_t count); /* after il_backward_nwise */
il_status il_get_opt_state(il_model* m, int idx, float* m_host, float* v_host, long long* step);
il_status il_set_opt_state(il_model* m, int idx, const float* m_host, const float* v_host, long long step);

/* One step.  tokens/targets: B*T int32 ids in [0, vocab), HOST pointers when on_device == 0
 * (copied with cudaMemcpyAsync before the call returns control; the caller may reuse the buffers
 * after il_sync or any synchronising call), DEVICE pointers when on_device != 0.  Ids outside
 * [0, vocab) are clamped on the device, never dereferenced out of bounds. */
il_status il_set_batch(il_model* m, const int* tokens, const int* targets, int B, int T, int on_device);
/* Forward of component k (Sec. 3: a_k = f_ck(a_{k-1}); k = 0 also performs the embedding lookup).
 * Must be called for k = 0..K-1 in order. */
il_status il_forward_component(il_model* m, int k);
/* Auxiliary head k (Sec. 3: h_ck and the local loss L_ck): LayerNorm, vocabulary projection and mean
 * cross-entropy.  The projection's epilogue turns each output tile into per-row softmax partials and the
 * target logit; the logits themselves are never stored.  What is kept for il_backward_nwise depends on
 * il_options.head_mode:
 *   IL_HEAD_STORED    the same epilogue also writes exp(logit) as a bf16 [B*T, vocab] matrix per head
 *                     (vocab * 2 bytes per token and head: 824 MB per head at 8192 tokens and a 50257-word
 *                     vocabulary); the backward runs its two contractions on that matrix without recomputing
 *                     anything.  Price besides the memory: every row's log-sum-exp must lie in [-80, 80]
 *                     (checked; a violation makes il_sync return IL_ERR_NONFINITE, skips the update and
 *                     switches the model to IL_HEAD_RECOMPUTE for all later steps, reusing the matrix's memory
 *                     as the chunk buffer: parameters and optimiser state are untouched, so the caller repeats
 *                     the step; il_head_mode reads the mode in force).
 *   IL_HEAD_RECOMPUTE nothing of size [B*T, vocab] is ever held: the backward walks the vocabulary in chunks of
 *                     8192 columns, forms the chunk's logits again, turns them into dZ in the epilogue and
 *                     feeds dZ to the two gradient contractions (one third more head flops, no range limit).
 * Needs il_forward_component(k).  loss_host != NULL makes the call wait for this head and return its loss;
 * NULL leaves it asynchronous. */
il_status il_aux_head_loss(il_model* m, int k, float* loss_host);
/* The head mode in force (IL_HEAD_STORED or IL_HEAD_RECOMPUTE; see above); -1 for a NULL model. */
int il_head_mode(const il_model* m);
/* Per-token negative log-likelihood of head k for the current step, fp32 [B*T] to host (their mean is
 * the head's loss).  Needs il_aux_head_loss(k); waits for it. */
il_status il_get_token_losses(il_model* m, int k, float* host, size_t count);
/* All K losses of the current step (waits for them). */
il_status il_get_losses(il_model* m, float* losses_host);
/* n-wise backward (Sec. 3, Fig. 2): for every head, back-propagation through the head and through
 * the n components below it, a stop at each window's lowest component input, contributions of
 * overlapping heads summed.  Overwrites all gradients.  Needs all K forwards and head losses. */
il_status il_backward_nwise(il_model* m);
/* Micro-batching (Sec. 3.1: a mini-batch is split into M micro-batches and one update follows).  With
 * M > 1 an update is M rounds of il_set_batch .. il_backward_nwise, one per micro-batch of equal size,
 * then il_adamw_step: the first il_backward_nwise of an update overwrites the gradients, the later ones
 * add to them, and each is scaled by 1/M, so that il_get_grad and il_adamw_step see the gradient of the
 * mean loss over the whole mini-batch.  An (M+1)-th il_backward_nwise and an il_adamw_step after fewer
 * than M return IL_ERR_STATE.  Calling this function (M >= 1; 1 is the default) starts a new update and
 * abandons gradients accumulated so far.  Losses are reported per micro-batch. */
il_status il_set_micro_batches(il_model* m, int micro_batches);
/* AdamW (decoupled weight decay on rank-2 tensors; weight_decay = 0 is the paper's Adam,
 * App. B.3: beta1 0.9, beta2 0.98, eps 1e-9).  Needs il_backward_nwise.  Increments the step.
 * The update kernels read the device-side error word: while it is set (a bounded wait expired, or a head left
 * the exp(logit) range) a component's parameters, Adam moments and bf16 copies are left untouched, and the next
 * il_sync reports the error and takes the skipped updates back off the step counter.  The check is per component
 * and per launch: a component whose update ran before another component raised the error keeps that update
 * (il_last_error then says so); the same holds for a head's vocabulary matrix, whose update is enqueued on a side
 * stream right behind the head's own backward and may therefore run before an error raised later in the step. */
il_status il_adamw_step(il_model* m, float lr, float beta1, float beta2, float eps, float weight_decay);
/* Wait for all enqueued work; reports device-side timeouts as IL_ERR_TIMEOUT and a head whose
 * log-sum-exp left [-80, 80] in il_backward_nwise as IL_ERR_NONFINITE (that step's gradients are invalid).
 * Reporting clears the error: the next step starts clean. */
il_status il_sync(il_model* m);
/* Boundary activation a_k, k = 0..K (a_0 = embeddings), fp32 [B*T, d] to host; synchronises. */
il_status il_get_boundary(il_model* m, int k, float* host, size_t count);
/* Bytes of device memory obtained so far, and kernels launched since creation. */
il_status il_stats(const il_model* m, long long* device_bytes, long long* kernel_launches);
/* Device time of the GEMM kernels launched since the last reset, measured with CUDA events on
 * their own streams when profiling is switched on (adds event records; off by default).
 * enable = 1: events only (with several component streams busy a kernel's interval includes its wait for
 * SMs); enable = 2: additionally every GEMM runs alone on the GPU (the other streams wait for it and it
 * for them), so the intervals are kernel durations — slower steps, for measurement only. */
il_status il_profile(il_model* m, int enable);
il_status il_profile_read(il_model* m, double* gemm_ms, long long* gemm_launches, double* gemm_flops);
/* Host-only helper (no device needed): the gradient streams component k carries under the n-wise rule
 * (Sec. 3, Fig. 2).  Head h stops at the input of component max(h-n+1, 0); the heads crossing component
 * k are grouped by that level.  Writes the distinct levels, descending, to terms[0..*count) (terms may be
 * NULL; it needs room for min(n, K) ints).  *count is the number of stacked backward passes of k. */
il_status il_nwise_streams(int K, int n, int k, int* terms, int* count);
/* Host-only: the tensors that cross component boundaries in one step of the pipeline placement (Sec. 3 and the
 * schedule of Fig. 3: activations are sent to the next accelerator, gradients back to the previous one), in the
 * order the step issues them.  Record i is records[3i .. 3i+2] = (direction, boundary, id): direction 0 = the
 * activation a_{boundary+1} from component `boundary` to component boundary+1 (id -1); direction 1 = one [B*T, d]
 * fp32 gradient tensor from component boundary+1 down to component `boundary`; id is, under IL_RULE_SUM, the
 * termination level of the gradient stream (the sum of the gradients of all heads crossing component boundary+1
 * that stop at or below the input of component id), and under the weighted rules the head whose gradient it is.
 * At most n-1 gradient tensors cross a boundary.  *count receives the number of records; at most `capacity` are
 * written (records may be NULL). */
il_status il_pipeline_transfers(int K, int n, int rule, int* records, int capacity, int* count);
/* The copies between components the pipeline placement actually issued since the last il_set_batch, in the same
 * record format (empty for IL_PLACE_SINGLE). */
il_status il_pipeline_last_transfers(il_model* m, int* records, int capacity, int* count);
/* Device address of the error word the kernels of component k report to (unsigned; 0 = no error; see il_sync).
 * For diagnostics and for tests of the error path: a caller may hand it to il_op_* calls as their err_word. */
il_status il_error_word(il_model* m, int k, void** device_ptr);
/* Host-only: the learning-rate schedule of the paper's Transformer runs (App. B.3),
 *   lr = d_model^-0.5 * min(step^-0.5, step * warmup_steps^-1.5),   step >= 1 (the paper: d_model 1024, warm-up 4000). */
il_status il_lr_schedule(long long step, int d_model, int warmup_steps, double* lr);
/* Host-only: the paper's time-per-batch model of synchronous depthwise model parallelism (Sec. 3.1):
 * A sequential accelerators (one module each), M micro-batches per mini-batch, N the n-wise parameter
 * (N = 1 local learning, N >= A end-to-end / GPipe), micro-batch cost c(M) = c0 + c1 / M.
 *   M = 1: 2N c;  M = 2 or A >= 2N-1: (N+1) M c;  otherwise (2+A-N) M c + 2 (2N-A-1) c.
 * *out is in the unit of c0 and c1 (the paper fits c0 = 0.025 s, c1 = 1.279 s to its Transformer runs).  It
 * models accelerators that idle while gradients travel; the single-GPU step of this library has no such idle
 * time, so this is a planning aid for the multi-device placement, not a prediction of il_* step times. */
il_status il_time_per_batch(int A, int M, int N, double c0, double c1, double* out);
/* The power of two M in [1, 2^max_log2] that minimises il_time_per_batch (App. C of the paper). */
il_status il_optimal_microbatches(int A, int N, double c0, double c1, int max_log2, int* M_out);
const char* il_last_error(const il_model* m); /* library-owned, valid until the next call on m */
const char* il_status_string(il_status s);

#ifdef __cplusplus
}
#endif
#endif /* IL_H_ */
