/*
 * fax.h -- C ABI of the single-GPU decoder-only Transformer training step
 * (forward pass, loss, backward pass and Adam update; arXiv 2204.06514,
 * Fig. 3 caption, Table 1 caption, Sec. 3) for NVIDIA B200 (sm_100a).
 *
 * Conventions that hold for every call
 *  - Plain C.  Every function returns a fax_status (0 = FAX_OK, negative =
 *    error class); nothing throws across the boundary.
 *  - Ownership: the caller owns every buffer (inputs, outputs, parameters,
 *    optimizer state, saved activations, scratch) and the CUDA stream.  The
 *    library allocates no device memory in any compute call; fax_create
 *    allocates one small device status block that fax_destroy frees.
 *  - Unless a parameter is marked "host", pointers are DEVICE pointers on the
 *    context's device, 16-byte aligned (tensor bases: 256-byte aligned), dense
 *    row-major with the innermost dimension contiguous.
 *  - Compute calls enqueue work on the context's stream and return without
 *    synchronising, except the *_host entry points and an explicit host loss
 *    readback, which synchronise the stream before returning.
 *  - Calls on one context are not thread-safe; contexts are independent.
 *  - Current device: fax_create and fax_destroy make the context's device
 *    current themselves (and leave it current); every other call must be made
 *    with the context's device current on the calling thread.  A process may
 *    hold contexts on several devices.
 *  - Inputs are never modified unless stated (AdamW updates state in place).
 *  - Shapes: tokens N = batch*seq; d_model = n_heads*head_dim; head_dim is 64
 *    or 128; in FAX_PREC_BF16 d_model, d_ff and vocab must be multiples of 128
 *    and N a multiple of 128 (tile constraints of the tensor-core kernels);
 *    otherwise FAX_ERR_UNSUPPORTED_SHAPE.  FAX_PREC_FP32_VALIDATE accepts any
 *    positive sizes with d_model and d_ff multiples of 4.
 *  - Weight layout: every linear weight is [in, out] row-major (y = x W).
 *    w_qkv is [d, 3d] with column blocks q | k | v, head h at columns
 *    h*head_dim .. (h+1)*head_dim-1 of each block.  wte is [vocab, d], wpe is
 *    [max_seq, d].
 *  - Element type "T" below is bf16 in FAX_PREC_BF16 and float in
 *    FAX_PREC_FP32_VALIDATE.
 */
#ifndef FAX_H_
#define FAX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t fax_status;
enum {
  FAX_OK = 0,
  FAX_ERR_INVALID_ARG = -1,         /* null / misaligned pointer, inconsistent cfg */
  FAX_ERR_UNSUPPORTED_SHAPE = -2,   /* violates the documented tile constraints */
  FAX_ERR_WORKSPACE_TOO_SMALL = -3, /* saved_bytes / scratch_bytes below *_sizes */
  FAX_ERR_CUDA = -4,                /* a CUDA call failed: see fax_last_cuda_error */
  FAX_ERR_ARCH = -5,                /* device is not compute capability 10.x */
  FAX_ERR_TIMEOUT = -6              /* a bounded device-side wait expired */
};

typedef struct fax_ctx fax_ctx;

/* Human-readable name of a status code (static storage, never NULL). */
const char* fax_status_string(fax_status s);

/* Create a context bound to a device ordinal and a CUDA stream (a cudaStream_t
 * passed as void*; NULL = the legacy default stream).  Fails with FAX_ERR_ARCH
 * on a device that is not sm_100.  `out` is a host pointer. */
fax_status fax_create(fax_ctx** out, int32_t device_ordinal, void* cuda_stream);
fax_status fax_destroy(fax_ctx* ctx);

/* Raw cudaError_t of the last failing CUDA call on this context (0 if none). */
int32_t fax_last_cuda_error(const fax_ctx* ctx);

/* Synchronise the stream, then read and clear the device status word that
 * kernels set when one of their bounded waits gives up.  Returns FAX_OK,
 * FAX_ERR_TIMEOUT or FAX_ERR_CUDA.  `detail_host` (host, may be NULL) receives
 * a kernel-specific code saying which wait expired. */
fax_status fax_check_device_status(fax_ctx* ctx, int32_t* detail_host);

/* Number of kernel launches this context has enqueued since creation. */
uint64_t fax_launch_count(const fax_ctx* ctx);

/* Per-kernel profile.  Between fax_profile_begin and fax_profile_end every
 * operator launch on this context is bracketed by a pair of CUDA events on the
 * context's stream.  fax_profile_end synchronises the stream and fills `out`
 * (HOST array of n_out >= FAX_KERNEL_CLASSES entries, indexed by kernel class)
 * with, per class: operator launches, summed device milliseconds, summed
 * algorithmic FLOPs (2 per multiply-add) and summed algorithmic bytes (what the
 * operator must read and write once).  Profiling costs two event records per
 * launch, so timed runs keep it off. */
#define FAX_KERNEL_CLASSES 10
typedef struct { int64_t launches; double ms, flops, bytes; } fax_profile_entry;
fax_status fax_profile_begin(fax_ctx* ctx);
fax_status fax_profile_end(fax_ctx* ctx, fax_profile_entry* out, int32_t n_out);
/* Name of a kernel class ("gemm_tcgen05", "attention_fwd", "layernorm_fwd", "adamw", ...). */
const char* fax_kernel_class_name(int32_t cls);

typedef enum { FAX_PREC_BF16 = 0, FAX_PREC_FP32_VALIDATE = 1 } fax_precision;

/* One pre-LayerNorm decoder block with a causal mask (always causal). */
typedef struct {
  int32_t batch, seq, d_model, n_heads, head_dim, d_ff;
  float ln_eps;
  int32_t prec; /* fax_precision */
  /* 0: forward keeps both LayerNorm outputs and GELU(h) in the saved arena.  1: it keeps them only in the
   * scratch arena for its own use and backward recomputes them (two LayerNorm passes and one GELU pass
   * more per block) with the same kernels, so the gradients are the same: the saved arena shrinks by
   * N*(2d + f) elements per block.  Forward then needs the scratch arena too. */
  int32_t recompute;
} fax_block_cfg;

/* Compute-precision parameters (type T), in this order everywhere. */
typedef struct {
  const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o,
             *ln2_g, *ln2_b, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
} fax_block_params;

/* float32 gradients of the same twelve tensors. */
typedef struct {
  float *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o,
        *ln2_g, *ln2_b, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
} fax_block_grads;

/* Bytes the caller must provide for the saved-activation arena and for the
 * scratch arena of one block.  Host pointers. */
fax_status fax_block_sizes(const fax_block_cfg* cfg, size_t* saved_bytes, size_t* scratch_bytes);

/* Where the pieces live inside the two block arenas (byte offsets from the
 * arena base), for inspection, checkpointing and tests.  saved_off[13]: x, a
 * (LN1 out), qkv, o, x1, m (LN2 out), h, g, mu1, rstd1, mu2, rstd2, lse
 * ((size_t)-1 for a, m, g when cfg->recompute is set: they are not saved).
 * scratch_off[4], valid after fax_block_backward: dh [N,f], dqkv [N,3d],
 * da [N,d] (gradient at LN1's output), dx1 [N,d].  Host pointers. */
fax_status fax_block_arena_layout(const fax_block_cfg* cfg, size_t* saved_off, size_t* scratch_off);

/* Forward pass of the block (Fig. 3 "forward pass"):
 *   a = LN(x; ln1)            qkv = a Wqkv + bqkv
 *   o = causal multi-head softmax attention of qkv (log-sum-exp kept)
 *   x1 = x + o Wo + bo        m = LN(x1; ln2)
 *   h = m W1 + b1             g = GELU_tanh(h)          y = x1 + g W2 + b2
 * x [N,d] T in; y [N,d] T out; `saved` receives what backward needs
 * (x, LN statistics, a, qkv, o, log-sum-exp, x1, m, h, g).  y may not alias x.
 * `scratch` is used (and must hold fax_block_sizes' scratch bytes) only when cfg->recompute is set. */
fax_status fax_block_forward(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_params* params,
                             const void* x, void* y, void* saved, size_t saved_bytes,
                             void* scratch, size_t scratch_bytes);

/* Backward pass of the block (Fig. 3 "backward pass"): given dy [N,d] T and
 * the arena fax_block_forward filled, writes dx [N,d] T and the twelve float32
 * parameter gradients (accumulate != 0: adds to them instead of overwriting).
 * `grads` is a host struct of device pointers. */
fax_status fax_block_backward(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_params* params,
                              const void* dy, const void* saved, size_t saved_bytes,
                              void* dx, const fax_block_grads* grads, int32_t accumulate,
                              void* scratch, size_t scratch_bytes);

/* AdamW (Adam, Table 1 caption, with decoupled weight decay) on float32
 * master weights (Sec. 3: parameters are stored as float32).  Per element, at
 * step t >= 1:
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2
 *   w <- w - lr*wd*w - lr * (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps)
 * w, m, v are updated in place; if w_compute != NULL the bf16 rounding of the
 * new w is written there.  g is float32, or bf16 when grad_is_bf16 != 0. */
typedef struct {
  float* w; float* m; float* v;
  const void* g;
  void* w_compute;
  uint64_t n;
  float weight_decay;
} fax_adamw_tensor;

typedef struct {
  float lr, beta1, beta2, eps;
  int32_t step;          /* t >= 1 */
  int32_t grad_is_bf16;
} fax_adamw_hparams;

/* `tensors` is a HOST array of n_tensors descriptors of device buffers. */
fax_status fax_adamw_step(fax_ctx* ctx, const fax_adamw_tensor* tensors, int32_t n_tensors,
                          const fax_adamw_hparams* hp);

/* The whole-step calls (fax_block_step*, fax_lm_step*) run the AdamW update of
 * each tensor on a second stream owned by the context as soon as that tensor's
 * gradient is complete and its old value is no longer needed, i.e. under the
 * rest of the backward pass; the calls join that stream before they return
 * control of the main stream.  enable = 0 keeps everything on the main stream.
 * Results are identical either way.  Default: enabled. */
fax_status fax_set_adamw_overlap(fax_ctx* ctx, int32_t enable);

/* Fused update: in the whole-step calls the AdamW update of the four weight
 * matrices of a block happens in the epilogue of the GEMM that produces their
 * gradient (w, m, v read and written there, the bf16 copy refreshed), so the
 * float32 gradient does not go to HBM and back: 26 instead of 34 bytes of
 * traffic per parameter.  Where the kernel slices K (few output tiles) the
 * ordinary path is used.  With keep_gradients = 0 the weight-matrix gradients
 * of fused tensors are NOT stored in st->...g (biases, LayerNorm and embedding
 * gradients always are); with keep_gradients != 0 they are stored as well.
 * Same arithmetic as the separate update.  Default: disabled. */
fax_status fax_set_fused_update(fax_ctx* ctx, int32_t enable, int32_t keep_gradients);

/* fax_block_step and fax_lm_step replay a CUDA graph of the step from the third
 * call on with the same configuration and the same buffers (first call: run as
 * is; second call: captured on the context's stream in thread-local capture
 * mode; later calls: the AdamW scalars are patched into the graph and it is
 * launched).  Up to 8 graphs are kept per context.  enable = 0 turns this off
 * and drops the graphs.  Do not call the whole-step functions while the stream
 * is itself being captured by the caller.  Default: enabled. */
fax_status fax_set_graph_replay(fax_ctx* ctx, int32_t enable);

/* GEMMs whose M and N are multiples of 256 run on pairs of SMs (two-CTA
 * clusters, one 256 x 256 tile per pair); enable = 0 keeps every GEMM on the
 * one-CTA 128 x N kernel.  Same arithmetic either way.  Default: enabled. */
fax_status fax_set_gemm_two_cta(fax_ctx* ctx, int32_t enable);

/* Kernels are launched with programmatic dependent launch allowed: a kernel's
 * blocks may become resident, and run their set-up, while the kernel before it
 * on the stream is finishing; each kernel waits for that predecessor to
 * complete before it touches global memory, so results are the same.
 * enable = 0 launches every kernel fully serialised.  Default: enabled. */
fax_status fax_set_dependent_launch(fax_ctx* ctx, int32_t enable);

/* Tile order of the GEMMs.  The output tiles are visited in groups that keep
 * one operand's panels (a tile's rows or columns over all of K) in L2 from one
 * wave of tiles to the next while the other operand streams past once per
 * group; the group is as large as `bytes` of L2 allow, along the dimension
 * that costs fewer DRAM reads.  bytes = 0 restores the fixed order (groups of
 * 8 row-tiles).  Results are bit-identical for every value.  Default: 48e6. */
fax_status fax_set_gemm_l2_budget(fax_ctx* ctx, int64_t bytes);

/* Which attention-backward kernel runs.  mode 0: one 128-query tile in flight,
 * four row warps (head_dim 64 and 128).  mode 1: sixteen row warps with half-tile
 * hand-offs (both head dims).  mode 2 (default): as 1, and at head_dim 64 the
 * kernel that keeps two score tiles in flight (the exponentials of the next
 * query tile run while the tensor core works on the current one).  Same
 * arithmetic in every mode (the float32 dQ additions arrive in another order).
 * Other values: FAX_ERR_INVALID_ARG. */
fax_status fax_set_attention_backward_two_chains(fax_ctx* ctx, int32_t enable);

/* One trainable tensor of a training state: float32 master, compute-precision
 * copy (bf16; in FP32_VALIDATE may equal w or be NULL), Adam moments, float32
 * gradient, element count and its weight decay. */
typedef struct {
  float* w; void* w_compute; float* m; float* v; float* g;
  uint64_t n;
  float weight_decay;
} fax_param;

typedef struct {
  fax_param ln1_g, ln1_b, w_qkv, b_qkv, w_o, b_o, ln2_g, ln2_b, w_fc1, b_fc1, w_fc2, b_fc2;
} fax_layer_state;

typedef struct {
  fax_layer_state layer;
  void* saved; size_t saved_bytes;
  void* scratch; size_t scratch_bytes;
} fax_block_state;

/* One whole training step of a single block: forward, backward (gradients
 * overwritten), AdamW on the twelve tensors.  x, dy in; y, dx out (device).
 * Backward reads x in place, so afterwards the saved arena holds this step's
 * activations but no copy of x (it does when dx == x); a later
 * fax_block_backward on that arena needs a fax_block_forward first.
 * hp is checked before anything is enqueued (step >= 1, betas in [0, 1), lr
 * and eps finite, eps >= 0): FAX_ERR_INVALID_ARG otherwise, on every call. */
fax_status fax_block_step(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_state* st,
                          const void* x, const void* dy, void* y, void* dx,
                          const fax_adamw_hparams* hp);

/* Same step with HOST buffers (pinned memory recommended): copies x and dy to
 * the device (staged in the scratch arena), runs the step, copies y and dx
 * back and synchronises.  dy travels to the device and y back to the host on
 * a copy stream owned by the context while forward / backward run.  scratch must hold fax_block_sizes' bytes plus
 * 4*N*d*sizeof(T) of staging (fax_block_host_scratch_bytes). */
fax_status fax_block_host_scratch_bytes(const fax_block_cfg* cfg, size_t* scratch_bytes);
fax_status fax_block_step_host(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_state* st,
                               const void* x_host, const void* dy_host, void* y_host, void* dx_host,
                               const fax_adamw_hparams* hp);

/* N-layer language model: token + learned position embedding, n_layers
 * blocks, final LayerNorm, output projection tied to wte, mean softmax
 * cross-entropy over all batch*seq positions. */
typedef struct {
  int32_t n_layers, vocab, max_seq;
  fax_block_cfg block;
  int32_t head_rows;   /* rows of logits held at a time by the output projection + loss; 0 = as many as
                          fit a 4 GiB logits buffer (at least 8192).  Positive values must be multiples of
                          128; the head then walks the batch*seq rows in chunks of that many (the last
                          one shorter), adding each chunk's share into the gradient of wte. */
} fax_lm_cfg;

typedef struct {
  fax_param wte, wpe, lnf_g, lnf_b;
  const fax_layer_state* layers;   /* HOST array [n_layers] */
  void* saved; size_t saved_bytes;
  void* scratch; size_t scratch_bytes;
} fax_lm_state;

fax_status fax_lm_sizes(const fax_lm_cfg* cfg, size_t* saved_bytes, size_t* scratch_bytes);

/* Layout of the LM arenas (byte offsets, host pointers): act_off[n_layers+1]
 * (input of block l; last = output of the last block), layer_saved_off[n_layers]
 * (base of block l's saved pieces, laid out as fax_block_arena_layout's
 * saved_off minus its x entry, which is act_off[l]), xf_off (final LayerNorm
 * output), all in the saved arena; row_loss_off (per-token loss, float [N])
 * and block_scratch_off (base of the block scratch, as scratch_off above) in
 * the scratch arena. */
fax_status fax_lm_arena_layout(const fax_lm_cfg* cfg, size_t* act_off, size_t* layer_saved_off,
                               size_t* xf_off, size_t* row_loss_off, size_t* block_scratch_off);

/* Full LM training step (Fig. 3: forward pass, loss, backward pass; then the
 * Adam update): ids, targets are device int32 [batch, seq].  Gradients of
 * every tensor are overwritten in st->...g, then AdamW updates every tensor.
 * The mean loss is written to loss_device (float, device); if loss_host is not
 * NULL the stream is synchronised and the loss also copied there. */
fax_status fax_lm_step(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                       const int32_t* ids, const int32_t* targets,
                       const fax_adamw_hparams* hp, float* loss_device, float* loss_host);

/* Forward + loss + backward only (no update): for gradient checks. */
fax_status fax_lm_forward_backward(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                   const int32_t* ids, const int32_t* targets, float* loss_device);

/* Gradient accumulation over micro-batches: forward + loss + backward of one
 * micro-batch, its gradients scaled by grad_scale (normally 1 / number of
 * micro-batches: the loss of each call is the mean over its own batch*seq
 * tokens) and written (accumulate = 0) or added (accumulate != 0) to st->...g.
 * loss_device receives this micro-batch's unscaled mean loss.  After the last
 * micro-batch fax_lm_apply_adamw updates every tensor from the accumulated
 * gradients.  k calls on k micro-batches followed by fax_lm_apply_adamw equal
 * one fax_lm_step on the concatenated batch. */
fax_status fax_lm_accumulate(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                             const int32_t* ids, const int32_t* targets, float* loss_device,
                             int32_t accumulate, float grad_scale);
fax_status fax_lm_apply_adamw(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                              const fax_adamw_hparams* hp);

/* Same as fax_lm_step with HOST ids / targets (int32 [batch, seq], pinned
 * recommended): copies them into the head of the scratch arena, runs the
 * step, copies the loss back and synchronises. */
fax_status fax_lm_step_host(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                            const int32_t* ids_host, const int32_t* targets_host,
                            const fax_adamw_hparams* hp, float* loss_device, float* loss_host);

#ifdef __cplusplus
}
#endif
#endif /* FAX_H_ */
