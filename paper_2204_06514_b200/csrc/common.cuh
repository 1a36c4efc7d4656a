// Shared host/device helpers of the CUDA library: context, status handling,
// launch bookkeeping and small numeric utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <vector>

#include "../../include/fax.h"

typedef __nv_bfloat16 bf16;

// Kernel classes of the per-kernel profile (order fixed by fax.h).
enum FaxKernelClass {
  KC_GEMM_TC = 0, KC_GEMM_SIMT, KC_ATTN_FWD, KC_ATTN_BWD, KC_LN_FWD, KC_LN_BWD, KC_ADAMW, KC_COLSUM,
  KC_EMBED, KC_XENT, KC_COUNT
};
struct FaxProfRec { int cls; cudaEvent_t e0, e1; double flops, bytes; };

struct FaxGemmPatch {
  cudaGraphNode_t node; cudaKernelNodeParams params;
  std::vector<unsigned char> blob;     // copy of the kernel's parameter struct, scalars patched per launch
  size_t sc_offset;
};
struct FaxGraphEntry {
  std::vector<FaxGemmPatch> gemm_nodes;
  uint64_t key;
  std::vector<unsigned char> material;   // the bytes the key was hashed from (compared on a hash hit)
  cudaGraph_t graph; cudaGraphExec_t exec;
  std::vector<cudaGraphNode_t> adam_nodes;
  std::vector<cudaKernelNodeParams> adam_params;
  uint64_t launches, last_use;
  bool failed;
};

// Device status block owned by the context: word 0 = error flag, word 1 = detail.
struct fax_ctx {
  int device;
  cudaStream_t stream;
  int32_t* dev_status;       // 2 x int32 on the device
  int32_t last_cuda_error;
  uint64_t launches;
  int sm_count;
  void* encode_tiled;        // cuTensorMapEncodeTiled, resolved at create
  bool prof_on;
  std::vector<FaxProfRec> prof;
  cudaStream_t side;         // optimizer stream: AdamW of finished tensors overlaps the rest of backward
  cudaEvent_t ev_fork, ev_join;
  cudaStream_t copy;         // host <-> device copies of the *_host entry points
  cudaEvent_t ev_copy_a, ev_copy_b;
  bool side_busy;
  bool overlap_adamw;
  bool use_graphs;           // whole-step calls are captured into CUDA graphs and replayed
  std::vector<FaxGraphEntry> graphs;
  uint64_t graph_clock;
  bool fused_update;         // whole-step calls fuse AdamW of the weight matrices into the dW GEMM epilogue
  bool keep_fused_grads;     // ... and still store those gradients
  bool use_2cta;             // GEMMs whose M and N are multiples of 256 use the two-CTA kernel
  bool use_pdl;              // kernels are launched with programmatic stream serialization allowed
  double gemm_l2_budget;     // bytes of L2 a GEMM may count on for the operand panels it keeps between waves (0: fixed raster)
  int attn_bwd_mode;         // attention backward: 0 one-tile kernel, 1 sixteen row warps, 2 also two score tiles in flight at head_dim 64
};

// Brackets the launches of one operator with CUDA events while profiling is on.
struct FaxProfScope {
  fax_ctx* c; int idx;
  FaxProfScope(fax_ctx* ctx, int cls, double flops, double bytes) : c(ctx), idx(-1) {
    if (!ctx->prof_on) return;
    FaxProfRec r; r.cls = cls; r.flops = flops; r.bytes = bytes; r.e0 = nullptr; r.e1 = nullptr;
    if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) return;
    cudaEventRecord(r.e0, ctx->stream);
    ctx->prof.push_back(r);
    idx = (int)ctx->prof.size() - 1;
  }
  ~FaxProfScope() { if (idx >= 0) cudaEventRecord(c->prof[idx].e1, c->stream); }
};

#define FAX_CUDA_TRY(ctx, expr)                                   \
  do {                                                            \
    cudaError_t e__ = (expr);                                     \
    if (e__ != cudaSuccess) {                                     \
      (ctx)->last_cuda_error = (int32_t)e__;                      \
      return FAX_ERR_CUDA;                                        \
    }                                                             \
  } while (0)

#define FAX_TRY(expr)                                             \
  do {                                                            \
    fax_status s__ = (expr);                                      \
    if (s__ != FAX_OK) return s__;                                \
  } while (0)

// Count a launch and pick up a launch-configuration error without syncing.
static inline fax_status fax_after_launch(fax_ctx* ctx) {
  ctx->launches++;
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    ctx->last_cuda_error = (int32_t)e;
    (void)cudaGetLastError();
    return FAX_ERR_CUDA;
  }
  return FAX_OK;
}

// Launch on the context's stream with programmatic dependent launch allowed: the grid may be
// scheduled while its predecessor on the stream is still running, so its blocks become resident
// as SMs free up and run their set-up (barrier initialisation, tensor-memory allocation,
// descriptor prefetch) under the predecessor's tail.  ONLY for kernels whose every thread calls
// fax_grid_dependency_wait() before its first access to global memory: that call returns once
// the predecessor has completed and its writes are visible, which keeps the stream's ordering.
template <typename... KArgs, typename... Args>
static inline void fax_launch(fax_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = ctx->stream;
  cudaLaunchAttribute attr = {};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = ctx->use_pdl ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);     // errors surface in fax_after_launch
}

// Kernels that need more than 48 KB of dynamic shared memory opt in once per device (the attribute is
// per device, a process may hold contexts on several): `done` is the call site's own flag array.
constexpr int FAX_MAX_DEVICES = 64;
template <typename K>
static inline fax_status fax_opt_in_shared_memory(fax_ctx* ctx, K* kernel, int bytes, bool* done) {
  const bool tracked = ctx->device >= 0 && ctx->device < FAX_MAX_DEVICES;
  if (tracked && done[ctx->device]) return FAX_OK;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) {
    ctx->last_cuda_error = (int32_t)e;
    return FAX_ERR_CUDA;
  }
  if (tracked) done[ctx->device] = true;
  return FAX_OK;
}

static inline bool fax_aligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) == 0; }
static inline size_t fax_round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline size_t fax_elem_size(int prec) { return prec == FAX_PREC_BF16 ? 2 : 4; }

// Bump allocator over a caller-provided arena (256-byte aligned pieces).
struct FaxArena {
  char* base; size_t off; size_t cap;
  FaxArena(void* b, size_t c) : base((char*)b), off(0), cap(c) {}
  void* take(size_t bytes) {
    size_t o = fax_round_up(off, 256);
    off = o + bytes;
    return base ? (void*)(base + o) : (void*)0;
  }
  size_t used() const { return fax_round_up(off, 256); }
};

// Counterpart of fax_launch in the kernel: blocks until the preceding grid on the stream has
// completed (a no-op when the kernel was launched without the attribute), then lets the grid
// that follows be scheduled behind this one.
__device__ __forceinline__ void fax_grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- device numeric helpers -------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// tanh-form GELU and its derivative, float32.
__device__ __forceinline__ float gelu_tanh_f(float h) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  float t = tanhf(c * (h + a * h * h * h));
  return 0.5f * h * (1.0f + t);
}
__device__ __forceinline__ float gelu_tanh_grad_f(float h) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  float t = tanhf(c * (h + a * h * h * h));
  return 0.5f * (1.0f + t) + 0.5f * h * (1.0f - t * t) * c * (1.0f + 3.0f * a * h * h);
}

// ---- internal operator interfaces (host functions that enqueue kernels) ------
enum FaxEpilogue {
  EPI_NONE = 0,        // C = acc
  EPI_BIAS = 1,        // C = acc + bias[n]
  EPI_BIAS_GELU = 2,   // C = acc + bias (pre-activation), aux = GELU(C)
  EPI_BIAS_RESID = 3,  // C = acc + bias + resid
  EPI_DGELU = 4,       // C = acc * GELU'(aux)          (aux read-only, [M,N])
  EPI_ADAMW = 5        // internal: acc is a weight gradient, consumed by AdamW in the epilogue
};

// AdamW fused into the epilogue of a weight-gradient GEMM: the accumulator tile is the
// gradient; w, m, v (float, [M,N] with the row pitch of C) are updated in place and the
// bf16 copy refreshed, so the gradient never travels to HBM and back.
struct FaxFusedAdam {
  float* w; float* m; float* v; void* w_compute;
  float weight_decay;
  float sc[8];               // lr, beta1, beta2, eps, 1/(1-beta1^t), 1/(1-beta2^t)
  bool keep_grad;            // also store the gradient to C
};

struct FaxGemm {
  int M, N, K;
  const void* A; int64_t lda; bool a_mn_major;  // false: A is [M,K] row-major; true: A is [K,M] row-major
  const void* B; int64_t ldb; bool b_mn_major;  // false: B is [N,K] row-major; true: B is [K,N] row-major
  void* C; int64_t ldc; bool c_f32;             // C is [M,N] row-major, type T or float
  bool accumulate;                              // C += result (float output only)
  int epi;
  const void* bias;                             // [N] type T
  const void* resid; int64_t ldr;               // [M,N] type T
  void* aux; int64_t ldaux;                     // [M,N] type T
  float alpha;                                  // scales acc before the epilogue
  const FaxFusedAdam* adam;                     // non-null: EPI_ADAMW (float C, epi NONE, no accumulate)
};

fax_status fax_gemm_simt(fax_ctx* ctx, int prec, const FaxGemm& g);
fax_status fax_gemm_tc(fax_ctx* ctx, const FaxGemm& g);       // bf16 tcgen05 path
bool fax_gemm_tc_supported(const FaxGemm& g);
bool fax_gemm_tc2_supported(const FaxGemm& g);                 // two-CTA 256 x 256 tiles
fax_status fax_gemm_tc2(fax_ctx* ctx, const FaxGemm& g);
// dispatch; allow_simt: a bf16 problem that the tensor-core kernels do not take may run on the SIMT kernel
// (otherwise FAX_ERR_UNSUPPORTED_SHAPE); kernel_class (optional) receives KC_GEMM_TC or KC_GEMM_SIMT
fax_status fax_gemm(fax_ctx* ctx, int prec, const FaxGemm& g, bool allow_simt = false, int* kernel_class = nullptr);
// Would fax_gemm run this (bf16) problem on a tensor-core kernel without slicing K?  Only then
// can AdamW be fused into its epilogue.
bool fax_gemm_can_fuse_adam(fax_ctx* ctx, const FaxGemm& g);
// If `func` is a GEMM kernel launched with EPI_ADAMW parameters at `param`, gives the size of the
// parameter struct and the offset of the six AdamW scalars in it (for graph replay).
bool fax_gemm_patch_info_1cta(const void* func, const void* param, size_t* size, size_t* sc_offset);
bool fax_gemm_patch_info_2cta(const void* func, const void* param, size_t* size, size_t* sc_offset);

fax_status fax_layernorm_fwd(fax_ctx* ctx, int prec, int rows, int d, const void* x, const void* gamma,
                             const void* beta, float eps, void* out, float* mu, float* rstd, void* x_copy);
// dx = (add ? add : 0) + LNbwd(da); partial: float scratch [2 * slabs * d] ([4 * slabs * d] with the sums).
// sum_add, sum_out (both or neither; need add): also sum_add[c] (+)= sum_r add[r, c] and
// sum_out[c] (+)= sum_r dx[r, c], taken inside the LayerNorm kernel where the row width allows.
fax_status fax_layernorm_bwd(fax_ctx* ctx, int prec, int rows, int d, const void* da, const void* x,
                             const float* mu, const float* rstd, const void* gamma, const void* add,
                             void* dx, float* dgamma, float* dbeta, bool accumulate, float* partial,
                             size_t partial_floats, float* sum_add = nullptr, float* sum_out = nullptr);
size_t fax_layernorm_bwd_partial_floats(int rows, int d);

// out[c] (+)= sum_r in[r, c]
fax_status fax_colsum(fax_ctx* ctx, int prec, int rows, int cols, const void* in, int64_t ld, float* out,
                      bool accumulate, float* partial, size_t partial_floats);
size_t fax_colsum_partial_floats(int rows, int cols);

fax_status fax_attention_fwd(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                             void* o, float* lse);
fax_status fax_attention_bwd(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                             const void* o, const float* lse, const void* d_o, void* dqkv,
                             void* scratch, size_t scratch_bytes);
size_t fax_attention_bwd_scratch_bytes(int prec, int B, int T, int H, int hd);

// step >= 1, both betas in [0, 1), lr and eps finite and eps >= 0.  Checked before anything of a step is
// enqueued, on the direct path and on graph replay alike.
static inline fax_status fax_adamw_check_hparams(const fax_adamw_hparams* hp) {
  if (!hp || hp->step < 1) return FAX_ERR_INVALID_ARG;
  if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f)) return FAX_ERR_INVALID_ARG;
  if (!(hp->lr == hp->lr) || !(hp->eps >= 0.f) || hp->lr - hp->lr != 0.f || hp->eps - hp->eps != 0.f) return FAX_ERR_INVALID_ARG;
  return FAX_OK;
}
fax_status fax_adamw_launch(fax_ctx* ctx, const fax_adamw_tensor* tensors, int n, const fax_adamw_hparams* hp);
// Enqueue AdamW on the context's optimizer stream, ordered after everything enqueued on the main
// stream so far; fax_adamw_join makes the main stream wait for all of it.
fax_status fax_adamw_async(fax_ctx* ctx, const fax_adamw_tensor* tensors, int n, const fax_adamw_hparams* hp);
fax_status fax_adamw_join(fax_ctx* ctx);
bool fax_adamw_is_kernel(const void* func);                        // one of the AdamW kernels?
void fax_adamw_scalars(const fax_adamw_hparams* hp, void* out32);  // the kernels' by-value scalar argument
struct FaxAdamHook { const fax_adamw_tensor* t; const fax_adamw_hparams* hp; };   // t: 12 tensors in parameter order

fax_status fax_block_validate(const fax_block_cfg* cfg);

fax_status fax_attention_fwd_simt(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                                  void* o, float* lse);
fax_status fax_attention_bwd_simt(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                                  const void* o, const float* lse, const void* d_o, void* dqkv, float* Dv);
fax_status fax_embed_fwd(fax_ctx* ctx, int prec, int B, int T, int d, int vocab, const int32_t* ids,
                         const void* wte, const void* wpe, void* x0);
fax_status fax_embed_bwd(fax_ctx* ctx, int prec, int B, int T, int max_seq, int d, int vocab,
                         const int32_t* ids, const void* dx0, float* dwte, float* dwpe, bool accumulate_wpe);
fax_status fax_xent(fax_ctx* ctx, int prec, int rows, int vocab, void* logits, int64_t ld,
                    const int32_t* targets, float inv_n, float* row_loss);
fax_status fax_loss_mean(fax_ctx* ctx, int n, const float* row_loss, float* loss);

bool fax_attention_tc_supported(int B, int T, int H, int hd);
fax_status fax_attention_fwd_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, void* o, float* lse);
// g = GELU_tanh(h) element-wise with the function the FC1 epilogue uses (n elements of the precision's type)
fax_status fax_gelu_fwd(fax_ctx* ctx, int prec, size_t n, const void* h, void* g);
bool fax_attention_fwd2_supported(int B, int T, int H, int hd);
fax_status fax_attention_fwd2_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, void* o, float* lse);
size_t fax_attention_bwd_tc_scratch_bytes(int B, int T, int H, int hd);
// backward with sixteen row warps and half-tile hand-offs (the main kernel only; see its definition)
bool fax_attention_bwd4_supported(int B, int T, int H, int hd);
fax_status fax_attention_bwd4_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const float* lse,
                                 const void* d_o, void* dqkv, const float* Dv, float* dq_acc);
bool fax_attention_bwd3_supported(int B, int T, int H, int hd);
fax_status fax_attention_bwd3_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const float* lse,
                                 const void* d_o, void* dqkv, const float* Dv, float* dq_acc);
fax_status fax_attention_bwd_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const void* o,
                                const float* lse, const void* d_o, void* dqkv, void* scratch, size_t scratch_bytes);
