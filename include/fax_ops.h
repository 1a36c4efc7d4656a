/*
 * fax_ops.h -- operator-level entry points of the same library: the single
 * kernels the block and LM step are made of, exposed so that each can be
 * checked against the oracle and timed against its roofline on its own.
 * All conventions of fax.h hold (device pointers, caller-owned buffers,
 * asynchronous on the context's stream, fax_status results).  "T" is bf16 for
 * FAX_PREC_BF16 and float for FAX_PREC_FP32_VALIDATE.
 */
#ifndef FAX_OPS_H_
#define FAX_OPS_H_

#include "fax.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Epilogues of the GEMM (the fused tails the block's linear layers need). */
enum {
  FAX_EPI_NONE = 0,        /* C = alpha * A B                                     */
  FAX_EPI_BIAS = 1,        /* C = alpha * A B + bias[n]                           */
  FAX_EPI_BIAS_GELU = 2,   /* C = alpha * A B + bias (stored), aux = GELU_tanh(C) */
  FAX_EPI_BIAS_RESID = 3,  /* C = alpha * A B + bias + resid                      */
  FAX_EPI_DGELU = 4        /* C = (alpha * A B) * GELU_tanh'(aux)                 */
};

/* C[M,N] = op(A) op(B) with float accumulation -- the QKV, attention-output,
 * MLP and output-head contractions of the step and their backward forms
 * (Sec. 3.2: the large matrix multiplications of the transformer).
 * A is [M,K] row-major (a_mn_major = 0) or [K,M] row-major (a_mn_major = 1);
 * B is [N,K] row-major (b_mn_major = 0) or [K,N] row-major (b_mn_major = 1);
 * lda / ldb / ldc / ldr / ldaux are row strides in elements.  C is T, or
 * float when c_f32 != 0; accumulate != 0 adds into a float C.  bias [N],
 * resid [M,N] and aux [M,N] are T.  In FAX_PREC_BF16 the problem runs on the
 * tensor-core kernels (M a multiple of 128, N and K of 64, 16-byte aligned rows)
 * and any other shape is refused with FAX_ERR_UNSUPPORTED_SHAPE: it never lands
 * on the far slower float-FMA kernel unasked.  force_simt != 0 selects that
 * kernel, for any shape and in either precision (FAX_PREC_FP32_VALIDATE always
 * uses it). */
typedef struct {
  int32_t M, N, K;
  const void* A; int64_t lda; int32_t a_mn_major;
  const void* B; int64_t ldb; int32_t b_mn_major;
  void* C; int64_t ldc; int32_t c_f32; int32_t accumulate;
  int32_t epilogue;
  const void* bias;
  const void* resid; int64_t ldr;
  void* aux; int64_t ldaux;
  float alpha;
  int32_t force_simt;
} fax_gemm_desc;

fax_status fax_op_gemm(fax_ctx* ctx, int32_t prec, const fax_gemm_desc* desc);

/* Row-wise LayerNorm over d (biased variance, eps inside the square root):
 * out = gamma * (x - mu) * rstd + beta; mu, rstd [rows] float are saved. */
fax_status fax_op_layernorm_forward(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d, const void* x,
                                    const void* gamma, const void* beta, float eps, void* out,
                                    float* mu, float* rstd);

/* Reverse of the above: dx = (add ? add : 0) + dLN(da); dgamma, dbeta [d]
 * float are overwritten.  scratch: fax_op_layernorm_backward_scratch_bytes. */
fax_status fax_op_layernorm_backward_scratch_bytes(int32_t rows, int32_t d, size_t* bytes);
fax_status fax_op_layernorm_backward(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d, const void* da,
                                     const void* x, const float* mu, const float* rstd, const void* gamma,
                                     const void* add, void* dx, float* dgamma, float* dbeta,
                                     void* scratch, size_t scratch_bytes);

/* LayerNorm backward without caller scratch and without any allocation.  (The
 * paper has no counterpart of this call; it exists for deployment reasons.)
 * Some hosts of this library cannot give it scratch memory or let it call
 * cudaMalloc: a serving or training process whose own pool already owns all
 * device memory, a plug-in that runs under a fixed memory budget, or a
 * latency-critical loop that cannot afford the device-wide synchronisation an
 * allocation implies.  For them the column-sum partials of dgamma / dbeta live
 * in a fixed array inside the library image: FAX_LN_STATIC_SCRATCH_FLOATS
 * floats (8 MiB), resident on every GPU that loads the library until the
 * process exits.  The call computes exactly what fax_op_layernorm_backward
 * computes (same kernels) and calls no cudaMalloc, cudaFree or allocating
 * library routine.
 *  - Limit: d <= FAX_LN_STATIC_MAX_D (4096) at any row count (the array holds
 *    the partial sums of up to 256 row slabs of that width); a wider row makes
 *    the call do nothing and return FAX_ERR_WORKSPACE_TOO_SMALL.
 *  - The first call on each device looks the array's device address up (one
 *    cudaGetSymbolAddress with that device current).  Make that first call
 *    before starting any stream capture on the device.
 *  - All calls on a device share the one array, and it keeps whatever the last
 *    call left.  Nothing in it needs clearing (every slot is written before it
 *    is read), but two calls whose kernels overlap on the GPU (different
 *    streams or contexts) race on it: serialise them. */
#define FAX_LN_STATIC_MAX_D 4096
#define FAX_LN_STATIC_SCRATCH_FLOATS (2 * 256 * FAX_LN_STATIC_MAX_D)
fax_status fax_op_layernorm_backward_static(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d, const void* da,
                                            const void* x, const float* mu, const float* rstd,
                                            const void* gamma, const void* add, void* dx, float* dgamma,
                                            float* dbeta);

/* Causal multi-head attention (Sec. 3.2: multi-headed attention blocks) on a
 * fused qkv [batch*seq, 3*n_heads*head_dim] T buffer (layout in fax.h):
 * o [batch*seq, n_heads*head_dim] T, lse [batch, n_heads, seq] float
 * (natural-log sum of exponentials of the scaled, masked scores). */
fax_status fax_op_attention_forward(fax_ctx* ctx, int32_t prec, int32_t batch, int32_t seq, int32_t n_heads,
                                    int32_t head_dim, const void* qkv, void* o, float* lse);

/* Reverse: given d_o [batch*seq, d] T writes dqkv [batch*seq, 3d] T. */
fax_status fax_op_attention_backward_scratch_bytes(int32_t prec, int32_t batch, int32_t seq,
                                                   int32_t n_heads, int32_t head_dim, size_t* bytes);
fax_status fax_op_attention_backward(fax_ctx* ctx, int32_t prec, int32_t batch, int32_t seq,
                                     int32_t n_heads, int32_t head_dim, const void* qkv, const void* o,
                                     const float* lse, const void* d_o, void* dqkv, void* scratch,
                                     size_t scratch_bytes);

#ifdef __cplusplus
}
#endif
#endif /* FAX_OPS_H_ */
