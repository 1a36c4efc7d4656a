// extern "C" wrappers of the single operators (include/fax_ops.h).
#include "common.cuh"
#include "../../include/fax_ops.h"

extern "C" fax_status fax_op_gemm(fax_ctx* ctx, int32_t prec, const fax_gemm_desc* d) {
  if (!ctx || !d || !d->A || !d->B || !d->C) return FAX_ERR_INVALID_ARG;
  if (prec != FAX_PREC_BF16 && prec != FAX_PREC_FP32_VALIDATE) return FAX_ERR_INVALID_ARG;
  if (d->M <= 0 || d->N <= 0 || d->K <= 0) return FAX_ERR_INVALID_ARG;
  if (d->epilogue < FAX_EPI_NONE || d->epilogue > FAX_EPI_DGELU) return FAX_ERR_INVALID_ARG;
  if ((d->epilogue == FAX_EPI_BIAS || d->epilogue == FAX_EPI_BIAS_GELU || d->epilogue == FAX_EPI_BIAS_RESID) && !d->bias)
    return FAX_ERR_INVALID_ARG;
  if (d->epilogue == FAX_EPI_BIAS_RESID && !d->resid) return FAX_ERR_INVALID_ARG;
  if ((d->epilogue == FAX_EPI_BIAS_GELU || d->epilogue == FAX_EPI_DGELU) && !d->aux) return FAX_ERR_INVALID_ARG;
  if (d->accumulate && !d->c_f32) return FAX_ERR_INVALID_ARG;
  FaxGemm g;
  g.M = d->M; g.N = d->N; g.K = d->K;
  g.A = d->A; g.lda = d->lda; g.a_mn_major = d->a_mn_major != 0;
  g.B = d->B; g.ldb = d->ldb; g.b_mn_major = d->b_mn_major != 0;
  g.C = d->C; g.ldc = d->ldc; g.c_f32 = d->c_f32 != 0; g.accumulate = d->accumulate != 0;
  g.epi = d->epilogue; g.bias = d->bias; g.resid = d->resid; g.ldr = d->ldr; g.aux = d->aux; g.ldaux = d->ldaux;
  g.alpha = d->alpha;
  g.adam = nullptr;
  if (d->force_simt) return fax_gemm_simt(ctx, prec, g);
  return fax_gemm(ctx, prec, g);
}

extern "C" fax_status fax_op_layernorm_forward(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d,
                                               const void* x, const void* gamma, const void* beta, float eps,
                                               void* out, float* mu, float* rstd) {
  if (!ctx || !x || !gamma || !beta || !out || !mu || !rstd || rows <= 0 || d <= 0) return FAX_ERR_INVALID_ARG;
  return fax_layernorm_fwd(ctx, prec, rows, d, x, gamma, beta, eps, out, mu, rstd, nullptr);
}

extern "C" fax_status fax_op_layernorm_backward_scratch_bytes(int32_t rows, int32_t d, size_t* bytes) {
  if (!bytes || rows <= 0 || d <= 0) return FAX_ERR_INVALID_ARG;
  *bytes = fax_layernorm_bwd_partial_floats(rows, d) * sizeof(float);
  return FAX_OK;
}

extern "C" fax_status fax_op_layernorm_backward(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d,
                                                const void* da, const void* x, const float* mu,
                                                const float* rstd, const void* gamma, const void* add,
                                                void* dx, float* dgamma, float* dbeta, void* scratch,
                                                size_t scratch_bytes) {
  if (!ctx || !da || !x || !mu || !rstd || !gamma || !dx || !dgamma || !dbeta || !scratch || rows <= 0 || d <= 0)
    return FAX_ERR_INVALID_ARG;
  return fax_layernorm_bwd(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, false,
                           (float*)scratch, scratch_bytes / sizeof(float));
}

static fax_status attn_args(int32_t prec, int32_t B, int32_t T, int32_t H, int32_t hd) {
  if (B <= 0 || T <= 0 || H <= 0 || hd <= 0) return FAX_ERR_INVALID_ARG;
  if (prec != FAX_PREC_BF16 && prec != FAX_PREC_FP32_VALIDATE) return FAX_ERR_INVALID_ARG;
  if (hd > 128) return FAX_ERR_UNSUPPORTED_SHAPE;
  return FAX_OK;
}

extern "C" fax_status fax_op_attention_forward(fax_ctx* ctx, int32_t prec, int32_t B, int32_t T, int32_t H,
                                               int32_t hd, const void* qkv, void* o, float* lse) {
  if (!ctx || !qkv || !o || !lse) return FAX_ERR_INVALID_ARG;
  FAX_TRY(attn_args(prec, B, T, H, hd));
  return fax_attention_fwd(ctx, prec, B, T, H, hd, qkv, o, lse);
}

extern "C" fax_status fax_op_attention_backward_scratch_bytes(int32_t prec, int32_t B, int32_t T, int32_t H,
                                                              int32_t hd, size_t* bytes) {
  if (!bytes) return FAX_ERR_INVALID_ARG;
  FAX_TRY(attn_args(prec, B, T, H, hd));
  *bytes = fax_attention_bwd_scratch_bytes(prec, B, T, H, hd);
  return FAX_OK;
}

extern "C" fax_status fax_op_attention_backward(fax_ctx* ctx, int32_t prec, int32_t B, int32_t T, int32_t H,
                                                int32_t hd, const void* qkv, const void* o, const float* lse,
                                                const void* d_o, void* dqkv, void* scratch, size_t scratch_bytes) {
  if (!ctx || !qkv || !o || !lse || !d_o || !dqkv || !scratch) return FAX_ERR_INVALID_ARG;
  FAX_TRY(attn_args(prec, B, T, H, hd));
  return fax_attention_bwd(ctx, prec, B, T, H, hd, qkv, o, lse, d_o, dqkv, scratch, scratch_bytes);
}
