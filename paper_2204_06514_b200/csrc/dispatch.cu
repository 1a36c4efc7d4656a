// Operator dispatch between the tensor-core kernels and the SIMT kernels.
#include "common.cuh"

// bf16 problems run on the tensor cores or not at all, unless the caller has allowed the SIMT
// kernel for them: a shape the tensor-core kernels reject would otherwise run one to two orders of
// magnitude slower with nothing telling the caller.
fax_status fax_gemm(fax_ctx* ctx, int prec, const FaxGemm& g, bool allow_simt, int* kernel_class) {
  if (prec == FAX_PREC_BF16 && fax_gemm_tc_supported(g)) {
    if (kernel_class) *kernel_class = KC_GEMM_TC;
    return fax_gemm_tc(ctx, g);
  }
  if (g.adam) return FAX_ERR_INVALID_ARG;               // callers ask fax_gemm_can_fuse_adam first
  if (prec == FAX_PREC_BF16 && !allow_simt) return FAX_ERR_UNSUPPORTED_SHAPE;
  if (kernel_class) *kernel_class = KC_GEMM_SIMT;
  return fax_gemm_simt(ctx, prec, g);
}

size_t fax_attention_bwd_scratch_bytes(int prec, int B, int T, int H, int hd) {
  size_t simt = (size_t)B * H * T * sizeof(float);      // D = rowsum(dO * O)
  if (prec == FAX_PREC_BF16 && fax_attention_tc_supported(B, T, H, hd)) {
    size_t t = fax_attention_bwd_tc_scratch_bytes(B, T, H, hd);
    return t > simt ? t : simt;
  }
  return simt;
}

fax_status fax_attention_fwd(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                             void* o, float* lse) {
  // causal half of QK^T and PV
  FaxProfScope prof(ctx, KC_ATTN_FWD, 2.0 * B * H * (double)T * T * hd, 0.0);
  if (prec == FAX_PREC_BF16 && fax_attention_tc_supported(B, T, H, hd))
    return fax_attention_fwd_tc(ctx, B, T, H, hd, qkv, o, lse);
  return fax_attention_fwd_simt(ctx, prec, B, T, H, hd, qkv, o, lse);
}

fax_status fax_attention_bwd(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                             const void* o, const float* lse, const void* d_o, void* dqkv,
                             void* scratch, size_t scratch_bytes) {
  if (scratch_bytes < (size_t)B * H * T * sizeof(float)) return FAX_ERR_WORKSPACE_TOO_SMALL;
  // causal half of dV, dP, dQ, dK (the recomputed QK^T is not counted)
  FaxProfScope prof(ctx, KC_ATTN_BWD, 4.0 * B * H * (double)T * T * hd, 0.0);
  if (prec == FAX_PREC_BF16 && fax_attention_tc_supported(B, T, H, hd))
    return fax_attention_bwd_tc(ctx, B, T, H, hd, qkv, o, lse, d_o, dqkv, scratch, scratch_bytes);
  return fax_attention_bwd_simt(ctx, prec, B, T, H, hd, qkv, o, lse, d_o, dqkv, (float*)scratch);
}
