// Element-wise GELU (tanh form), used when backward recomputes g = GELU(h) instead of reading a saved
// copy: the same functions as the FC1 epilogues (hardware tanh on the bf16 path), so the recomputed
// values are the ones forward produced.
#include "gemm_common.cuh"

namespace {

__global__ void __launch_bounds__(256) gelu_bf16_kernel(size_t n8, const uint4* __restrict__ h, uint4* __restrict__ g) {
  fax_grid_dependency_wait();
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
    uint4 u = h[i], o;
    const __nv_bfloat162* hi = reinterpret_cast<const __nv_bfloat162*>(&u);
    __nv_bfloat162* go = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(hi[e]);
      go[e] = __floats2bfloat162_rn(tc::gelu_fast(f.x), tc::gelu_fast(f.y));
    }
    g[i] = o;
  }
}

__global__ void __launch_bounds__(256) gelu_f32_kernel(size_t n, const float* __restrict__ h, float* __restrict__ g) {
  fax_grid_dependency_wait();
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) g[i] = gelu_tanh_f(h[i]);
}

}  // namespace

fax_status fax_gelu_fwd(fax_ctx* ctx, int prec, size_t n, const void* h, void* g) {
  // accounted with the LayerNorm-forward class (an HBM-bound recomputation pass): read h, write g
  FaxProfScope prof(ctx, KC_LN_FWD, 0.0, 2.0 * (double)n * fax_elem_size(prec));
  const int blocks = 8 * ctx->sm_count;
  if (prec == FAX_PREC_BF16) {
    if (n % 8 || !fax_aligned(h, 16) || !fax_aligned(g, 16)) return FAX_ERR_UNSUPPORTED_SHAPE;
    fax_launch(ctx, gelu_bf16_kernel, dim3(blocks), dim3(256), 0, n / 8, (const uint4*)h, (uint4*)g);
  } else {
    fax_launch(ctx, gelu_f32_kernel, dim3(blocks), dim3(256), 0, n, (const float*)h, (float*)g);
  }
  return fax_after_launch(ctx);
}
