// Plain SIMT GEMM with float accumulation: the arithmetic of the float32
// validation mode, and the shape-agnostic fallback of the bf16 mode for
// problems the tensor-core kernel does not tile (it is never the fast path).
#include "common.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int M, int N, int K, const T* __restrict__ A, int64_t sam, int64_t sak,
                 const T* __restrict__ B, int64_t sbn, int64_t sbk, void* __restrict__ Cv, int64_t ldc,
                 int c_f32, int accumulate, int epi, const T* __restrict__ bias,
                 const T* __restrict__ resid, int64_t ldr, T* __restrict__ aux, int64_t ldaux, float alpha) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  // The thread-to-element map of the tile loads follows whichever index is contiguous.
  const bool a_k_contig = (sak == 1);
  const bool b_k_contig = (sbk == 1);
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int e = tid + i * 256;               // 0..1023
      int mm, kk;
      if (a_k_contig) { kk = e & 15; mm = e >> 4; } else { mm = e & 63; kk = e >> 6; }
      int gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < K) ? to_f32(A[gm * sam + gk * sak]) : 0.f;
      int nn, kb;
      if (b_k_contig) { kb = e & 15; nn = e >> 4; } else { nn = e & 63; kb = e >> 6; }
      int gn = n0 + nn, gkb = k0 + kb;
      Bs[kb][nn] = (gn < N && gkb < K) ? to_f32(B[gn * sbn + gkb * sbk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc[i][j] * alpha;
      if (epi == EPI_BIAS || epi == EPI_BIAS_GELU || epi == EPI_BIAS_RESID) v += to_f32(bias[gn]);
      if (epi == EPI_BIAS_RESID) v += to_f32(resid[gm * ldr + gn]);
      if (epi == EPI_DGELU) v *= gelu_tanh_grad_f(to_f32(aux[gm * ldaux + gn]));
      if (epi == EPI_BIAS_GELU) {
        // GELU acts on the stored (rounded) pre-activation so that backward sees the same h
        T hs = from_f32<T>(v);
        aux[gm * ldaux + gn] = from_f32<T>(gelu_tanh_f(to_f32(hs)));
      }
      if (c_f32) {
        float* C = (float*)Cv;
        C[gm * ldc + gn] = accumulate ? C[gm * ldc + gn] + v : v;
      } else {
        ((T*)Cv)[gm * ldc + gn] = from_f32<T>(v);
      }
    }
  }
}

template <typename T>
fax_status launch(fax_ctx* ctx, const FaxGemm& g) {
  if (g.accumulate && !g.c_f32) return FAX_ERR_INVALID_ARG;
  int64_t sam = g.a_mn_major ? 1 : g.lda, sak = g.a_mn_major ? g.lda : 1;
  int64_t sbn = g.b_mn_major ? 1 : g.ldb, sbk = g.b_mn_major ? g.ldb : 1;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  gemm_simt_kernel<T><<<grid, 256, 0, ctx->stream>>>(
      g.M, g.N, g.K, (const T*)g.A, sam, sak, (const T*)g.B, sbn, sbk, g.C, g.ldc, g.c_f32 ? 1 : 0,
      g.accumulate ? 1 : 0, g.epi, (const T*)g.bias, (const T*)g.resid, g.ldr, (T*)g.aux, g.ldaux, g.alpha);
  return fax_after_launch(ctx);
}

}  // namespace

fax_status fax_gemm_simt(fax_ctx* ctx, int prec, const FaxGemm& g) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return FAX_ERR_INVALID_ARG;
  FaxProfScope prof(ctx, KC_GEMM_SIMT, 2.0 * g.M * g.N * g.K, 0.0);
  return prec == FAX_PREC_BF16 ? launch<bf16>(ctx, g) : launch<float>(ctx, g);
}
