// Causal multi-head attention, forward and backward, as plain SIMT float32
// arithmetic (steps F3 / B5).  One warp per query row (forward, dq) or per key
// row (dk, dv).  This is the float32 validation path and the shape-agnostic
// fallback; the tensor-core kernels replace it for bf16.
#include "common.cuh"

namespace {

constexpr int WARPS = 4;
constexpr int MAX_HD = 128;

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ qs, const T* __restrict__ row, int hd) {
  float s = 0.f;
  for (int c = 0; c < hd; ++c) s = fmaf(qs[c], to_f32(row[c]), s);
  return s;
}

// grid.x = ceil(T / WARPS), grid.y = B*H
template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
attn_fwd_simt_kernel(int Bn, int Tn, int H, int hd, const T* __restrict__ qkv, T* __restrict__ o,
                     float* __restrict__ lse) {
  __shared__ float qs[WARPS][MAX_HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * WARPS + warp;
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  const int d = H * hd;
  const int64_t ld = 3 * (int64_t)d;
  if (i >= Tn) return;
  const T* base = qkv + (int64_t)b * Tn * ld + h * hd;
  const float scale = rsqrtf((float)hd);
  for (int c = lane; c < hd; c += 32) qs[warp][c] = to_f32(base[(int64_t)i * ld + c]);
  __syncwarp();
  float m = -INFINITY, l = 0.f;
  float acc[MAX_HD / 32];
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    int j = j0 + lane;
    float s = -INFINITY;
    if (j <= i) s = dot_row<T>(qs[warp], base + (int64_t)j * ld + d, hd) * scale;
    float mn = fmaxf(m, warp_max(s));
    float p = (j <= i) ? expf(s - mn) : 0.f;
    float corr = expf(m - mn);
    l = l * corr + warp_sum(p);
    m = mn;
#pragma unroll
    for (int c = 0; c < MAX_HD / 32; ++c) acc[c] *= corr;
    int lim = min(32, i - j0 + 1);
    for (int jj = 0; jj < lim; ++jj) {
      float pj = __shfl_sync(0xffffffffu, p, jj);
      const T* vrow = base + (int64_t)(j0 + jj) * ld + 2 * d;
#pragma unroll
      for (int c = 0; c < MAX_HD / 32; ++c)
        if (lane + 32 * c < hd) acc[c] = fmaf(pj, to_f32(vrow[lane + 32 * c]), acc[c]);
    }
  }
  T* orow = o + ((int64_t)b * Tn + i) * d + h * hd;
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c)
    if (lane + 32 * c < hd) orow[lane + 32 * c] = from_f32<T>(acc[c] / l);
  if (lane == 0) lse[((int64_t)b * H + h) * Tn + i] = m + logf(l);
}

// D[b,h,i] = sum_c do[i,c] * o[i,c]
template <typename T>
__global__ void attn_rowdot_kernel(int Bn, int Tn, int H, int hd, const T* __restrict__ d_o,
                                   const T* __restrict__ o, float* __restrict__ Dv) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * WARPS + warp;
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  if (i >= Tn) return;
  const int d = H * hd;
  const int64_t off = ((int64_t)b * Tn + i) * d + h * hd;
  float s = 0.f;
  for (int c = lane; c < hd; c += 32) s += to_f32(d_o[off + c]) * to_f32(o[off + c]);
  s = warp_sum(s);
  if (lane == 0) Dv[((int64_t)b * H + h) * Tn + i] = s;
}

// dq: one warp per query row
template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
attn_bwd_dq_simt_kernel(int Bn, int Tn, int H, int hd, const T* __restrict__ qkv,
                        const T* __restrict__ d_o, const float* __restrict__ lse,
                        const float* __restrict__ Dv, T* __restrict__ dqkv) {
  __shared__ float qs[WARPS][MAX_HD];
  __shared__ float dos[WARPS][MAX_HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * WARPS + warp;
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  const int d = H * hd;
  const int64_t ld = 3 * (int64_t)d;
  if (i >= Tn) return;
  const T* base = qkv + (int64_t)b * Tn * ld + h * hd;
  const float scale = rsqrtf((float)hd);
  for (int c = lane; c < hd; c += 32) {
    qs[warp][c] = to_f32(base[(int64_t)i * ld + c]);
    dos[warp][c] = to_f32(d_o[((int64_t)b * Tn + i) * d + h * hd + c]);
  }
  __syncwarp();
  const float L = lse[((int64_t)b * H + h) * Tn + i];
  const float Di = Dv[((int64_t)b * H + h) * Tn + i];
  float acc[MAX_HD / 32];
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    int j = j0 + lane;
    float ds = 0.f;
    if (j <= i) {
      float s = dot_row<T>(qs[warp], base + (int64_t)j * ld + d, hd) * scale;
      float p = expf(s - L);
      float dp = dot_row<T>(dos[warp], base + (int64_t)j * ld + 2 * d, hd);
      ds = p * (dp - Di);
    }
    int lim = min(32, i - j0 + 1);
    for (int jj = 0; jj < lim; ++jj) {
      float dsj = __shfl_sync(0xffffffffu, ds, jj);
      const T* krow = base + (int64_t)(j0 + jj) * ld + d;
#pragma unroll
      for (int c = 0; c < MAX_HD / 32; ++c)
        if (lane + 32 * c < hd) acc[c] = fmaf(dsj, to_f32(krow[lane + 32 * c]), acc[c]);
    }
  }
  T* out = dqkv + ((int64_t)b * Tn + i) * ld + h * hd;
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c)
    if (lane + 32 * c < hd) out[lane + 32 * c] = from_f32<T>(acc[c] * scale);
}

// dk, dv: one warp per key row
template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
attn_bwd_dkv_simt_kernel(int Bn, int Tn, int H, int hd, const T* __restrict__ qkv,
                         const T* __restrict__ d_o, const float* __restrict__ lse,
                         const float* __restrict__ Dv, T* __restrict__ dqkv) {
  __shared__ float ks[WARPS][MAX_HD];
  __shared__ float vs[WARPS][MAX_HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * WARPS + warp;
  const int b = blockIdx.y / H, h = blockIdx.y % H;
  const int d = H * hd;
  const int64_t ld = 3 * (int64_t)d;
  if (j >= Tn) return;
  const T* base = qkv + (int64_t)b * Tn * ld + h * hd;
  const T* dobase = d_o + (int64_t)b * Tn * d + h * hd;
  const float scale = rsqrtf((float)hd);
  for (int c = lane; c < hd; c += 32) {
    ks[warp][c] = to_f32(base[(int64_t)j * ld + d + c]);
    vs[warp][c] = to_f32(base[(int64_t)j * ld + 2 * d + c]);
  }
  __syncwarp();
  float acck[MAX_HD / 32], accv[MAX_HD / 32];
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c) { acck[c] = 0.f; accv[c] = 0.f; }
  const float* lrow = lse + ((int64_t)b * H + h) * Tn;
  const float* drow = Dv + ((int64_t)b * H + h) * Tn;
  for (int i0 = j; i0 < Tn; i0 += 32) {
    int i = i0 + lane;
    float p = 0.f, ds = 0.f;
    if (i < Tn) {
      float s = dot_row<T>(ks[warp], base + (int64_t)i * ld, hd) * scale;
      p = expf(s - lrow[i]);
      float dp = dot_row<T>(vs[warp], dobase + (int64_t)i * d, hd);
      ds = p * (dp - drow[i]);
    }
    int lim = min(32, Tn - i0);
    for (int ii = 0; ii < lim; ++ii) {
      float pi = __shfl_sync(0xffffffffu, p, ii);
      float dsi = __shfl_sync(0xffffffffu, ds, ii);
      const T* qrow = base + (int64_t)(i0 + ii) * ld;
      const T* dorow = dobase + (int64_t)(i0 + ii) * d;
#pragma unroll
      for (int c = 0; c < MAX_HD / 32; ++c)
        if (lane + 32 * c < hd) {
          accv[c] = fmaf(pi, to_f32(dorow[lane + 32 * c]), accv[c]);
          acck[c] = fmaf(dsi, to_f32(qrow[lane + 32 * c]), acck[c]);
        }
    }
  }
  T* out = dqkv + ((int64_t)b * Tn + j) * ld + h * hd;
#pragma unroll
  for (int c = 0; c < MAX_HD / 32; ++c)
    if (lane + 32 * c < hd) {
      out[d + lane + 32 * c] = from_f32<T>(acck[c] * scale);
      out[2 * d + lane + 32 * c] = from_f32<T>(accv[c]);
    }
}

template <typename T>
fax_status fwd_t(fax_ctx* ctx, int B, int Tn, int H, int hd, const void* qkv, void* o, float* lse) {
  dim3 grid((Tn + WARPS - 1) / WARPS, B * H);
  attn_fwd_simt_kernel<T><<<grid, WARPS * 32, 0, ctx->stream>>>(B, Tn, H, hd, (const T*)qkv, (T*)o, lse);
  return fax_after_launch(ctx);
}

template <typename T>
fax_status bwd_t(fax_ctx* ctx, int B, int Tn, int H, int hd, const void* qkv, const void* o,
                 const float* lse, const void* d_o, void* dqkv, float* Dv) {
  dim3 grid((Tn + WARPS - 1) / WARPS, B * H);
  attn_rowdot_kernel<T><<<grid, WARPS * 32, 0, ctx->stream>>>(B, Tn, H, hd, (const T*)d_o, (const T*)o, Dv);
  FAX_TRY(fax_after_launch(ctx));
  attn_bwd_dq_simt_kernel<T><<<grid, WARPS * 32, 0, ctx->stream>>>(B, Tn, H, hd, (const T*)qkv,
                                                                  (const T*)d_o, lse, Dv, (T*)dqkv);
  FAX_TRY(fax_after_launch(ctx));
  attn_bwd_dkv_simt_kernel<T><<<grid, WARPS * 32, 0, ctx->stream>>>(B, Tn, H, hd, (const T*)qkv,
                                                                   (const T*)d_o, lse, Dv, (T*)dqkv);
  return fax_after_launch(ctx);
}

}  // namespace

fax_status fax_attention_fwd_simt(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                                  void* o, float* lse) {
  if (hd > MAX_HD || hd <= 0) return FAX_ERR_UNSUPPORTED_SHAPE;
  return prec == FAX_PREC_BF16 ? fwd_t<bf16>(ctx, B, T, H, hd, qkv, o, lse)
                               : fwd_t<float>(ctx, B, T, H, hd, qkv, o, lse);
}

fax_status fax_attention_bwd_simt(fax_ctx* ctx, int prec, int B, int T, int H, int hd, const void* qkv,
                                  const void* o, const float* lse, const void* d_o, void* dqkv,
                                  float* Dv) {
  if (hd > MAX_HD || hd <= 0) return FAX_ERR_UNSUPPORTED_SHAPE;
  return prec == FAX_PREC_BF16 ? bwd_t<bf16>(ctx, B, T, H, hd, qkv, o, lse, d_o, dqkv, Dv)
                               : bwd_t<float>(ctx, B, T, H, hd, qkv, o, lse, d_o, dqkv, Dv);
}
