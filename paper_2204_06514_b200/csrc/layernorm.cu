// LayerNorm forward / backward (block steps F1, F5, B3, B7 and the LM's final
// LayerNorm).  HBM-bound: one block per row keeps the whole row in registers,
// 128-bit loads and stores, warp-shuffle reductions, two-pass mean / variance.
#include "common.cuh"
#include "../../include/fax_ops.h"

namespace {

template <typename T> struct Vec;              // 16-byte vector of T
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<bf16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load_vec(const T* p, float (&f)[Vec<T>::N]);
template <>
__device__ __forceinline__ void load_vec<float>(const float* p, float (&f)[4]) {
  float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <>
__device__ __forceinline__ void load_vec<bf16>(const bf16* p, float (&f)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
template <typename T>
__device__ __forceinline__ void store_vec(T* p, const float (&f)[Vec<T>::N]);
template <>
__device__ __forceinline__ void store_vec<float>(float* p, const float (&f)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
template <>
__device__ __forceinline__ void store_vec<bf16>(bf16* p, const float (&f)[8]) {
  uint4 v;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  *reinterpret_cast<uint4*>(p) = v;
}

// Sum over the block; every thread gets the result.  red: >= 32 floats of smem.
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
  return warp_sum(t);
}
__device__ __forceinline__ float2 block_sum2(float a, float b, float2* red) {
  a = warp_sum(a); b = warp_sum(b);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = make_float2(a, b);
  __syncthreads();
  float2 t = (lane < nw) ? red[lane] : make_float2(0.f, 0.f);
  return make_float2(warp_sum(t.x), warp_sum(t.y));
}

template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_fwd_kernel(int rows, int d, const T* __restrict__ x, const T* __restrict__ gamma,
                     const T* __restrict__ beta, float eps, T* __restrict__ out,
                     float* __restrict__ mu_out, float* __restrict__ rstd_out, T* __restrict__ x_copy) {
  constexpr int VN = Vec<T>::N;
  __shared__ float red[32];
  const int nvec = d / VN;
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    const T* xr = x + (size_t)row * d;
    float v[VPT][VN];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      int vi = threadIdx.x + i * blockDim.x;
      if (vi < nvec) {
        load_vec<T>(xr + vi * VN, v[i]);
#pragma unroll
        for (int j = 0; j < VN; ++j) s += v[i][j];
      }
    }
    float mu = block_sum(s, red) / (float)d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      int vi = threadIdx.x + i * blockDim.x;
      if (vi < nvec) {
#pragma unroll
        for (int j = 0; j < VN; ++j) { float t = v[i][j] - mu; q += t * t; }
      }
    }
    float rstd = rsqrtf(block_sum(q, red) / (float)d + eps);
    if (threadIdx.x == 0) { mu_out[row] = mu; rstd_out[row] = rstd; }
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      int vi = threadIdx.x + i * blockDim.x;
      if (vi < nvec) {
        float g[VN], b[VN], o[VN];
        load_vec<T>(gamma + vi * VN, g);
        load_vec<T>(beta + vi * VN, b);
#pragma unroll
        for (int j = 0; j < VN; ++j) o[j] = (v[i][j] - mu) * rstd * g[j] + b[j];
        store_vec<T>(out + (size_t)row * d + vi * VN, o);
        if (x_copy) store_vec<T>(x_copy + (size_t)row * d + vi * VN, v[i]);
      }
    }
  }
}

// Each block walks rows blockIdx.x, +gridDim.x, ...; column sums of da and
// da*xhat stay in registers and are written once per block to `partial`
// ([gridDim.x][2][d]); a second kernel folds the slabs.
template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_bwd_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                     const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                     const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx,
                     float* __restrict__ partial) {
  constexpr int VN = Vec<T>::N;
  __shared__ float2 red[32];
  const int nvec = d / VN;
  float g[VPT][VN], accg[VPT][VN], accb[VPT][VN];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    int vi = threadIdx.x + i * blockDim.x;
#pragma unroll
    for (int j = 0; j < VN; ++j) { accg[i][j] = 0.f; accb[i][j] = 0.f; g[i][j] = 0.f; }
    if (vi < nvec) load_vec<T>(gamma + vi * VN, g[i]);
  }
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    const float mu = mu_in[row], rstd = rstd_in[row];
    float u[VPT][VN], xh[VPT][VN];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      int vi = threadIdx.x + i * blockDim.x;
      if (vi < nvec) {
        float dv[VN], xv[VN];
        load_vec<T>(da + (size_t)row * d + vi * VN, dv);
        load_vec<T>(x + (size_t)row * d + vi * VN, xv);
#pragma unroll
        for (int j = 0; j < VN; ++j) {
          xh[i][j] = (xv[j] - mu) * rstd;
          u[i][j] = dv[j] * g[i][j];
          accg[i][j] += dv[j] * xh[i][j];
          accb[i][j] += dv[j];
          s1 += u[i][j];
          s2 += u[i][j] * xh[i][j];
        }
      }
    }
    float2 t = block_sum2(s1, s2, red);
    const float c1 = t.x / (float)d, c2 = t.y / (float)d;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      int vi = threadIdx.x + i * blockDim.x;
      if (vi < nvec) {
        float o[VN];
#pragma unroll
        for (int j = 0; j < VN; ++j) o[j] = rstd * (u[i][j] - c1 - xh[i][j] * c2);
        if (add) {
          float av[VN];
          load_vec<T>(add + (size_t)row * d + vi * VN, av);
#pragma unroll
          for (int j = 0; j < VN; ++j) o[j] += av[j];
        }
        store_vec<T>(dx + (size_t)row * d + vi * VN, o);
      }
    }
  }
  float* pg = partial + (size_t)blockIdx.x * 2 * d;
  float* pb = pg + d;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    int vi = threadIdx.x + i * blockDim.x;
    if (vi < nvec) {
#pragma unroll
      for (int j = 0; j < VN; ++j) { pg[vi * VN + j] = accg[i][j]; pb[vi * VN + j] = accb[i][j]; }
    }
  }
}

// out[k][c] (+)= sum_s partial[s][k][c], k in {0: dgamma, 1: dbeta}
__global__ void layernorm_bwd_fold_kernel(int slabs, int d, const float* __restrict__ partial,
                                          float* __restrict__ dgamma, float* __restrict__ dbeta,
                                          int accumulate) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= 2 * d) return;
  float s = 0.f;
  for (int i = 0; i < slabs; ++i) s += partial[(size_t)i * 2 * d + c];
  float* dst = (c < d) ? (dgamma + c) : (dbeta + (c - d));
  *dst = accumulate ? (*dst + s) : s;
}

// partial[s][c] = sum over the rows of slab s of in[r][c]
template <typename T>
__global__ void colsum_partial_kernel(int rows, int cols, const T* __restrict__ in, int64_t ld,
                                      float* __restrict__ partial) {
  constexpr int VN = Vec<T>::N;
  int vc = blockIdx.x * blockDim.x + threadIdx.x;   // vector column
  if (vc * VN >= cols) return;
  float acc[VN];
#pragma unroll
  for (int j = 0; j < VN; ++j) acc[j] = 0.f;
  for (int r = blockIdx.y; r < rows; r += gridDim.y) {
    float v[VN];
    load_vec<T>(in + (size_t)r * ld + vc * VN, v);
#pragma unroll
    for (int j = 0; j < VN; ++j) acc[j] += v[j];
  }
#pragma unroll
  for (int j = 0; j < VN; ++j) partial[(size_t)blockIdx.y * cols + vc * VN + j] = acc[j];
}
__global__ void colsum_fold_kernel(int slabs, int cols, const float* __restrict__ partial,
                                   float* __restrict__ out, int accumulate) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  float s = 0.f;
  for (int i = 0; i < slabs; ++i) s += partial[(size_t)i * cols + c];
  out[c] = accumulate ? out[c] + s : s;
}

int pick_vpt(int nvec, int max_threads, int* threads) {
  static const int opts[] = {1, 2, 3, 4, 6, 8, 12, 16};
  for (int v : opts) {
    int t = (nvec + v - 1) / v;
    if (t <= max_threads) { *threads = (t + 31) / 32 * 32; return v; }
  }
  *threads = 0;
  return 0;
}

int ln_bwd_slabs(fax_ctx* ctx, int rows) { return rows < ctx->sm_count ? rows : ctx->sm_count; }

template <typename T>
fax_status ln_fwd_t(fax_ctx* ctx, int rows, int d, const void* x, const void* gamma, const void* beta,
                    float eps, void* out, float* mu, float* rstd, void* x_copy) {
  int threads = 0;
  int vpt = pick_vpt(d / Vec<T>::N, 512, &threads);
  if (!vpt) return FAX_ERR_UNSUPPORTED_SHAPE;
  int grid = rows;
#define LN_FWD(V)                                                                                    \
  case V:                                                                                            \
    layernorm_fwd_kernel<T, V><<<grid, threads, 0, ctx->stream>>>(                                   \
        rows, d, (const T*)x, (const T*)gamma, (const T*)beta, eps, (T*)out, mu, rstd, (T*)x_copy);   \
    break;
  switch (vpt) { LN_FWD(1) LN_FWD(2) LN_FWD(3) LN_FWD(4) LN_FWD(6) LN_FWD(8) LN_FWD(12) LN_FWD(16) }
#undef LN_FWD
  return fax_after_launch(ctx);
}

template <typename T>
fax_status ln_bwd_t(fax_ctx* ctx, int rows, int d, const void* da, const void* x, const float* mu,
                    const float* rstd, const void* gamma, const void* add, void* dx, float* dgamma,
                    float* dbeta, bool accumulate, float* partial) {
  int threads = 0;
  int vpt = pick_vpt(d / Vec<T>::N, 512, &threads);
  if (!vpt || vpt > 8) return FAX_ERR_UNSUPPORTED_SHAPE;
  int slabs = ln_bwd_slabs(ctx, rows);
#define LN_BWD(V)                                                                                   \
  case V:                                                                                           \
    layernorm_bwd_kernel<T, V><<<slabs, threads, 0, ctx->stream>>>(                                 \
        rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx,       \
        partial);                                                                                   \
    break;
  switch (vpt) { LN_BWD(1) LN_BWD(2) LN_BWD(3) LN_BWD(4) LN_BWD(6) LN_BWD(8) }
#undef LN_BWD
  FAX_TRY(fax_after_launch(ctx));
  layernorm_bwd_fold_kernel<<<(2 * d + 255) / 256, 256, 0, ctx->stream>>>(slabs, d, partial, dgamma, dbeta,
                                                                          accumulate ? 1 : 0);
  return fax_after_launch(ctx);
}

}  // namespace

size_t fax_layernorm_bwd_partial_floats(int rows, int d) {
  int slabs = rows < 256 ? rows : 256;     // upper bound on the SM count used for slabs
  return (size_t)2 * slabs * d;
}

fax_status fax_layernorm_fwd(fax_ctx* ctx, int prec, int rows, int d, const void* x, const void* gamma,
                             const void* beta, float eps, void* out, float* mu, float* rstd, void* x_copy) {
  // read x, write out (and the optional copy of x)
  FaxProfScope prof(ctx, KC_LN_FWD, 0.0, (double)rows * d * fax_elem_size(prec) * (x_copy ? 3 : 2));
  if (prec == FAX_PREC_BF16) {
    if (d % 8) return FAX_ERR_UNSUPPORTED_SHAPE;
    return ln_fwd_t<bf16>(ctx, rows, d, x, gamma, beta, eps, out, mu, rstd, x_copy);
  }
  if (d % 4) return FAX_ERR_UNSUPPORTED_SHAPE;
  return ln_fwd_t<float>(ctx, rows, d, x, gamma, beta, eps, out, mu, rstd, x_copy);
}

fax_status fax_layernorm_bwd(fax_ctx* ctx, int prec, int rows, int d, const void* da, const void* x,
                             const float* mu, const float* rstd, const void* gamma, const void* add,
                             void* dx, float* dgamma, float* dbeta, bool accumulate, float* partial,
                             size_t partial_floats) {
  if (ctx->sm_count > 256) return FAX_ERR_ARCH;
  if (partial_floats < (size_t)2 * ln_bwd_slabs(ctx, rows) * d) return FAX_ERR_WORKSPACE_TOO_SMALL;
  // read da, x (and add), write dx
  FaxProfScope prof(ctx, KC_LN_BWD, 0.0, (double)rows * d * fax_elem_size(prec) * (add ? 4 : 3));
  if (prec == FAX_PREC_BF16) {
    if (d % 8) return FAX_ERR_UNSUPPORTED_SHAPE;
    return ln_bwd_t<bf16>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, accumulate, partial);
  }
  if (d % 4) return FAX_ERR_UNSUPPORTED_SHAPE;
  return ln_bwd_t<float>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, accumulate, partial);
}

size_t fax_colsum_partial_floats(int rows, int cols) {
  int slabs = rows < 256 ? rows : 256;
  return (size_t)slabs * cols;
}

fax_status fax_colsum(fax_ctx* ctx, int prec, int rows, int cols, const void* in, int64_t ld, float* out,
                      bool accumulate, float* partial, size_t partial_floats) {
  const int vn = prec == FAX_PREC_BF16 ? 8 : 4;
  if (cols % vn || ld % vn) return FAX_ERR_UNSUPPORTED_SHAPE;
  int vcols = cols / vn;
  int threads = 128;
  int gx = (vcols + threads - 1) / threads;
  // enough row slabs to fill the machine, at most 256
  int slabs = (2 * ctx->sm_count + gx - 1) / gx;
  if (slabs > rows) slabs = rows;
  if (slabs > 256) slabs = 256;
  if (slabs < 1) slabs = 1;
  if (partial_floats < (size_t)slabs * cols) return FAX_ERR_WORKSPACE_TOO_SMALL;
  FaxProfScope prof(ctx, KC_COLSUM, 0.0, (double)rows * cols * fax_elem_size(prec));
  dim3 grid(gx, slabs);
  if (prec == FAX_PREC_BF16)
    colsum_partial_kernel<bf16><<<grid, threads, 0, ctx->stream>>>(rows, cols, (const bf16*)in, ld, partial);
  else
    colsum_partial_kernel<float><<<grid, threads, 0, ctx->stream>>>(rows, cols, (const float*)in, ld, partial);
  FAX_TRY(fax_after_launch(ctx));
  colsum_fold_kernel<<<(cols + 255) / 256, 256, 0, ctx->stream>>>(slabs, cols, partial, out, accumulate ? 1 : 0);
  return fax_after_launch(ctx);
}

// ---------------------------------------------------------------------------
// LayerNorm backward for callers that have no device memory to hand over as
// scratch and may not allocate any: the column-sum partials live in a fixed
// array that is part of the library image (8 MiB on every GPU that loads it,
// until the process exits).
// ---------------------------------------------------------------------------
static __device__ __align__(256) float g_ln_static_partial[FAX_LN_STATIC_SCRATCH_FLOATS];

// Device address of the array above, per device ordinal.  In host code the
// array's name is only a handle for the runtime, not a device pointer; the
// address a kernel can use comes from cudaGetSymbolAddress, asked once per
// device with that device current.
static float* g_ln_static_ptr[64] = {nullptr};

extern "C" fax_status fax_op_layernorm_backward_static(fax_ctx* ctx, int32_t prec, int32_t rows, int32_t d,
                                                       const void* da, const void* x, const float* mu,
                                                       const float* rstd, const void* gamma, const void* add,
                                                       void* dx, float* dgamma, float* dbeta) {
  if (!ctx || !da || !x || !mu || !rstd || !gamma || !dx || !dgamma || !dbeta || rows <= 0 || d <= 0)
    return FAX_ERR_INVALID_ARG;
  if (prec != FAX_PREC_BF16 && prec != FAX_PREC_FP32_VALIDATE) return FAX_ERR_INVALID_ARG;
  if (ctx->device < 0 || ctx->device >= 64 || ctx->sm_count > 256) return FAX_ERR_ARCH;
  const size_t need = (size_t)2 * ln_bwd_slabs(ctx, rows) * d;
  if (need > (size_t)FAX_LN_STATIC_SCRATCH_FLOATS) return FAX_ERR_WORKSPACE_TOO_SMALL;   // beyond the fixed array
  if (!g_ln_static_ptr[ctx->device]) {
    // one-time set-up on this device (no allocation: the array already exists in the loaded module)
    FAX_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    float* ptr = nullptr;
    FAX_CUDA_TRY(ctx, cudaGetSymbolAddress((void**)&ptr, g_ln_static_partial));
    if (!ptr) return FAX_ERR_CUDA;
    g_ln_static_ptr[ctx->device] = ptr;
  }
  // Every slab writes its whole slice of the partials before the fold kernel reads it, so
  // nothing in the shared array has to start at zero and stale contents are harmless.
  return fax_layernorm_bwd(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, false,
                           g_ln_static_ptr[ctx->device], FAX_LN_STATIC_SCRATCH_FLOATS);
}
