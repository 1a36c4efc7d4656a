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

// ---- raw 16-byte vectors kept packed in registers ---------------------------
template <typename T> __device__ __forceinline__ void unpack(const uint4& u, float (&f)[Vec<T>::N]);
template <> __device__ __forceinline__ void unpack<float>(const uint4& u, float (&f)[4]) {
  f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
template <> __device__ __forceinline__ void unpack<bf16>(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}

// Forward, one warp per row (rows of up to 32*VPT vectors): the row stays packed in
// registers, reductions are warp shuffles only, no block barrier.
template <typename T, int VPT>
__global__ void __launch_bounds__(128)
layernorm_fwd_warp_kernel(int rows, int d, const T* __restrict__ x, const T* __restrict__ gamma,
                          const T* __restrict__ beta, float eps, T* __restrict__ out,
                          float* __restrict__ mu_out, float* __restrict__ rstd_out, T* __restrict__ x_copy) {
  constexpr int VN = Vec<T>::N;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int nvec = d / VN;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * d);
  uint4 raw[VPT];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      raw[i] = xr[vi];
      float f[VN]; unpack<T>(raw[i], f);
#pragma unroll
      for (int j = 0; j < VN; ++j) s += f[j];
    }
  }
  const float mu = warp_sum(s) / (float)d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    if (lane + 32 * i < nvec) {
      float f[VN]; unpack<T>(raw[i], f);
#pragma unroll
      for (int j = 0; j < VN; ++j) { float t = f[j] - mu; q += t * t; }
    }
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)d + eps);
  if (lane == 0) { mu_out[row] = mu; rstd_out[row] = rstd; }
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      float f[VN], g[VN], b[VN], o[VN];
      unpack<T>(raw[i], f);
      load_vec<T>(gamma + vi * VN, g);
      load_vec<T>(beta + vi * VN, b);
#pragma unroll
      for (int j = 0; j < VN; ++j) o[j] = (f[j] - mu) * rstd * g[j] + b[j];
      store_vec<T>(out + (size_t)row * d + vi * VN, o);
      if (x_copy) reinterpret_cast<uint4*>(x_copy + (size_t)row * d)[vi] = raw[i];
    }
  }
}

// Forward, one block per row (wide rows).
template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_fwd_kernel(int rows, int d, const T* __restrict__ x, const T* __restrict__ gamma,
                     const T* __restrict__ beta, float eps, T* __restrict__ out,
                     float* __restrict__ mu_out, float* __restrict__ rstd_out, T* __restrict__ x_copy) {
  constexpr int VN = Vec<T>::N;
  __shared__ float red[32];
  const int nvec = d / VN;
  const int row = blockIdx.x;
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

// Backward dx, one warp per row: da and x stay packed in registers.
//   u = da*gamma; dx = rstd*(u - mean(u) - xhat*mean(u*xhat)) (+ add)
template <typename T, int VPT>
__global__ void __launch_bounds__(128)
layernorm_bwd_dx_warp_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                             const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                             const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx) {
  constexpr int VN = Vec<T>::N;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int nvec = d / VN;
  const float mu = mu_in[row], rstd = rstd_in[row];
  const uint4* dar = reinterpret_cast<const uint4*>(da + (size_t)row * d);
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * d);
  uint4 rda[VPT], rx[VPT];
  float s1 = 0.f, s2 = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) { rda[i] = dar[vi]; rx[i] = xr[vi]; }
  }
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      float fd[VN], fx[VN], g[VN];
      unpack<T>(rda[i], fd); unpack<T>(rx[i], fx);
      load_vec<T>(gamma + vi * VN, g);
#pragma unroll
      for (int j = 0; j < VN; ++j) { float u = fd[j] * g[j]; s1 += u; s2 += u * (fx[j] - mu) * rstd; }
    }
  }
  const float c1 = warp_sum(s1) / (float)d, c2 = warp_sum(s2) / (float)d;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      float fd[VN], fx[VN], g[VN], o[VN];
      unpack<T>(rda[i], fd); unpack<T>(rx[i], fx);
      load_vec<T>(gamma + vi * VN, g);
#pragma unroll
      for (int j = 0; j < VN; ++j) o[j] = rstd * (fd[j] * g[j] - c1 - (fx[j] - mu) * rstd * c2);
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

// Backward dx with G warps per row (rows of more than 256 vectors): a lane holds at most 8
// vectors of da and of x, which keeps the kernel at 3 to 4 blocks per SM; the G partial sums of
// a row meet in shared memory behind a barrier of just those warps.
template <typename T, int VPT, int G>
__global__ void __launch_bounds__(256)
layernorm_bwd_dx_group_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                              const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                              const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx) {
  constexpr int VN = Vec<T>::N;
  constexpr int RG = 8 / G;
  __shared__ float2 red[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rg = warp / G, gw = warp % G;
  const int nvec = d / VN;
  const int row = blockIdx.x * RG + rg;
  const bool live = row < rows;
  uint4 rda[VPT], rx[VPT];
  float mu = 0.f, rstd = 0.f, s1 = 0.f, s2 = 0.f;
  if (live) {
    const uint4* dar = reinterpret_cast<const uint4*>(da + (size_t)row * d);
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * d);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = lane + 32 * (i + VPT * gw);
      if (vi < nvec) { rda[i] = dar[vi]; rx[i] = xr[vi]; }
    }
    mu = mu_in[row]; rstd = rstd_in[row];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = lane + 32 * (i + VPT * gw);
      if (vi < nvec) {
        float fd[VN], fx[VN], g[VN];
        unpack<T>(rda[i], fd); unpack<T>(rx[i], fx);
        load_vec<T>(gamma + vi * VN, g);
#pragma unroll
        for (int j = 0; j < VN; ++j) { const float u = fd[j] * g[j]; s1 += u; s2 += u * (fx[j] - mu) * rstd; }
      }
    }
    s1 = warp_sum(s1); s2 = warp_sum(s2);
  }
  if (G > 1) {
    if (lane == 0) red[warp] = make_float2(s1, s2);
    __syncthreads();
    s1 = 0.f; s2 = 0.f;
#pragma unroll
    for (int k = 0; k < G; ++k) { s1 += red[rg * G + k].x; s2 += red[rg * G + k].y; }
  }
  if (!live) return;
  const float c1 = s1 / (float)d, c2 = s2 / (float)d;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = lane + 32 * (i + VPT * gw);
    if (vi < nvec) {
      float fd[VN], fx[VN], g[VN], o[VN];
      unpack<T>(rda[i], fd); unpack<T>(rx[i], fx);
      load_vec<T>(gamma + vi * VN, g);
#pragma unroll
      for (int j = 0; j < VN; ++j) o[j] = rstd * (fd[j] * g[j] - c1 - (fx[j] - mu) * rstd * c2);
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

// Backward dx, one block per row (wide rows).
template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_bwd_dx_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                        const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                        const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx) {
  constexpr int VN = Vec<T>::N;
  __shared__ float2 red[32];
  const int nvec = d / VN;
  const int row = blockIdx.x;
  const float mu = mu_in[row], rstd = rstd_in[row];
  float u[VPT][VN], xh[VPT][VN];
  float s1 = 0.f, s2 = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    int vi = threadIdx.x + i * blockDim.x;
    if (vi < nvec) {
      float dv[VN], xv[VN], g[VN];
      load_vec<T>(da + (size_t)row * d + vi * VN, dv);
      load_vec<T>(x + (size_t)row * d + vi * VN, xv);
      load_vec<T>(gamma + vi * VN, g);
#pragma unroll
      for (int j = 0; j < VN; ++j) {
        xh[i][j] = (xv[j] - mu) * rstd;
        u[i][j] = dv[j] * g[j];
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

// Column reductions over row slabs.  Block = 32 vector columns x 8 row phases;
// grid = (column groups, slabs).  LN = false: partial[slab][c] = sum_r in[r][c].
// LN = true: partial[slab][0][c] = sum_r in[r][c] * xhat[r][c] (dgamma) and
// partial[slab][1][c] = sum_r in[r][c] (dbeta), xhat from x, mu, rstd.
template <typename T, bool LN>
__global__ void __launch_bounds__(256)
colreduce_kernel(int rows, int cols, const T* __restrict__ in, int64_t ld, const T* __restrict__ x,
                 const float* __restrict__ mu, const float* __restrict__ rstd, float* __restrict__ partial) {
  constexpr int VN = Vec<T>::N;
  __shared__ float sm[LN ? 2 : 1][8][32 * VN + 1];
  const int lane = threadIdx.x & 31, ph = threadIdx.x >> 5;
  const int vc = blockIdx.x * 32 + lane;
  const bool active = vc * VN < cols;
  const int per = (rows + gridDim.y - 1) / gridDim.y;
  const int r0 = blockIdx.y * per, r1 = min(rows, r0 + per);
  float a0[VN], a1[VN];
#pragma unroll
  for (int j = 0; j < VN; ++j) { a0[j] = 0.f; a1[j] = 0.f; }
  if (active) {
#pragma unroll 4
    for (int r = r0 + ph; r < r1; r += 8) {
      float v[VN];
      load_vec<T>(in + (size_t)r * ld + vc * VN, v);
      if (LN) {
        float xv[VN];
        load_vec<T>(x + (size_t)r * ld + vc * VN, xv);
        const float m = mu[r], rs = rstd[r];
#pragma unroll
        for (int j = 0; j < VN; ++j) { a0[j] += v[j] * (xv[j] - m) * rs; a1[j] += v[j]; }
      } else {
#pragma unroll
        for (int j = 0; j < VN; ++j) a0[j] += v[j];
      }
    }
  }
#pragma unroll
  for (int j = 0; j < VN; ++j) {
    sm[0][ph][lane * VN + j] = a0[j];
    if (LN) sm[LN ? 1 : 0][ph][lane * VN + j] = a1[j];
  }
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * VN; c += 256) {
    const int gc = blockIdx.x * 32 * VN + c;
    if (gc >= cols) continue;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) { s0 += sm[0][k][c]; if (LN) s1 += sm[LN ? 1 : 0][k][c]; }
    if (LN) {
      partial[(size_t)blockIdx.y * 2 * cols + gc] = s0;
      partial[(size_t)blockIdx.y * 2 * cols + cols + gc] = s1;
    } else {
      partial[(size_t)blockIdx.y * cols + gc] = s0;
    }
  }
}

// out[c] (+)= sum_s partial[s][c] for c < width (width = cols, or 2*cols with out split in two)
__global__ void colreduce_fold_kernel(int slabs, int width, int cols, const float* __restrict__ partial,
                                      float* __restrict__ out0, float* __restrict__ out1, int accumulate) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= width) return;
  float s = 0.f;
  for (int i = 0; i < slabs; ++i) s += partial[(size_t)i * width + c];
  float* dst = (c < cols) ? (out0 + c) : (out1 + (c - cols));
  *dst = accumulate ? (*dst + s) : s;
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

// Row slabs of the column reductions: enough blocks to fill the machine, at most 256 slabs.
int colreduce_slabs(fax_ctx* ctx, int rows, int nvec) {
  const int gx = (nvec + 31) / 32;
  int slabs = (8 * ctx->sm_count + gx - 1) / gx;
  const int max_by_rows = (rows + 31) / 32;
  if (slabs > max_by_rows) slabs = max_by_rows;
  if (slabs > 256) slabs = 256;
  if (slabs < 1) slabs = 1;
  return slabs;
}
int ln_bwd_slabs(fax_ctx* ctx, int rows, int d, int prec) {
  return colreduce_slabs(ctx, rows, d / (prec == FAX_PREC_BF16 ? 8 : 4));
}

template <typename T>
fax_status ln_fwd_t(fax_ctx* ctx, int rows, int d, const void* x, const void* gamma, const void* beta,
                    float eps, void* out, float* mu, float* rstd, void* x_copy) {
  const int nvec = d / Vec<T>::N;
  if (nvec <= 512) {
    const int need = (nvec + 31) / 32;
#define LN_FWDW(V)                                                                                      \
    if (need <= V) {                                                                                    \
      layernorm_fwd_warp_kernel<T, V><<<(rows + 3) / 4, 128, 0, ctx->stream>>>(                         \
          rows, d, (const T*)x, (const T*)gamma, (const T*)beta, eps, (T*)out, mu, rstd, (T*)x_copy);   \
      return fax_after_launch(ctx);                                                                     \
    }
    LN_FWDW(1) LN_FWDW(2) LN_FWDW(3) LN_FWDW(4) LN_FWDW(6) LN_FWDW(8) LN_FWDW(12) LN_FWDW(16)
#undef LN_FWDW
  }
  int threads = 0;
  int vpt = pick_vpt(nvec, 512, &threads);
  if (!vpt) return FAX_ERR_UNSUPPORTED_SHAPE;
#define LN_FWD(V)                                                                                    \
  case V:                                                                                            \
    layernorm_fwd_kernel<T, V><<<rows, threads, 0, ctx->stream>>>(                                   \
        rows, d, (const T*)x, (const T*)gamma, (const T*)beta, eps, (T*)out, mu, rstd, (T*)x_copy);   \
    break;
  switch (vpt) { LN_FWD(1) LN_FWD(2) LN_FWD(3) LN_FWD(4) LN_FWD(6) LN_FWD(8) LN_FWD(12) LN_FWD(16) }
#undef LN_FWD
  return fax_after_launch(ctx);
}

template <typename T>
fax_status ln_bwd_dx_t(fax_ctx* ctx, int rows, int d, const void* da, const void* x, const float* mu,
                       const float* rstd, const void* gamma, const void* add, void* dx) {
  const int nvec = d / Vec<T>::N;
  if (nvec > 256 && nvec <= 512) {
    // two warps per row, 8 vectors per lane
    layernorm_bwd_dx_group_kernel<T, 8, 2><<<(rows + 3) / 4, 256, 0, ctx->stream>>>(
        rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx);
    return fax_after_launch(ctx);
  }
  if (nvec <= 512) {
    const int need = (nvec + 31) / 32;
#define LN_BWDW(V)                                                                                      \
    if (need <= V) {                                                                                    \
      layernorm_bwd_dx_warp_kernel<T, V><<<(rows + 3) / 4, 128, 0, ctx->stream>>>(                      \
          rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx);        \
      return fax_after_launch(ctx);                                                                     \
    }
    LN_BWDW(1) LN_BWDW(2) LN_BWDW(3) LN_BWDW(4) LN_BWDW(6) LN_BWDW(8) LN_BWDW(12) LN_BWDW(16)
#undef LN_BWDW
  }
  int threads = 0;
  int vpt = pick_vpt(nvec, 512, &threads);
  if (!vpt || vpt > 8) return FAX_ERR_UNSUPPORTED_SHAPE;
#define LN_BWD(V)                                                                                   \
  case V:                                                                                           \
    layernorm_bwd_dx_kernel<T, V><<<rows, threads, 0, ctx->stream>>>(                               \
        rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx);      \
    break;
  switch (vpt) { LN_BWD(1) LN_BWD(2) LN_BWD(3) LN_BWD(4) LN_BWD(6) LN_BWD(8) }
#undef LN_BWD
  return fax_after_launch(ctx);
}

template <typename T, bool LN>
fax_status colreduce_t(fax_ctx* ctx, int rows, int cols, const void* in, int64_t ld, const void* x,
                       const float* mu, const float* rstd, float* out0, float* out1, bool accumulate,
                       float* partial) {
  const int nvec = cols / Vec<T>::N;
  const int slabs = colreduce_slabs(ctx, rows, nvec);
  dim3 grid((nvec + 31) / 32, slabs);
  colreduce_kernel<T, LN><<<grid, 256, 0, ctx->stream>>>(rows, cols, (const T*)in, ld, (const T*)x, mu, rstd, partial);
  FAX_TRY(fax_after_launch(ctx));
  const int width = LN ? 2 * cols : cols;
  colreduce_fold_kernel<<<(width + 255) / 256, 256, 0, ctx->stream>>>(slabs, width, cols, partial, out0, out1,
                                                                      accumulate ? 1 : 0);
  return fax_after_launch(ctx);
}

}  // namespace

size_t fax_layernorm_bwd_partial_floats(int rows, int d) {
  (void)rows;
  return (size_t)2 * 256 * d;     // 256 = upper bound of the slab count
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
  if (d % (prec == FAX_PREC_BF16 ? 8 : 4)) return FAX_ERR_UNSUPPORTED_SHAPE;
  if (partial_floats < (size_t)2 * ln_bwd_slabs(ctx, rows, d, prec) * d) return FAX_ERR_WORKSPACE_TOO_SMALL;
  // dx pass reads da, x (and add) and writes dx; the dgamma/dbeta pass reads da and x again
  FaxProfScope prof(ctx, KC_LN_BWD, 0.0, (double)rows * d * fax_elem_size(prec) * (add ? 4 : 3));
  if (prec == FAX_PREC_BF16) {
    FAX_TRY(ln_bwd_dx_t<bf16>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx));
    return colreduce_t<bf16, true>(ctx, rows, d, da, d, x, mu, rstd, dgamma, dbeta, accumulate, partial);
  }
  FAX_TRY(ln_bwd_dx_t<float>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx));
  return colreduce_t<float, true>(ctx, rows, d, da, d, x, mu, rstd, dgamma, dbeta, accumulate, partial);
}

size_t fax_colsum_partial_floats(int rows, int cols) {
  (void)rows;
  return (size_t)256 * cols;
}

fax_status fax_colsum(fax_ctx* ctx, int prec, int rows, int cols, const void* in, int64_t ld, float* out,
                      bool accumulate, float* partial, size_t partial_floats) {
  const int vn = prec == FAX_PREC_BF16 ? 8 : 4;
  if (cols % vn || ld % vn) return FAX_ERR_UNSUPPORTED_SHAPE;
  if (partial_floats < (size_t)colreduce_slabs(ctx, rows, cols / vn) * cols) return FAX_ERR_WORKSPACE_TOO_SMALL;
  FaxProfScope prof(ctx, KC_COLSUM, 0.0, (double)rows * cols * fax_elem_size(prec));
  if (prec == FAX_PREC_BF16)
    return colreduce_t<bf16, false>(ctx, rows, cols, in, ld, nullptr, nullptr, nullptr, out, out, accumulate, partial);
  return colreduce_t<float, false>(ctx, rows, cols, in, ld, nullptr, nullptr, nullptr, out, out, accumulate, partial);
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
  if (ctx->device < 0 || ctx->device >= 64) return FAX_ERR_ARCH;
  if (d % (prec == FAX_PREC_BF16 ? 8 : 4)) return FAX_ERR_UNSUPPORTED_SHAPE;
  // the array holds 2 * 256 * FAX_LN_STATIC_MAX_D partial sums: any row count, d up to the stated maximum
  if (d > FAX_LN_STATIC_MAX_D || (size_t)2 * ln_bwd_slabs(ctx, rows, d, prec) * d > (size_t)FAX_LN_STATIC_SCRATCH_FLOATS)
    return FAX_ERR_WORKSPACE_TOO_SMALL;
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
