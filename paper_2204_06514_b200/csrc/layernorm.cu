// LayerNorm forward / backward (block steps F1, F5, B3, B7 and the LM's final
// LayerNorm).  HBM-bound: rows stay packed in registers between the reductions and the
// output pass, 128-bit loads and stores, two-pass mean / variance.  Rows of up to 512
// vectors: groups of warps walk rows with the next row in flight, and the backward pass
// accumulates dgamma / dbeta in registers on the way; wider rows: one block per row and a
// separate column reduction.
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

// Forward for rows of up to 512 vectors: a block of 512 threads holds 16 / WG row groups of WG
// warps; a group walks rows, gamma and beta stay in registers, the next row is requested before
// the current one is reduced (two-pass mean / variance, each a shuffle reduction plus, for
// WG > 1, one barrier of the group's own).
template <typename T, int VPT, int WG>
__global__ void __launch_bounds__(512, (VPT <= 2) ? 2 : 1)
layernorm_fwd_group_kernel(int rows, int d, const T* __restrict__ x, const T* __restrict__ gamma,
                           const T* __restrict__ beta, float eps, T* __restrict__ out,
                           float* __restrict__ mu_out, float* __restrict__ rstd_out, T* __restrict__ x_copy) {
  fax_grid_dependency_wait();
  constexpr int VN = Vec<T>::N;
  constexpr int NG = 16 / WG, TG = 32 * WG;
  __shared__ float red[2][16];
  const int grp = threadIdx.x / TG, t = threadIdx.x % TG;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = d / VN;
  const int stride = NG * gridDim.x;
  const float inv_d = 1.f / (float)d;
  uint4 gm[VPT], bt[VPT], nxt[VPT];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = t + TG * i;
    const bool in = vi < nvec;
    gm[i] = in ? reinterpret_cast<const uint4*>(gamma)[vi] : make_uint4(0, 0, 0, 0);
    bt[i] = in ? reinterpret_cast<const uint4*>(beta)[vi] : make_uint4(0, 0, 0, 0);
    nxt[i] = make_uint4(0, 0, 0, 0);
  }
  int row = NG * blockIdx.x + grp;
  if (row < rows) {
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * d);
#pragma unroll
    for (int i = 0; i < VPT; ++i) if (t + TG * i < nvec) nxt[i] = xr[t + TG * i];
  }
  for (; row < rows; row += stride) {
    uint4 cur[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) cur[i] = nxt[i];
    if (row + stride < rows) {
      const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)(row + stride) * d);
#pragma unroll
      for (int i = 0; i < VPT; ++i) if (t + TG * i < nvec) nxt[i] = xr[t + TG * i];
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      if (t + TG * i < nvec) {
        float f[VN]; unpack<T>(cur[i], f);
#pragma unroll
        for (int j = 0; j < VN; ++j) s += f[j];
      }
    }
    s = warp_sum(s);
    if (WG > 1) {
      if (lane == 0) red[0][warp] = s;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(TG) : "memory");
      s = 0.f;
#pragma unroll
      for (int k = 0; k < WG; ++k) s += red[0][grp * WG + k];
    }
    const float mu = s * inv_d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      if (t + TG * i < nvec) {
        float f[VN]; unpack<T>(cur[i], f);
#pragma unroll
        for (int j = 0; j < VN; ++j) { const float c = f[j] - mu; q += c * c; }
      }
    }
    q = warp_sum(q);
    if (WG > 1) {
      if (lane == 0) red[1][warp] = q;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(TG) : "memory");
      q = 0.f;
#pragma unroll
      for (int k = 0; k < WG; ++k) q += red[1][grp * WG + k];
    }
    const float rstd = rsqrtf(q * inv_d + eps);
    if (t == 0) { mu_out[row] = mu; rstd_out[row] = rstd; }
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = t + TG * i;
      if (vi < nvec) {
        float f[VN], g[VN], b[VN], o[VN];
        unpack<T>(cur[i], f); unpack<T>(gm[i], g); unpack<T>(bt[i], b);
#pragma unroll
        for (int j = 0; j < VN; ++j) o[j] = (f[j] - mu) * rstd * g[j] + b[j];
        store_vec<T>(out + (size_t)row * d + vi * VN, o);
        if (x_copy) reinterpret_cast<uint4*>(x_copy + (size_t)row * d)[vi] = cur[i];
      }
    }
  }
}

// Forward, one block per row (wide rows).
template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_fwd_kernel(int rows, int d, const T* __restrict__ x, const T* __restrict__ gamma,
                     const T* __restrict__ beta, float eps, T* __restrict__ out,
                     float* __restrict__ mu_out, float* __restrict__ rstd_out, T* __restrict__ x_copy) {
  fax_grid_dependency_wait();
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

// ---- asynchronous copies into shared memory (each thread later reads only what it copied) ----
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
               ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int LN_RING = 3;        // rows in flight per row group: the current one and two ahead

// Backward, fused: dx and the per-block column sums for dgamma / dbeta in one pass over da and x.
// A block of 512 threads holds 16 / WG row groups of WG warps; a group walks rows
// (group index + k * groups in the grid), every thread owning the same VPT vector columns in all
// of them, so the column sums accumulate in registers.  Rows are staged through shared memory: a
// group keeps LN_RING rows of da, x (and the residual gradient) in flight as asynchronous 16-byte
// copies, each thread copying exactly the vectors it will read, so no barrier guards the ring and
// the memory latency of two rows hides under the current one.  At the end the groups of a block add
// their sums in shared memory and the block writes one slab: partial[block][0][c] = sum da*xhat,
// partial[block][1][c] = sum da.
// Dynamic shared memory: 2 (with SUMS: 4) * d floats for the final reduction, then the ring
// [row group][slot][da | x | add][32 * WG * VPT vectors].
// SUMS: also the column sums of `add` and of the output dx (the bias gradients of the linear layers on
// either side of the LayerNorm: partial[block][2][c] = sum add, partial[block][3][c] = sum dx), which
// costs two more accumulators per column and no memory traffic.
template <typename T, int VPT, int WG, bool SUMS>
__global__ void __launch_bounds__(512, 1)
layernorm_bwd_ring_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                          const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                          const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx,
                          float* __restrict__ partial) {
  fax_grid_dependency_wait();
  constexpr int VN = Vec<T>::N;
  constexpr int NG = 16 / WG, TG = 32 * WG, PER = TG * VPT;
  extern __shared__ uint4 ring_sm_raw[];
  constexpr int NS = SUMS ? 4 : 2;                                     // column sums per column
  float* fuse_sm = reinterpret_cast<float*>(ring_sm_raw);              // NS * d floats
  __shared__ float2 red[2][16];
  const int grp = threadIdx.x / TG, t = threadIdx.x % TG;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = d / VN;
  const int stride = NG * gridDim.x;
  const float inv_d = 1.f / (float)d;
  uint4* ring = ring_sm_raw + (NS * d * 4 + 15) / 16 + (size_t)grp * LN_RING * 3 * PER;
  float ag[VPT][VN], ab[VPT][VN], aa[SUMS ? VPT : 1][VN], ao[SUMS ? VPT : 1][VN];
  uint4 gm[VPT];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
#pragma unroll
    for (int j = 0; j < VN; ++j) { ag[i][j] = 0.f; ab[i][j] = 0.f; if (SUMS) { aa[i][j] = 0.f; ao[i][j] = 0.f; } }
    const int vi = t + TG * i;
    gm[i] = (vi < nvec) ? reinterpret_cast<const uint4*>(gamma)[vi] : make_uint4(0, 0, 0, 0);
  }
  auto issue = [&](int r, int slot) {
    if (r < rows) {
      uint4* s0 = ring + (size_t)slot * 3 * PER;
      const uint4* dar = reinterpret_cast<const uint4*>(da + (size_t)r * d);
      const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)r * d);
      const uint4* adr = reinterpret_cast<const uint4*>(add + (size_t)r * d);
#pragma unroll
      for (int i = 0; i < VPT; ++i) {
        const int vi = t + TG * i;
        if (vi < nvec) {
          cp_async16(s0 + vi, dar + vi);
          cp_async16(s0 + PER + vi, xr + vi);
          if (add) cp_async16(s0 + 2 * PER + vi, adr + vi);
        }
      }
    }
    cp_async_commit();          // one group per call, empty past the last row, so the counting stays uniform
  };
  int row = NG * blockIdx.x + grp;
  issue(row, 0);
  issue(row + stride, 1);
  float mu0 = 0.f, rs0 = 0.f, mu1 = 0.f, rs1 = 0.f;
  if (row < rows) { mu0 = mu_in[row]; rs0 = rstd_in[row]; }
  if (row + stride < rows) { mu1 = mu_in[row + stride]; rs1 = rstd_in[row + stride]; }
  int slot = 0;
  for (int it = 0; row < rows; row += stride, ++it) {
    const int ahead = row + 2 * stride;
    issue(ahead, slot >= 1 ? slot - 1 : LN_RING - 1);        // the slot read in the iteration before this one
    float mu2 = 0.f, rs2 = 0.f;
    if (ahead < rows) { mu2 = mu_in[ahead]; rs2 = rstd_in[ahead]; }
    cp_async_wait<2>();                                       // all but the two newest groups: this row has landed
    const float mu = mu0, rstd = rs0;
    mu0 = mu1; rs0 = rs1; mu1 = mu2; rs1 = rs2;
    const uint4* s0 = ring + (size_t)slot * 3 * PER;
    uint4 cda[VPT], cx[VPT];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = t + TG * i;
      if (vi < nvec) {
        cda[i] = s0[vi]; cx[i] = s0[PER + vi];
        float fd[VN], fx[VN], g[VN];
        unpack<T>(cda[i], fd); unpack<T>(cx[i], fx); unpack<T>(gm[i], g);
#pragma unroll
        for (int j = 0; j < VN; ++j) { const float u = fd[j] * g[j]; s1 += u; s2 += u * (fx[j] - mu) * rstd; }
      }
    }
    s1 = warp_sum(s1); s2 = warp_sum(s2);
    if (WG > 1) {
      if (lane == 0) red[it & 1][warp] = make_float2(s1, s2);
      asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(TG) : "memory");
      s1 = 0.f; s2 = 0.f;
#pragma unroll
      for (int k = 0; k < WG; ++k) { const float2 v = red[it & 1][grp * WG + k]; s1 += v.x; s2 += v.y; }
    }
    const float c1 = s1 * inv_d, c2 = s2 * inv_d;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = t + TG * i;
      if (vi < nvec) {
        float fd[VN], fx[VN], g[VN], o[VN];
        unpack<T>(cda[i], fd); unpack<T>(cx[i], fx); unpack<T>(gm[i], g);
#pragma unroll
        for (int j = 0; j < VN; ++j) {
          const float xh = (fx[j] - mu) * rstd;
          o[j] = rstd * (fd[j] * g[j] - c1 - xh * c2);
          ag[i][j] += fd[j] * xh;
          ab[i][j] += fd[j];
        }
        if (add) {
          float av[VN];
          unpack<T>(s0[2 * PER + vi], av);
#pragma unroll
          for (int j = 0; j < VN; ++j) { o[j] += av[j]; if (SUMS) aa[i][j] += av[j]; }
        }
        if (SUMS) {
#pragma unroll
          for (int j = 0; j < VN; ++j) ao[i][j] += o[j];
        }
        store_vec<T>(dx + (size_t)row * d + vi * VN, o);
      }
    }
    slot = (slot + 1 == LN_RING) ? 0 : slot + 1;
  }
  cp_async_wait<0>();
  __syncthreads();
  // the groups add their column sums one after the other (fixed order: deterministic)
  auto fold4 = [&](float* base, const float (&v)[VN], int vi, bool first) {
#pragma unroll
    for (int j = 0; j < VN; j += 4) {
      float4* pp = reinterpret_cast<float4*>(base + vi * VN + j);
      float4 w = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      if (!first) { const float4 o4 = *pp; w.x += o4.x; w.y += o4.y; w.z += o4.z; w.w += o4.w; }
      *pp = w;
    }
  };
  for (int g = 0; g < NG; ++g) {
    if (grp == g) {
#pragma unroll
      for (int i = 0; i < VPT; ++i) {
        const int vi = t + TG * i;
        if (vi < nvec) {
          fold4(fuse_sm, ag[i], vi, g == 0);
          fold4(fuse_sm + d, ab[i], vi, g == 0);
          if (SUMS) {
            fold4(fuse_sm + 2 * d, aa[i], vi, g == 0);
            fold4(fuse_sm + 3 * d, ao[i], vi, g == 0);
          }
        }
      }
    }
    __syncthreads();
  }
  float4* dst = reinterpret_cast<float4*>(partial + (size_t)blockIdx.x * NS * d);
  for (int c = threadIdx.x; c < NS * d / 4; c += blockDim.x) dst[c] = reinterpret_cast<const float4*>(fuse_sm)[c];
}

// Backward, fused, rows of 513 .. 2048 vectors: the same one pass as the ring kernel with the whole block
// (16 warps) on one row at a time.  Thread t owns vectors t + 512 i, i < VPT, of every row the block walks
// (blockIdx.x + k * gridDim.x), so the column sums stay in registers and each block writes its slab
// straight from them.  The ring holds RING rows of da, x (and add) per block; the second pass over a row
// re-reads the slot (it stays valid until the next iteration's copy is issued) instead of keeping the
// row in registers, which leaves the registers to the column sums.  One block-wide barrier per row.
// Dynamic shared memory: [slot][da | x | add][512 * VPT vectors].
template <typename T, int VPT, int RING, bool SUMS>
__global__ void __launch_bounds__(512, 1)
layernorm_bwd_wide_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                          const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                          const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx,
                          float* __restrict__ partial) {
  fax_grid_dependency_wait();
  constexpr int VN = Vec<T>::N;
  constexpr int PER = 512 * VPT;
  constexpr int NS = SUMS ? 4 : 2;
  extern __shared__ uint4 ring_sm_raw[];
  uint4* ring = ring_sm_raw;
  __shared__ float2 red[2][16];
  const int t = threadIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = d / VN;
  const int stride = gridDim.x;
  const float inv_d = 1.f / (float)d;
  float ag[VPT][VN], ab[VPT][VN], aa[SUMS ? VPT : 1][VN], ao[SUMS ? VPT : 1][VN];
  uint4 gm[VPT];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
#pragma unroll
    for (int j = 0; j < VN; ++j) { ag[i][j] = 0.f; ab[i][j] = 0.f; if (SUMS) { aa[i][j] = 0.f; ao[i][j] = 0.f; } }
    const int vi = t + 512 * i;
    gm[i] = (vi < nvec) ? reinterpret_cast<const uint4*>(gamma)[vi] : make_uint4(0, 0, 0, 0);
  }
  auto issue = [&](int r, int slot) {
    if (r < rows) {
      uint4* s0 = ring + (size_t)slot * 3 * PER;
      const uint4* dar = reinterpret_cast<const uint4*>(da + (size_t)r * d);
      const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)r * d);
      const uint4* adr = reinterpret_cast<const uint4*>(add + (size_t)r * d);
#pragma unroll
      for (int i = 0; i < VPT; ++i) {
        const int vi = t + 512 * i;
        if (vi < nvec) {
          cp_async16(s0 + vi, dar + vi);
          cp_async16(s0 + PER + vi, xr + vi);
          if (add) cp_async16(s0 + 2 * PER + vi, adr + vi);
        }
      }
    }
    cp_async_commit();          // one group per call, empty past the last row, so the counting stays uniform
  };
  int row = blockIdx.x;
#pragma unroll
  for (int k = 0; k < RING - 1; ++k) issue(row + k * stride, k);
  int slot = 0;
  float mu_next = 0.f, rstd_next = 0.f;                                     // the row statistics, one row ahead
  if (row < rows) { mu_next = mu_in[row]; rstd_next = rstd_in[row]; }
  for (int it = 0; row < rows; row += stride, ++it) {
    issue(row + (RING - 1) * stride, slot >= 1 ? slot - 1 : RING - 1);      // the slot read in the iteration before this one
    const float mu = mu_next, rstd = rstd_next;
    if (row + stride < rows) { mu_next = mu_in[row + stride]; rstd_next = rstd_in[row + stride]; }
    cp_async_wait<RING - 1>();                                              // all but the newest groups: this row has landed
    const uint4* s0 = ring + (size_t)slot * 3 * PER;
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = t + 512 * i;
      if (vi < nvec) {
        float fd[VN], fx[VN], g[VN];
        unpack<T>(s0[vi], fd); unpack<T>(s0[PER + vi], fx); unpack<T>(gm[i], g);
#pragma unroll
        for (int j = 0; j < VN; ++j) { const float u = fd[j] * g[j]; s1 += u; s2 += u * (fx[j] - mu) * rstd; }
      }
    }
    s1 = warp_sum(s1); s2 = warp_sum(s2);
    if (lane == 0) red[it & 1][warp] = make_float2(s1, s2);
    __syncthreads();
    s1 = 0.f; s2 = 0.f;
#pragma unroll
    for (int k = 0; k < 16; ++k) { const float2 v = red[it & 1][k]; s1 += v.x; s2 += v.y; }
    const float c1 = s1 * inv_d, c2 = s2 * inv_d;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int vi = t + 512 * i;
      if (vi < nvec) {
        float fd[VN], fx[VN], g[VN], o[VN];
        unpack<T>(s0[vi], fd); unpack<T>(s0[PER + vi], fx); unpack<T>(gm[i], g);
#pragma unroll
        for (int j = 0; j < VN; ++j) {
          const float xh = (fx[j] - mu) * rstd;
          o[j] = rstd * (fd[j] * g[j] - c1 - xh * c2);
          ag[i][j] += fd[j] * xh;
          ab[i][j] += fd[j];
        }
        if (add) {
          float av[VN];
          unpack<T>(s0[2 * PER + vi], av);
#pragma unroll
          for (int j = 0; j < VN; ++j) { o[j] += av[j]; if (SUMS) aa[i][j] += av[j]; }
        }
        if (SUMS) {
#pragma unroll
          for (int j = 0; j < VN; ++j) ao[i][j] += o[j];
        }
        store_vec<T>(dx + (size_t)row * d + vi * VN, o);
      }
    }
    slot = (slot + 1 == RING) ? 0 : slot + 1;
  }
  cp_async_wait<0>();
  float* slab = partial + (size_t)blockIdx.x * NS * d;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int vi = t + 512 * i;
    if (vi < nvec) {
#pragma unroll
      for (int j = 0; j < VN; j += 4) {
        *reinterpret_cast<float4*>(slab + vi * VN + j) = make_float4(ag[i][j], ag[i][j + 1], ag[i][j + 2], ag[i][j + 3]);
        *reinterpret_cast<float4*>(slab + d + vi * VN + j) = make_float4(ab[i][j], ab[i][j + 1], ab[i][j + 2], ab[i][j + 3]);
        if (SUMS) {
          *reinterpret_cast<float4*>(slab + 2 * d + vi * VN + j) = make_float4(aa[i][j], aa[i][j + 1], aa[i][j + 2], aa[i][j + 3]);
          *reinterpret_cast<float4*>(slab + 3 * d + vi * VN + j) = make_float4(ao[i][j], ao[i][j + 1], ao[i][j + 2], ao[i][j + 3]);
        }
      }
    }
  }
}

// Backward dx, one block per row (wide rows).
template <typename T, int VPT>
__global__ void __launch_bounds__(512)
layernorm_bwd_dx_kernel(int rows, int d, const T* __restrict__ da, const T* __restrict__ x,
                        const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                        const T* __restrict__ gamma, const T* __restrict__ add, T* __restrict__ dx) {
  fax_grid_dependency_wait();
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
  fax_grid_dependency_wait();
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

// out[c] (+)= sum_s partial[s][c] for c < width (width = cols, 2*cols or 4*cols with out split accordingly).
// Block = 32 columns x 8 slab phases, summed in a fixed order.
__global__ void __launch_bounds__(256)
colreduce_fold_kernel(int slabs, int width, int cols, const float* __restrict__ partial,
                      float* __restrict__ out0, float* __restrict__ out1, float* __restrict__ out2,
                      float* __restrict__ out3, int accumulate) {
  fax_grid_dependency_wait();
  __shared__ float sm[8][33];
  const int lane = threadIdx.x & 31, ph = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  float s = 0.f;
  if (c < width) {
#pragma unroll 4
    for (int i = ph; i < slabs; i += 8) s += partial[(size_t)i * width + c];
  }
  sm[ph][lane] = s;
  __syncthreads();
  if (ph == 0 && c < width) {
    s = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) s += sm[k][lane];
    const int q = c / cols;                      // which of the (up to four) sums of width `cols`
    float* dst = (q == 0 ? out0 : q == 1 ? out1 : q == 2 ? out2 : out3) + (c - q * cols);
    *dst = accumulate ? (*dst + s) : s;
  }
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

// Row slabs of the column reductions: as many blocks as are resident at once (a grid a little
// larger than that would leave a second, nearly empty wave), at most 256 slabs.
int colreduce_slabs(fax_ctx* ctx, int rows, int nvec, int blocks_per_sm) {
  const int gx = (nvec + 31) / 32;
  int slabs = blocks_per_sm * ctx->sm_count / gx;
  const int max_by_rows = (rows + 31) / 32;
  if (slabs > max_by_rows) slabs = max_by_rows;
  if (slabs > 256) slabs = 256;
  if (slabs < 1) slabs = 1;
  return slabs;
}
// Resident 256-thread blocks per SM: 8 for the plain column sum (32 registers), 5 for the
// LayerNorm variant (48 registers).
constexpr int kColsumBlocksPerSm = 8, kLnColBlocksPerSm = 5;
// The fused backward covers rows of up to 2048 vectors (up to 512: row groups inside a block, above: one
// row per block at a time); one slab per block, one block per SM.  The bias-gradient sums ride along up
// to 1024 vectors (wider rows have no registers left for four sums per column).
// The one-row-per-block kernel takes every register of an SM, so it cannot be placed beside the persistent
// AdamW blocks of the optimizer stream and waits for a whole AdamW launch to finish (measured: +1.7 % on the
// step at hidden 5120 and 8192 with the overlap on): while that stream is busy the wide rows take the
// block-per-row dx kernel and a column reduction, whose small blocks fit beside the optimizer's.
bool ln_bwd_is_fused(const fax_ctx* ctx, int nvec) { return nvec <= 512 || (nvec <= 2048 && !ctx->side_busy); }
bool ln_bwd_fuses_sums(int nvec) { return nvec <= 1024; }
int ln_row_groups(int nvec) { return nvec <= 64 ? 16 : nvec <= 128 ? 8 : nvec <= 256 ? 4 : 2; }
int ln_bwd_fused_grid(fax_ctx* ctx, int rows, int nvec) {
  const int ng = nvec > 512 ? 1 : ln_row_groups(nvec);
  int grid = (rows + ng - 1) / ng;
  if (grid > ctx->sm_count) grid = ctx->sm_count;
  if (grid > 256) grid = 256;
  return grid < 1 ? 1 : grid;
}
int ln_bwd_slabs(fax_ctx* ctx, int rows, int d, int prec) {
  const int nvec = d / (prec == FAX_PREC_BF16 ? 8 : 4);
  return ln_bwd_is_fused(ctx, nvec) ? ln_bwd_fused_grid(ctx, rows, nvec) : colreduce_slabs(ctx, rows, nvec, kLnColBlocksPerSm);
}

template <typename T>
fax_status ln_fwd_t(fax_ctx* ctx, int rows, int d, const void* x, const void* gamma, const void* beta,
                    float eps, void* out, float* mu, float* rstd, void* x_copy) {
  const int nvec = d / Vec<T>::N;
  if (nvec <= 512) {
    // narrow rows: one warp per row with 3 or 4 vectors per lane (more bytes in flight per thread)
    const bool wide_lane = nvec > 64 && nvec <= 128;
    const int ng = wide_lane ? 16 : ln_row_groups(nvec);
    int grid = (rows + ng - 1) / ng;
    const int cap = (wide_lane ? 1 : 2) * ctx->sm_count;
    if (grid > cap) grid = cap;
#define LN_FWDG(V, W)                                                                                   \
    fax_launch(ctx, layernorm_fwd_group_kernel<T, V, W>, dim3(grid), dim3(512), 0,                      \
               rows, d, (const T*)x, (const T*)gamma, (const T*)beta, eps, (T*)out, mu, rstd, (T*)x_copy)
    if (nvec <= 32) LN_FWDG(1, 1);
    else if (nvec <= 64) LN_FWDG(2, 1);
    else if (nvec <= 96) LN_FWDG(3, 1);
    else if (nvec <= 128) LN_FWDG(4, 1);
    else if (nvec <= 256) LN_FWDG(2, 4);
    else LN_FWDG(2, 8);
#undef LN_FWDG
    return fax_after_launch(ctx);
  }
  int threads = 0;
  int vpt = pick_vpt(nvec, 512, &threads);
  if (!vpt) return FAX_ERR_UNSUPPORTED_SHAPE;
#define LN_FWD(V)                                                                                    \
  case V:                                                                                            \
    fax_launch(ctx, layernorm_fwd_kernel<T, V>, dim3(rows), dim3(threads), 0,                        \
               rows, d, (const T*)x, (const T*)gamma, (const T*)beta, eps, (T*)out, mu, rstd, (T*)x_copy); \
    break;
  switch (vpt) { LN_FWD(1) LN_FWD(2) LN_FWD(3) LN_FWD(4) LN_FWD(6) LN_FWD(8) LN_FWD(12) LN_FWD(16) }
#undef LN_FWD
  return fax_after_launch(ctx);
}

template <typename T>
fax_status ln_bwd_dx_t(fax_ctx* ctx, int rows, int d, const void* da, const void* x, const float* mu,
                       const float* rstd, const void* gamma, const void* add, void* dx) {
  const int nvec = d / Vec<T>::N;
  int threads = 0;
  int vpt = pick_vpt(nvec, 512, &threads);
  if (!vpt || vpt > 8) return FAX_ERR_UNSUPPORTED_SHAPE;
#define LN_BWD(V)                                                                                   \
  case V:                                                                                           \
    fax_launch(ctx, layernorm_bwd_dx_kernel<T, V>, dim3(rows), dim3(threads), 0,                    \
               rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx); \
    break;
  switch (vpt) { LN_BWD(1) LN_BWD(2) LN_BWD(3) LN_BWD(4) LN_BWD(6) LN_BWD(8) }
#undef LN_BWD
  return fax_after_launch(ctx);
}

template <typename T>
fax_status ln_bwd_fused_t(fax_ctx* ctx, int rows, int d, const void* da, const void* x, const float* mu,
                          const float* rstd, const void* gamma, const void* add, void* dx, float* dgamma,
                          float* dbeta, bool accumulate, float* partial, float* sum_add, float* sum_out) {
  const int nvec = d / Vec<T>::N;
  const int grid = ln_bwd_fused_grid(ctx, rows, nvec);
  const bool sums = sum_add && sum_out && add;
  const int ns = sums ? 4 : 2;
  if (nvec > 512) {
    // one row per block at a time: ring of R slots x 3 arrays x 512 * V vectors of 16 bytes
#define LN_WIDE_S(V, R, S)                                                                             \
    {                                                                                                  \
      const size_t smem = (size_t)(R) * 3 * 512 * (V) * 16;                                            \
      static bool attr_set[FAX_MAX_DEVICES] = {};                                                      \
      FAX_TRY(fax_opt_in_shared_memory(ctx, layernorm_bwd_wide_kernel<T, V, R, S>, (int)smem, attr_set)); \
      fax_launch(ctx, layernorm_bwd_wide_kernel<T, V, R, S>, dim3(grid), dim3(512), smem,              \
                 rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx, partial); \
    }
    if (nvec <= 1024) { if (sums) LN_WIDE_S(2, 3, true) else LN_WIDE_S(2, 3, false) }
    else if (sums) return FAX_ERR_INVALID_ARG;
    else if (nvec <= 1536) LN_WIDE_S(3, 3, false)
    else LN_WIDE_S(4, 2, false)
#undef LN_WIDE_S
    FAX_TRY(fax_after_launch(ctx));
    fax_launch(ctx, colreduce_fold_kernel, dim3((ns * d + 31) / 32), dim3(256), 0, grid, ns * d, d, (const float*)partial,
               dgamma, dbeta, sum_add, sum_out, accumulate ? 1 : 0);
    return fax_after_launch(ctx);
  }
  // dynamic shared memory: 2 * d floats for the final reduction (rounded up to whole 16-byte vectors),
  // then the ring: 16 / W groups x LN_RING slots x 3 arrays x 32 * W * V vectors of 16 bytes; the
  // opt-in limit covers the widest row an instantiation serves (512 vectors)
  auto ring_bytes = [](int V, int W) { return (size_t)(16 / W) * LN_RING * 3 * (32 * W * V) * 16; };
#define LN_FUSED_S(V, W, S)                                                                            \
  {                                                                                                    \
    const size_t smem = ((size_t)ns * d * sizeof(float) + 15) / 16 * 16 + ring_bytes(V, W);            \
    static bool attr_set[FAX_MAX_DEVICES] = {};                                                        \
    FAX_TRY(fax_opt_in_shared_memory(ctx, layernorm_bwd_ring_kernel<T, V, W, S>,                       \
                                     (int)((size_t)(S ? 4 : 2) * 512 * Vec<T>::N * sizeof(float) + ring_bytes(V, W)), \
                                     attr_set));                                                       \
    fax_launch(ctx, layernorm_bwd_ring_kernel<T, V, W, S>, dim3(grid), dim3(512), smem,                \
               rows, d, (const T*)da, (const T*)x, mu, rstd, (const T*)gamma, (const T*)add, (T*)dx, partial); \
  }
#define LN_FUSED(V, W) { if (sums) LN_FUSED_S(V, W, true) else LN_FUSED_S(V, W, false) }
  if (nvec <= 32) LN_FUSED(1, 1)
  else if (nvec <= 64) LN_FUSED(2, 1)
  else if (nvec <= 128) LN_FUSED(2, 2)
  else if (nvec <= 256) LN_FUSED(2, 4)
  else LN_FUSED(2, 8)
#undef LN_FUSED
#undef LN_FUSED_S
  FAX_TRY(fax_after_launch(ctx));
  fax_launch(ctx, colreduce_fold_kernel, dim3((ns * d + 31) / 32), dim3(256), 0, grid, ns * d, d, (const float*)partial,
             dgamma, dbeta, sum_add, sum_out, accumulate ? 1 : 0);
  return fax_after_launch(ctx);
}

template <typename T, bool LN>
fax_status colreduce_t(fax_ctx* ctx, int rows, int cols, const void* in, int64_t ld, const void* x,
                       const float* mu, const float* rstd, float* out0, float* out1, bool accumulate,
                       float* partial) {
  const int nvec = cols / Vec<T>::N;
  const int slabs = colreduce_slabs(ctx, rows, nvec, LN ? kLnColBlocksPerSm : kColsumBlocksPerSm);
  dim3 grid((nvec + 31) / 32, slabs);
  fax_launch(ctx, colreduce_kernel<T, LN>, grid, dim3(256), 0, rows, cols, (const T*)in, ld, (const T*)x, mu, rstd, partial);
  FAX_TRY(fax_after_launch(ctx));
  const int width = LN ? 2 * cols : cols;
  fax_launch(ctx, colreduce_fold_kernel, dim3((width + 31) / 32), dim3(256), 0, slabs, width, cols, (const float*)partial,
             out0, out1, (float*)nullptr, (float*)nullptr, accumulate ? 1 : 0);
  return fax_after_launch(ctx);
}

}  // namespace

size_t fax_layernorm_bwd_partial_floats(int rows, int d) {
  (void)rows;
  return (size_t)4 * 256 * d;     // 256 = upper bound of the slab count; four sums per column with the bias gradients
}

fax_status fax_layernorm_fwd(fax_ctx* ctx, int prec, int rows, int d, const void* x, const void* gamma,
                             const void* beta, float eps, void* out, float* mu, float* rstd, void* x_copy) {
  // read x, write out (and the optional copy of x)
  // algorithmic bytes: read x, write the normalised rows (a copy of x kept for backward, where a caller
  // asks for one, is extra traffic and not counted)
  FaxProfScope prof(ctx, KC_LN_FWD, 0.0, (double)rows * d * fax_elem_size(prec) * 2);
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
                             size_t partial_floats, float* sum_add, float* sum_out) {
  if (d % (prec == FAX_PREC_BF16 ? 8 : 4)) return FAX_ERR_UNSUPPORTED_SHAPE;
  const bool sums = sum_add && sum_out && add;
  const int nvec_all = d / (prec == FAX_PREC_BF16 ? 8 : 4);
  const bool fused = ln_bwd_is_fused(ctx, nvec_all);
  const bool fused_sums = fused && ln_bwd_fuses_sums(nvec_all);
  if (partial_floats < (size_t)(sums && fused_sums ? 4 : 2) * ln_bwd_slabs(ctx, rows, d, prec) * d) return FAX_ERR_WORKSPACE_TOO_SMALL;
  if (sums && !fused_sums) {
    // wide rows: the column sums of add and dx as reductions of their own, after the LayerNorm kernels
    FAX_TRY(fax_layernorm_bwd(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, accumulate, partial,
                              partial_floats, nullptr, nullptr));
    FAX_TRY(fax_colsum(ctx, prec, rows, d, add, d, sum_add, accumulate, partial, partial_floats));
    return fax_colsum(ctx, prec, rows, d, dx, d, sum_out, accumulate, partial, partial_floats);
  }
  // dx pass reads da, x (and add) and writes dx; the dgamma/dbeta pass reads da and x again
  FaxProfScope prof(ctx, KC_LN_BWD, 0.0, (double)rows * d * fax_elem_size(prec) * (add ? 4 : 3));
  if (fused) {
    if (prec == FAX_PREC_BF16)
      return ln_bwd_fused_t<bf16>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, accumulate, partial,
                                  sum_add, sum_out);
    return ln_bwd_fused_t<float>(ctx, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, accumulate, partial,
                                 sum_add, sum_out);
  }
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
  if (partial_floats < (size_t)colreduce_slabs(ctx, rows, cols / vn, kColsumBlocksPerSm) * cols) return FAX_ERR_WORKSPACE_TOO_SMALL;
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
    // (the symbol is looked up on the current device, so the context's device is made current
    // for the query and the caller's choice put back afterwards)
    int caller_device = -1;
    FAX_CUDA_TRY(ctx, cudaGetDevice(&caller_device));
    FAX_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    float* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_ln_static_partial);
    if (caller_device != ctx->device) (void)cudaSetDevice(caller_device);
    FAX_CUDA_TRY(ctx, e);
    if (!ptr) return FAX_ERR_CUDA;
    g_ln_static_ptr[ctx->device] = ptr;
  }
  // Every slab writes its whole slice of the partials before the fold kernel reads it, so
  // nothing in the shared array has to start at zero and stale contents are harmless.
  return fax_layernorm_bwd(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, false,
                           g_ln_static_ptr[ctx->device], FAX_LN_STATIC_SCRATCH_FLOATS);
}
