// Pieces shared by the one-CTA and the two-CTA GEMM kernels: parameters, tile order,
// and the fused epilogue that moves one warp's share of an accumulator tile from
// tensor memory to global memory.
#pragma once
#include "tc_common.cuh"

namespace tc {

struct GemmParams {
  int M, N, K;
  int a_mn, b_mn;
  void* C; long long ldc; int c_f32; int accumulate;
  int epi;
  const bf16* bias;
  const bf16* resid; long long ldr;
  bf16* aux; long long ldaux;
  float alpha;
  int32_t* status;
  int group_m;         // row-tiles per raster group
  int splits;          // > 1: each work item covers a slice of K and adds its partial tile into a float C
};

// GELU (tanh form) and its derivative with the hardware tanh approximation: its error
// (about 5e-4 relative) is below the bf16 rounding of the values the epilogue stores.
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_fast(float h) {
  const float t = tanh_fast(0.7978845608028654f * (h + 0.044715f * h * h * h));
  return 0.5f * h * (1.0f + t);
}
__device__ __forceinline__ float gelu_grad_fast(float h) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  const float t = tanh_fast(c * (h + a * h * h * h));
  return 0.5f * (1.0f + t) + 0.5f * h * (1.0f - t * t) * c * (1.0f + 3.0f * a * h * h);
}

// Tile order: groups of group_m row-tiles are swept across all column-tiles before the next
// group starts, so the ~148 tiles in flight share few A row-panels and B column-panels in L2.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int group_m, int& tm, int& tn) {
  const int per_group = group_m * tiles_n;
  const int g = tile / per_group;
  const int first_m = g * group_m;
  const int rows = min(group_m, tiles_m - first_m);
  const int in = tile - g * per_group;
  tm = first_m + in % rows;
  tn = in / rows;
}

// Epilogue of one 32-column chunk held in registers: row `row`, columns col .. col+31.
__device__ __forceinline__ void gemm_epilogue_chunk(const GemmParams& p, const uint32_t (&r)[32], long long row, int col) {
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) * p.alpha;
        if (p.epi == EPI_BIAS || p.epi == EPI_BIAS_GELU || p.epi == EPI_BIAS_RESID) {
          const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col);
#pragma unroll
          for (int j4 = 0; j4 < 4; ++j4) {
            uint4 u = __ldg(bp + j4);
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int e = 0; e < 4; ++e) { float2 f = __bfloat1622float2(h[e]); v[8 * j4 + 2 * e] += f.x; v[8 * j4 + 2 * e + 1] += f.y; }
          }
        }
        if (p.epi == EPI_BIAS_RESID) {
          const bf16* rp = p.resid + row * p.ldr + col;
#pragma unroll
          for (int j8 = 0; j8 < 2; ++j8) {
            const U8 u = ld_global_v8(rp + 16 * j8);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.w[e]));
              v[16 * j8 + 2 * e] += f.x; v[16 * j8 + 2 * e + 1] += f.y;
            }
          }
        }
        if (p.epi == EPI_DGELU) {
          const bf16* ap = p.aux + row * p.ldaux + col;
#pragma unroll
          for (int j8 = 0; j8 < 2; ++j8) {
            const U8 u = ld_global_v8(ap + 16 * j8);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.w[e]));
              v[16 * j8 + 2 * e] *= gelu_grad_fast(f.x);
              v[16 * j8 + 2 * e + 1] *= gelu_grad_fast(f.y);
            }
          }
        }
        if (p.c_f32) {
          float* cp = (float*)p.C + row * p.ldc + col;
          if (p.splits > 1) {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4)
              atomicAdd(reinterpret_cast<float4*>(cp) + j4, make_float4(v[4 * j4], v[4 * j4 + 1], v[4 * j4 + 2], v[4 * j4 + 3]));
          } else {
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8) {
              U8 o;
#pragma unroll
              for (int e = 0; e < 8; ++e) o.w[e] = __float_as_uint(v[8 * j8 + e]);
              if (p.accumulate) {
                const U8 c = ld_global_v8(cp + 8 * j8);
#pragma unroll
                for (int e = 0; e < 8; ++e) o.w[e] = __float_as_uint(__uint_as_float(o.w[e]) + __uint_as_float(c.w[e]));
              }
              st_global_v8(cp + 8 * j8, o);
            }
          }
        } else {
          bf16* cp = (bf16*)p.C + row * p.ldc + col;
          bf16* gp = (p.epi == EPI_BIAS_GELU) ? (p.aux + row * p.ldaux + col) : nullptr;
#pragma unroll
          for (int j8 = 0; j8 < 2; ++j8) {
            U8 u;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(v[16 * j8 + 2 * e], v[16 * j8 + 2 * e + 1]);
              u.w[e] = *reinterpret_cast<uint32_t*>(&h2);
            }
            st_global_v8(cp + 16 * j8, u);
            if (gp) {
              // GELU of the stored (rounded) pre-activation, so backward sees the same h
              U8 g;
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.w[e]));
                __nv_bfloat162 g2 = __floats2bfloat162_rn(gelu_fast(f.x), gelu_fast(f.y));
                g.w[e] = *reinterpret_cast<uint32_t*>(&g2);
              }
              st_global_v8(gp + 16 * j8, g);
            }
          }
        }
}

// One warp's share of a tile: NCH chunks of 32 columns starting at tensor-memory address
// t_base / global column col0.  Two register buffers keep the load of the next chunk in
// flight while the current one is stored.
template <int NCH>
__device__ __forceinline__ void gemm_epilogue_warp(const GemmParams& p, uint32_t t_base, long long row, int col0) {
  uint32_t ra[32], rb[32];
  tc_ld32(t_base, ra);
#pragma unroll
  for (int i = 0; i < NCH; i += 2) {
    tc_wait_ld();
    if (i + 1 < NCH) tc_ld32(t_base + 32 * (i + 1), rb);
    gemm_epilogue_chunk(p, ra, row, col0 + 32 * i);
    if (i + 1 < NCH) {
      tc_wait_ld();
      if (i + 2 < NCH) tc_ld32(t_base + 32 * (i + 2), ra);
      gemm_epilogue_chunk(p, rb, row, col0 + 32 * (i + 1));
    }
  }
}

}  // namespace tc
