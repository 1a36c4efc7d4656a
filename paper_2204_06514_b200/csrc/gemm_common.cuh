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
  float* ad_w; float* ad_m; float* ad_v; bf16* ad_wc;   // EPI_ADAMW: state of the weight this GEMM's result updates
  float ad_wd; float ad_sc[8]; int ad_keep;
  int group_m;         // tiles per raster group along the grouped dimension
  int group_along_n;   // 0: groups of row-tiles swept across the columns; 1: groups of column-tiles swept down the rows
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

// Tile order: groups of `group` row-tiles are swept across all column-tiles before the next group
// starts (along_n: groups of column-tiles swept down all row-tiles), so the tiles in flight share
// few A row-panels and B column-panels in L2, and the group's own panels stay in L2 from one wave
// of tiles to the next while the other operand streams past once per group.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int group, int along_n, int& tm, int& tn) {
  const int t_g = along_n ? tiles_n : tiles_m;      // tiles along the grouped dimension
  const int t_s = along_n ? tiles_m : tiles_n;      // tiles along the swept dimension
  const int per_group = group * t_s;
  const int g = tile / per_group;
  const int first = g * group;
  const int width = min(group, t_g - first);
  const int in = tile - g * per_group;
  const int ig = first + in % width, is = in / width;
  tm = along_n ? is : ig;
  tn = along_n ? ig : is;
}

// Epilogue of one 32-column chunk held in registers: row `row`, columns col .. col+31.
// EPI >= 0: the epilogue mode is a compile-time constant (the kernels are instantiated per mode,
// which keeps each one's epilogue code short and branch-free): EPI_NONE .. EPI_DGELU with bf16
// output, EPI_STATIC_F32 = plain float output (stored, accumulated or added by K slices);
// EPI < 0: mode, output type, accumulation and K-slicing are read from the parameters.
constexpr int EPI_STATIC_F32 = 6;

// The residual / pre-activation values one chunk needs (32 bf16 of row `row` from column col),
// requested ahead of the chunk's turn so that their latency hides under the previous chunk.
// (Only the kernels with a compile-time mode fetch ahead; the run-time-mode epilogue loads the
// values when it needs them, which keeps it within its register budget.)
template <int EPI, bool NOW = false>
__device__ __forceinline__ void gemm_epilogue_fetch(const GemmParams& p, long long row, int col, U8 (&x)[2]) {
  if (EPI < 0 && !NOW) return;
  const int epi = EPI == EPI_STATIC_F32 ? (int)EPI_NONE : (EPI >= 0 ? EPI : p.epi);
  if (epi == EPI_BIAS_RESID) {
    const bf16* rp = p.resid + row * p.ldr + col;
    x[0] = ld_global_v8(rp); x[1] = ld_global_v8(rp + 16);
  } else if (epi == EPI_DGELU) {
    const bf16* ap = p.aux + row * p.ldaux + col;
    x[0] = ld_global_v8(ap); x[1] = ld_global_v8(ap + 16);
  }
}

// Values of one chunk before they are stored: alpha * accumulator (+ bias) (+ residual) (* GELU'(pre-activation));
// xv holds the chunk's 32 residual / pre-activation values where the mode reads any.
template <int EPI>
__device__ __forceinline__ void gemm_epilogue_values(const GemmParams& p, const uint32_t (&r)[32], const U8* xv, int p_epi,
                                                     int col, float (&v)[32]) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) * p.alpha;
        if (p_epi == EPI_BIAS || p_epi == EPI_BIAS_GELU || p_epi == EPI_BIAS_RESID) {
          const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col);
#pragma unroll
          for (int j4 = 0; j4 < 4; ++j4) {
            uint4 u = __ldg(bp + j4);
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int e = 0; e < 4; ++e) { float2 f = __bfloat1622float2(h[e]); v[8 * j4 + 2 * e] += f.x; v[8 * j4 + 2 * e + 1] += f.y; }
          }
        }
        if (p_epi == EPI_BIAS_RESID) {
#pragma unroll
          for (int j8 = 0; j8 < 2; ++j8) {
            const U8& u = xv[j8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.w[e]));
              v[16 * j8 + 2 * e] += f.x; v[16 * j8 + 2 * e + 1] += f.y;
            }
          }
        }
        if (p_epi == EPI_DGELU) {
#pragma unroll
          for (int j8 = 0; j8 < 2; ++j8) {
            const U8& u = xv[j8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.w[e]));
              v[16 * j8 + 2 * e] *= gelu_grad_fast(f.x);
              v[16 * j8 + 2 * e + 1] *= gelu_grad_fast(f.y);
            }
          }
        }
}

template <int EPI>
__device__ __forceinline__ void gemm_epilogue_chunk(const GemmParams& pr, const uint32_t (&r)[32], const U8 (&x)[2],
                                                    long long row, int col) {
        const GemmParams& p = pr;
        const int p_epi = EPI == EPI_STATIC_F32 ? (int)EPI_NONE : (EPI >= 0 ? EPI : pr.epi);
        const bool p_c_f32 = EPI == EPI_STATIC_F32 ? true : (EPI >= 0 ? false : (pr.c_f32 != 0));
        U8 xn[2];
        if (EPI < 0) gemm_epilogue_fetch<EPI, true>(pr, row, col, xn);
        const U8* xv = EPI < 0 ? xn : x;
        float v[32];
        gemm_epilogue_values<EPI>(p, r, xv, p_epi, col, v);
        if (p_epi == EPI_ADAMW) {
          // the accumulator is the gradient of w[row, col..]: AdamW here, w / m / v in place
          const long long off = row * p.ldc + col;
          const float lr = p.ad_sc[0], b1 = p.ad_sc[1], b2 = p.ad_sc[2], eps = p.ad_sc[3];
          const float ibc1 = p.ad_sc[4], ibc2 = p.ad_sc[5];
#pragma unroll
          for (int j8 = 0; j8 < 4; ++j8) {
            U8 w8 = ld_global_v8(p.ad_w + off + 8 * j8);
            U8 m8 = ld_global_v8(p.ad_m + off + 8 * j8);
            U8 v8 = ld_global_v8(p.ad_v + off + 8 * j8);
            uint4 c8;
            __nv_bfloat162* ch = reinterpret_cast<__nv_bfloat162*>(&c8);
            float wn[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float g = v[8 * j8 + e];
              float w = __uint_as_float(w8.w[e]), m = __uint_as_float(m8.w[e]), vv = __uint_as_float(v8.w[e]);
              m = b1 * m + (1.f - b1) * g;
              vv = b2 * vv + (1.f - b2) * g * g;
              const float mh = m * ibc1, vh = vv * ibc2;
              w = w - lr * p.ad_wd * w - lr * mh / (sqrtf(vh) + eps);
              w8.w[e] = __float_as_uint(w); m8.w[e] = __float_as_uint(m); v8.w[e] = __float_as_uint(vv);
              wn[e] = w;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) ch[e] = __floats2bfloat162_rn(wn[2 * e], wn[2 * e + 1]);
            st_global_v8(p.ad_w + off + 8 * j8, w8);
            st_global_v8(p.ad_m + off + 8 * j8, m8);
            st_global_v8(p.ad_v + off + 8 * j8, v8);
            *reinterpret_cast<uint4*>(p.ad_wc + off + 8 * j8) = c8;
            if (p.ad_keep) {
              U8 g8;
#pragma unroll
              for (int e = 0; e < 8; ++e) g8.w[e] = __float_as_uint(v[8 * j8 + e]);
              st_global_v8((float*)p.C + off + 8 * j8, g8);
            }
          }
        } else if (p_c_f32) {
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
          bf16* gp = (p_epi == EPI_BIAS_GELU) ? (p.aux + row * p.ldaux + col) : nullptr;
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

// The compile-time epilogue mode a problem runs with (see gemm_epilogue_chunk).
static inline int gemm_static_epi(const FaxGemm& g) {
  if (g.adam) return -1;
  if (g.c_f32) return g.epi == EPI_NONE ? EPI_STATIC_F32 : -1;
  return (g.epi >= EPI_NONE && g.epi <= EPI_DGELU) ? g.epi : -1;
}

// Fills the kernel parameters that do not depend on the tile shape.
static inline void fill_gemm_params(GemmParams& p, const FaxGemm& g, int32_t* status) {
  p.M = g.M; p.N = g.N; p.K = g.K; p.a_mn = g.a_mn_major; p.b_mn = g.b_mn_major;
  p.C = g.C; p.ldc = g.ldc; p.c_f32 = g.c_f32; p.accumulate = g.accumulate; p.epi = g.epi;
  p.bias = (const bf16*)g.bias; p.resid = (const bf16*)g.resid; p.ldr = g.ldr; p.aux = (bf16*)g.aux; p.ldaux = g.ldaux;
  p.alpha = g.alpha; p.status = status;
  p.group_m = 8; p.group_along_n = 0;
  p.splits = 1;
  p.ad_w = p.ad_m = p.ad_v = nullptr; p.ad_wc = nullptr; p.ad_wd = 0.f; p.ad_keep = 0;
  for (int i = 0; i < 8; ++i) p.ad_sc[i] = 0.f;
  if (g.adam) {
    p.epi = EPI_ADAMW;
    p.ad_w = g.adam->w; p.ad_m = g.adam->m; p.ad_v = g.adam->v; p.ad_wc = (bf16*)g.adam->w_compute;
    p.ad_wd = g.adam->weight_decay; p.ad_keep = g.adam->keep_grad ? 1 : 0;
    for (int i = 0; i < 8; ++i) p.ad_sc[i] = g.adam->sc[i];
  }
}

// Raster order of a problem with tile_m x tile_n tiles, `units` of them in flight.  DRAM reads are
// (panel = one tile's rows or columns of an operand over all of K):
//   grouped along M, G row-panels of A kept in L2:  A once + B once per group  = A + B * ceil(tiles_m / G)
//   grouped along N, G column-panels of B kept:      B once + A once per group  = B + A * ceil(tiles_n / G)
// as long as the group's panels fit the share of L2 that is left to them (l2_budget bytes); when even
// a few panels do not fit (long K), nothing survives from wave to wave and the square-ish 8-tile group,
// which minimises the panels one wave touches, stays.
static inline void gemm_choose_raster(GemmParams& p, int tile_m, int tile_n, int units, double l2_budget) {
  const int tiles_m = p.M / tile_m, tiles_n = p.N / tile_n;
  const double a_bytes = 2.0 * p.M * p.K, b_bytes = 2.0 * p.N * p.K;
  const double pa = 2.0 * tile_m * p.K, pb = 2.0 * tile_n * p.K;
  p.group_m = 8; p.group_along_n = 0;
  if (tiles_m * tiles_n <= units) return;                          // a single wave
  const int g0 = tiles_m < 8 ? tiles_m : 8;
  const double waves = (double)tiles_m * tiles_n / units;
  double best = waves * (g0 * pa + ((double)units / g0) * pb);     // no reuse between waves
  auto consider = [&](bool along_n) {
    const int t_g = along_n ? tiles_n : tiles_m;
    const double panel = along_n ? pb : pa;
    int g = (int)(l2_budget / panel);
    if (g < 4) return;                                             // too few panels in a wave to be worth keeping
    if (g > t_g) g = t_g;
    const int groups = (t_g + g - 1) / g;
    g = (t_g + groups - 1) / groups;                               // even groups
    const double traffic = along_n ? b_bytes + a_bytes * groups : a_bytes + b_bytes * groups;
    if (traffic < best) { best = traffic; p.group_m = g; p.group_along_n = along_n ? 1 : 0; }
  };
  consider(false);
  consider(true);
}

// Number of K slices the launchers use for a problem with `tiles` output tiles on `units`
// tile-processing units (SMs, or SM pairs).  Only plain float outputs are sliced (the partial tiles
// are added into C).  Cost model in K blocks: waves of work items x (K blocks per item + a per-item
// overhead for the epilogue and the pipeline refill); slicing pays when the tiles alone leave units
// idle (fewer tiles than units) or fill the last wave badly.
static inline int gemm_split_count(const FaxGemm& g, int tiles, int units, int bk) {
  const int kb_total = g.K / bk;
  if (!(g.c_f32 && g.epi == EPI_NONE && g.alpha == 1.f && !g.adam && kb_total >= 16)) return 1;
  if (tiles >= 4 * units) return 1;
  auto slices = [&](int sp) { const int kb_per = (kb_total + sp - 1) / sp; return (kb_total + kb_per - 1) / kb_per; };
  auto cost = [&](int sp) {
    const int kb_per = (kb_total + sp - 1) / sp;
    const long long items = (long long)tiles * slices(sp);
    const long long waves = (items + units - 1) / units;
    return (double)waves * (kb_per + (sp > 1 ? 6 : 3));
  };
  int best = 1;
  for (int sp = 2; sp <= 16 && kb_total / sp >= 8; ++sp)
    if (cost(sp) < 0.95 * cost(best)) best = sp;
  return slices(best);                              // no empty slices
}

// One warp's share of a tile: NCH chunks of 32 columns starting at tensor-memory address
// t_base / global column col0.  Two register buffers keep the load of the next chunk in
// flight while the current one is stored; x0 holds the first chunk's residual / pre-activation
// values (gemm_epilogue_fetch, issued by the caller before it waits for the accumulator).  `drained` runs as soon as the last chunk has been
// read out of tensor memory (before its stores): the accumulator can be handed back to the MMA
// issuer while this warp is still writing to global memory.
template <int NCH, int EPI, typename Drained>
__device__ __forceinline__ void gemm_epilogue_warp(const GemmParams& p, uint32_t t_base, long long row, int col0,
                                                   const U8 (&x0)[2], Drained drained) {
  uint32_t ra[32], rb[32];
  U8 xa[2], xb[2];
  xa[0] = x0[0]; xa[1] = x0[1];
  tc_ld32(t_base, ra);
#pragma unroll
  for (int i = 0; i < NCH; i += 2) {
    if (i + 1 < NCH) gemm_epilogue_fetch<EPI>(p, row, col0 + 32 * (i + 1), xb);
    tc_wait_ld();
    if (i + 1 < NCH) tc_ld32(t_base + 32 * (i + 1), rb); else drained();
    gemm_epilogue_chunk<EPI>(p, ra, xa, row, col0 + 32 * i);
    if (i + 1 < NCH) {
      if (i + 2 < NCH) gemm_epilogue_fetch<EPI>(p, row, col0 + 32 * (i + 2), xa);
      tc_wait_ld();
      if (i + 2 < NCH) tc_ld32(t_base + 32 * (i + 2), ra); else drained();
      gemm_epilogue_chunk<EPI>(p, rb, xb, row, col0 + 32 * (i + 1));
    }
  }
}

// ---- K-sliced float output: partial tiles added into C by bulk tensor reductions ----
//
// A warp owns 32 rows x 128 columns of the tile, four chunks of 32 columns, and one 4 KB staging buffer.
// Each thread writes its own row of a chunk (32 floats) into the buffer in the 128-byte-swizzled layout
// the tensor map expects; one lane then issues the bulk add-reduction (float add at L2), which replaces
// eight float4 atomics per thread and chunk.  Only this mode stages its output: for the stored outputs
// the shared-memory traffic of a staged tile (written once, read once by the copy engine) slows the main
// loop, whose operand staging already uses the shared-memory bandwidth, by more than the scattered
// 32-byte stores from registers cost.
constexpr int EPI_STAGING_BYTES = 4096;      // per epilogue warp
constexpr int EPI_TMA_CHUNKS = 4;

// Byte offset of the 16-byte unit `unit` of row `r` in a staging buffer (128-byte rows, 128-byte swizzle;
// buffers are 1024-byte aligned).
__device__ __forceinline__ uint32_t epi_sw128(int r, int unit) { return (uint32_t)(r * 128 + ((unit ^ (r & 7)) << 4)); }

template <typename Drained>
__device__ __forceinline__ void gemm_epilogue_warp_reduce(const GemmParams& p, const CUtensorMap* mc, uint32_t t_base,
                                                          int row0, int col0, int lane, uint32_t stg, Drained drained) {
  uint32_t rr[2][32];
  tc_ld32(t_base, rr[0]);
#pragma unroll
  for (int i = 0; i < EPI_TMA_CHUNKS; ++i) {
    tc_wait_ld();
    if (i + 1 < EPI_TMA_CHUNKS) tc_ld32(t_base + 32 * (i + 1), rr[(i + 1) & 1]); else drained();
    if (lane == 0) bulk_wait_read<0>();        // the previous chunk's reduction has read the buffer
    __syncwarp();
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint32_t* r = rr[i & 1];
      st_shared_v4(stg + epi_sw128(lane, u), __float_as_uint(__uint_as_float(r[4 * u]) * p.alpha),
                   __float_as_uint(__uint_as_float(r[4 * u + 1]) * p.alpha),
                   __float_as_uint(__uint_as_float(r[4 * u + 2]) * p.alpha),
                   __float_as_uint(__uint_as_float(r[4 * u + 3]) * p.alpha));
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      tma_reduce_add_2d(mc, stg, col0 + 32 * i, row0);
      bulk_commit_group();
    }
  }
}

}  // namespace tc
