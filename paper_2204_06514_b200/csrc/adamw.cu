// Multi-tensor AdamW over float32 master weights (step U).  HBM-bound: 128-bit
// loads and stores, one pass, writes the bf16 compute copy in the same pass.
// Algorithmic traffic per element: read w, m, v, g (16 B) + write w, m, v
// (12 B) + write bf16 copy (2 B) = 30 B.
#include "common.cuh"

#include <cstring>

namespace {

constexpr int MAX_T = 40;              // tensors per launch (kernel-parameter space)
constexpr int CHUNK = 4096;            // elements per block iteration
constexpr int THREADS = 256;

struct AdamTensor {
  float* w; float* m; float* v; const void* g; bf16* wc;
  unsigned long long n;
  float wd;
  unsigned int first_chunk;            // prefix sum of chunk counts
};
struct AdamBatch {
  AdamTensor t[MAX_T];
  int n_tensors;
  unsigned int total_chunks;
};

struct AdamScalars { float lr, b1, b2, eps, inv_bc1, inv_bc2; };

template <bool G_BF16>
__device__ __forceinline__ void adam_elem(float& w, float& m, float& v, float g, float wd,
                                          const AdamScalars& s) {
  m = s.b1 * m + (1.f - s.b1) * g;
  v = s.b2 * v + (1.f - s.b2) * g * g;
  float mh = m * s.inv_bc1;
  float vh = v * s.inv_bc2;
  w = w - s.lr * wd * w - s.lr * mh / (sqrtf(vh) + s.eps);
}

template <bool G_BF16>
__global__ void __launch_bounds__(THREADS)
adamw_kernel(const __grid_constant__ AdamBatch batch, AdamScalars sc) {
  fax_grid_dependency_wait();
  for (unsigned int chunk = blockIdx.x; chunk < batch.total_chunks; chunk += gridDim.x) {
    // find the tensor this chunk belongs to (few tensors: linear scan from a binary start)
    int lo = 0, hi = batch.n_tensors - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (batch.t[mid].first_chunk <= chunk) lo = mid; else hi = mid - 1;
    }
    const AdamTensor& t = batch.t[lo];
    unsigned long long base = (unsigned long long)(chunk - t.first_chunk) * CHUNK;
    unsigned long long end = base + CHUNK < t.n ? base + CHUNK : t.n;
    const bool vec_ok = ((t.n & 3ull) == 0);
    if (vec_ok) {
      // a full chunk is 4 float4 groups per thread: issue all loads first, then update and store
      constexpr int U = CHUNK / (4 * THREADS);
      float4 w[U], m[U], v[U], g[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const unsigned long long e = base + 4ull * (threadIdx.x + u * THREADS);
        if (e < end) {
          w[u] = *reinterpret_cast<const float4*>(t.w + e);
          m[u] = *reinterpret_cast<const float4*>(t.m + e);
          v[u] = *reinterpret_cast<const float4*>(t.v + e);
          if (G_BF16) {
            uint2 raw = *reinterpret_cast<const uint2*>((const bf16*)t.g + e);
            float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.x));
            float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.y));
            g[u] = make_float4(a.x, a.y, b.x, b.y);
          } else {
            g[u] = *reinterpret_cast<const float4*>((const float*)t.g + e);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const unsigned long long e = base + 4ull * (threadIdx.x + u * THREADS);
        if (e < end) {
          adam_elem<G_BF16>(w[u].x, m[u].x, v[u].x, g[u].x, t.wd, sc);
          adam_elem<G_BF16>(w[u].y, m[u].y, v[u].y, g[u].y, t.wd, sc);
          adam_elem<G_BF16>(w[u].z, m[u].z, v[u].z, g[u].z, t.wd, sc);
          adam_elem<G_BF16>(w[u].w, m[u].w, v[u].w, g[u].w, t.wd, sc);
          *reinterpret_cast<float4*>(t.w + e) = w[u];
          *reinterpret_cast<float4*>(t.m + e) = m[u];
          *reinterpret_cast<float4*>(t.v + e) = v[u];
          if (t.wc) {
            uint2 o;
            *reinterpret_cast<__nv_bfloat162*>(&o.x) = __floats2bfloat162_rn(w[u].x, w[u].y);
            *reinterpret_cast<__nv_bfloat162*>(&o.y) = __floats2bfloat162_rn(w[u].z, w[u].w);
            *reinterpret_cast<uint2*>(t.wc + e) = o;
          }
        }
      }
    } else {
      for (unsigned long long e = base + threadIdx.x; e < end; e += THREADS) {
        float w = t.w[e], m = t.m[e], v = t.v[e];
        float g = G_BF16 ? __bfloat162float(((const bf16*)t.g)[e]) : ((const float*)t.g)[e];
        adam_elem<G_BF16>(w, m, v, g, t.wd, sc);
        t.w[e] = w; t.m[e] = m; t.v[e] = v;
        if (t.wc) t.wc[e] = __float2bfloat16_rn(w);
      }
    }
  }
}

}  // namespace

static AdamScalars make_scalars(const fax_adamw_hparams* hp) {
  AdamScalars sc;
  sc.lr = hp->lr; sc.b1 = hp->beta1; sc.b2 = hp->beta2; sc.eps = hp->eps;
  sc.inv_bc1 = (float)(1.0 / (1.0 - pow((double)hp->beta1, (double)hp->step)));
  sc.inv_bc2 = (float)(1.0 / (1.0 - pow((double)hp->beta2, (double)hp->step)));
  return sc;
}

bool fax_adamw_is_kernel(const void* func) {
  return func == (const void*)adamw_kernel<false> || func == (const void*)adamw_kernel<true>;
}

void fax_adamw_scalars(const fax_adamw_hparams* hp, void* out32) {
  static_assert(sizeof(AdamScalars) <= 32, "scalar block");
  AdamScalars sc = make_scalars(hp);
  memcpy(out32, &sc, sizeof(sc));
}

fax_status fax_adamw_launch(fax_ctx* ctx, const fax_adamw_tensor* tensors, int n, const fax_adamw_hparams* hp) {
  if (!tensors || !hp || n < 0) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  AdamScalars sc = make_scalars(hp);
  for (int i = 0; i < n; ++i) {
    const fax_adamw_tensor& t = tensors[i];
    if (!t.w || !t.m || !t.v || !t.g) return FAX_ERR_INVALID_ARG;
    if (!fax_aligned(t.w, 16) || !fax_aligned(t.m, 16) || !fax_aligned(t.v, 16) || !fax_aligned(t.g, 16) ||
        (t.w_compute && !fax_aligned(t.w_compute, 8)))
      return FAX_ERR_INVALID_ARG;
  }
  double total = 0;
  for (int j = 0; j < n; ++j) total += (double)tensors[j].n;
  // read w, m, v, g; write w, m, v and the bf16 copy
  FaxProfScope prof(ctx, KC_ADAMW, 0.0, total * (hp->grad_is_bf16 ? 28.0 : 30.0));
  int i = 0;
  while (i < n) {
    AdamBatch batch;
    int k = 0;
    unsigned long long chunks = 0;
    while (i < n && k < MAX_T) {
      const fax_adamw_tensor& t = tensors[i++];
      if (t.n == 0) continue;
      unsigned long long c = (t.n + CHUNK - 1) / CHUNK;
      if (chunks + c > 0xffffffffull) { --i; break; }
      batch.t[k].w = t.w; batch.t[k].m = t.m; batch.t[k].v = t.v; batch.t[k].g = t.g;
      batch.t[k].wc = (bf16*)t.w_compute; batch.t[k].n = t.n; batch.t[k].wd = t.weight_decay;
      batch.t[k].first_chunk = (unsigned int)chunks;
      chunks += c;
      ++k;
    }
    if (k == 0) { if (i < n && chunks == 0 && tensors[i].n > 0) return FAX_ERR_UNSUPPORTED_SHAPE; continue; }
    batch.n_tensors = k;
    batch.total_chunks = (unsigned int)chunks;
    unsigned long long want = chunks;
    // on the optimizer stream keep two blocks per SM so that the main stream's kernels still fit beside them
    const unsigned long long cap = (unsigned long long)ctx->sm_count * (ctx->stream == ctx->side ? 2 : 16);
    unsigned int grid = (unsigned int)(want < cap ? want : cap);
    if (hp->grad_is_bf16)
      fax_launch(ctx, adamw_kernel<true>, dim3(grid), dim3(THREADS), 0, batch, sc);
    else
      fax_launch(ctx, adamw_kernel<false>, dim3(grid), dim3(THREADS), 0, batch, sc);
    FAX_TRY(fax_after_launch(ctx));
  }
  return FAX_OK;
}

fax_status fax_adamw_async(fax_ctx* ctx, const fax_adamw_tensor* tensors, int n, const fax_adamw_hparams* hp) {
  if (!ctx->overlap_adamw) return fax_adamw_launch(ctx, tensors, n, hp);
  FAX_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
  FAX_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
  cudaStream_t main_stream = ctx->stream;
  ctx->stream = ctx->side;
  fax_status s = fax_adamw_launch(ctx, tensors, n, hp);
  ctx->stream = main_stream;
  ctx->side_busy = true;
  return s;
}

fax_status fax_adamw_join(fax_ctx* ctx) {
  if (!ctx->side_busy) return FAX_OK;
  FAX_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
  FAX_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0));
  ctx->side_busy = false;
  return FAX_OK;
}

extern "C" fax_status fax_adamw_step(fax_ctx* ctx, const fax_adamw_tensor* tensors, int32_t n_tensors,
                                     const fax_adamw_hparams* hp) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  return fax_adamw_launch(ctx, tensors, n_tensors, hp);
}
