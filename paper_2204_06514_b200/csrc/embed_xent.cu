// Embedding lookup / scatter and softmax cross-entropy of the LM step
// (steps LM-E, LM-H loss part, LM-B).  All HBM-bound.
#include "common.cuh"

namespace {

template <typename T>
__global__ void embed_fwd_kernel(int n_tok, int Tn, int d, int vocab, const int32_t* __restrict__ ids,
                                 const T* __restrict__ wte, const T* __restrict__ wpe, T* __restrict__ x0) {
  fax_grid_dependency_wait();
  int n = blockIdx.x;
  int id = ids[n];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);     // ids are validated upstream; clamp keeps reads in bounds
  const T* e = wte + (size_t)id * d;
  const T* p = wpe + (size_t)(n % Tn) * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    x0[(size_t)n * d + c] = from_f32<T>(to_f32(e[c]) + to_f32(p[c]));
}

// dwte[ids[n]] += dx0[n]   (float atomics on top of the head gradient)
template <typename T>
__global__ void embed_bwd_wte_kernel(int n_tok, int d, int vocab, const int32_t* __restrict__ ids,
                                     const T* __restrict__ dx0, float* __restrict__ dwte) {
  fax_grid_dependency_wait();
  int n = blockIdx.x;
  int id = ids[n];
  if (id < 0 || id >= vocab) return;
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    atomicAdd(dwte + (size_t)id * d + c, to_f32(dx0[(size_t)n * d + c]));
}

// dwpe[t] = sum_b dx0[b, t]   (fixed order: deterministic); rows t >= Tn are zeroed
template <typename T>
__global__ void embed_bwd_wpe_kernel(int Bn, int Tn, int max_seq, int d, const T* __restrict__ dx0,
                                     float* __restrict__ dwpe, int accumulate) {
  fax_grid_dependency_wait();
  int t = blockIdx.x;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float s = 0.f;
    if (t < Tn)
      for (int b = 0; b < Bn; ++b) s += to_f32(dx0[((size_t)b * Tn + t) * d + c]);
    dwpe[(size_t)t * d + c] = accumulate ? dwpe[(size_t)t * d + c] + s : s;
  }
}

__device__ __forceinline__ float block_reduce_max(float v, float* red) {
  v = warp_max(v);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = lane < nw ? red[lane] : -INFINITY;
  return warp_max(t);
}
__device__ __forceinline__ float block_reduce_sum(float v, float* red) {
  v = warp_sum(v);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = lane < nw ? red[lane] : 0.f;
  return warp_sum(t);
}

// One block per row of a logits chunk.  In place: logits -> (softmax - onehot) * inv_n.
// row_loss[row0 + r] = logsumexp - logit[target].
template <typename T>
__global__ void __launch_bounds__(512)
xent_kernel(int rows, int vocab, T* __restrict__ logits, int64_t ld, const int32_t* __restrict__ targets,
            float inv_n, float* __restrict__ row_loss) {
  fax_grid_dependency_wait();
  __shared__ float red[32];
  int r = blockIdx.x;
  T* row = logits + (size_t)r * ld;
  float mx = -INFINITY;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) mx = fmaxf(mx, to_f32(row[c]));
  mx = block_reduce_max(mx, red);
  float s = 0.f;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) s += __expf(to_f32(row[c]) - mx);
  s = block_reduce_sum(s, red);
  int tg = targets[r];
  float lse = mx + logf(s);
  if (threadIdx.x == 0) {
    float lt = (tg >= 0 && tg < vocab) ? to_f32(row[tg]) : lse;
    row_loss[r] = lse - lt;
  }
  __syncthreads();
  float inv_s = 1.f / s;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
    float p = __expf(to_f32(row[c]) - mx) * inv_s;
    if (c == tg) p -= 1.f;
    row[c] = from_f32<T>(p * inv_n);
  }
}

// bf16 rows that fit in shared memory: the row is read from HBM once.  Pass 1 copies it to
// shared memory and takes the maximum; pass 2 replaces each logit by exp(logit - max)
// (bf16) while summing the unrounded exponentials; pass 3 writes (e / sum - onehot) * inv_n.
__global__ void __launch_bounds__(512)
xent_smem_kernel(int rows, int vocab, bf16* __restrict__ logits, int64_t ld, const int32_t* __restrict__ targets,
                 float inv_n, float* __restrict__ row_loss) {
  fax_grid_dependency_wait();
  extern __shared__ uint4 xrow[];               // vocab / 8 vectors of 8 bf16
  __shared__ float red[32];
  const int r = blockIdx.x;
  uint4* grow = reinterpret_cast<uint4*>(logits + (size_t)r * ld);
  const int nvec = vocab >> 3;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    const uint4 u = grow[i];
    xrow[i] = u;
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) { float2 f = __bfloat1622float2(h[e]); mx = fmaxf(mx, fmaxf(f.x, f.y)); }
  }
  mx = block_reduce_max(mx, red);
  const int tg = targets[r];
  float s = 0.f;
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    uint4 u = xrow[i];
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 f = __bfloat1622float2(h[e]);
      const float e0 = __expf(f.x - mx), e1 = __expf(f.y - mx);
      s += e0 + e1;
      h[e] = __floats2bfloat162_rn(e0, e1);
    }
    xrow[i] = u;
  }
  float lt = 0.f;
  if (threadIdx.x == 0 && tg >= 0 && tg < vocab) lt = __bfloat162float(logits[(size_t)r * ld + tg]);   // still the logit: global row not yet rewritten
  s = block_reduce_sum(s, red);
  if (threadIdx.x == 0) {
    const float lse = mx + logf(s);
    row_loss[r] = (tg >= 0 && tg < vocab) ? lse - lt : 0.f;
  }
  const float k = inv_n / s;
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    uint4 u = xrow[i];
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
    const int c0 = i << 3;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 f = __bfloat1622float2(h[e]);
      float p0 = f.x * k, p1 = f.y * k;
      if (c0 + 2 * e == tg) p0 -= inv_n;
      if (c0 + 2 * e + 1 == tg) p1 -= inv_n;
      h[e] = __floats2bfloat162_rn(p0, p1);
    }
    grow[i] = u;
  }
}

__global__ void loss_mean_kernel(int n, const float* __restrict__ row_loss, float* __restrict__ loss) {
  fax_grid_dependency_wait();
  __shared__ double red[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) s += (double)row_loss[i];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) red[warp] = s;
  __syncthreads();
  if (warp == 0) {
    double t = lane < nw ? red[lane] : 0.0;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) *loss = (float)(t / (double)n);
  }
}

}  // namespace

fax_status fax_embed_fwd(fax_ctx* ctx, int prec, int B, int T, int d, int vocab, const int32_t* ids,
                         const void* wte, const void* wpe, void* x0) {
  int n = B * T;
  FaxProfScope prof(ctx, KC_EMBED, 0.0, 3.0 * n * d * fax_elem_size(prec));
  if (prec == FAX_PREC_BF16)
    fax_launch(ctx, embed_fwd_kernel<bf16>, dim3(n), dim3(128), 0, n, T, d, vocab, ids, (const bf16*)wte, (const bf16*)wpe, (bf16*)x0);
  else
    fax_launch(ctx, embed_fwd_kernel<float>, dim3(n), dim3(128), 0, n, T, d, vocab, ids, (const float*)wte, (const float*)wpe, (float*)x0);
  return fax_after_launch(ctx);
}

fax_status fax_embed_bwd(fax_ctx* ctx, int prec, int B, int T, int max_seq, int d, int vocab,
                         const int32_t* ids, const void* dx0, float* dwte, float* dwpe, bool accumulate_wpe) {
  int n = B * T;
  FaxProfScope prof(ctx, KC_EMBED, 0.0, (double)n * d * (2.0 * fax_elem_size(prec) + 8.0));
  if (prec == FAX_PREC_BF16) {
    fax_launch(ctx, embed_bwd_wte_kernel<bf16>, dim3(n), dim3(128), 0, n, d, vocab, ids, (const bf16*)dx0, dwte);
    FAX_TRY(fax_after_launch(ctx));
    fax_launch(ctx, embed_bwd_wpe_kernel<bf16>, dim3(max_seq), dim3(128), 0, B, T, max_seq, d, (const bf16*)dx0, dwpe, accumulate_wpe ? 1 : 0);
  } else {
    fax_launch(ctx, embed_bwd_wte_kernel<float>, dim3(n), dim3(128), 0, n, d, vocab, ids, (const float*)dx0, dwte);
    FAX_TRY(fax_after_launch(ctx));
    fax_launch(ctx, embed_bwd_wpe_kernel<float>, dim3(max_seq), dim3(128), 0, B, T, max_seq, d, (const float*)dx0, dwpe, accumulate_wpe ? 1 : 0);
  }
  return fax_after_launch(ctx);
}

fax_status fax_xent(fax_ctx* ctx, int prec, int rows, int vocab, void* logits, int64_t ld,
                    const int32_t* targets, float inv_n, float* row_loss) {
  // read the logits once, write dlogits once
  FaxProfScope prof(ctx, KC_XENT, 0.0, 2.0 * rows * (double)vocab * fax_elem_size(prec));
  const size_t row_bytes = (size_t)vocab * 2;
  if (prec == FAX_PREC_BF16 && vocab % 8 == 0 && ld % 8 == 0 && row_bytes <= 110 * 1024 && fax_aligned(logits, 16)) {
    static bool attr_set = false;
    if (!attr_set) {
      FAX_CUDA_TRY(ctx, cudaFuncSetAttribute(xent_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
      attr_set = true;
    }
    fax_launch(ctx, xent_smem_kernel, dim3(rows), dim3(512), row_bytes, rows, vocab, (bf16*)logits, ld, targets, inv_n, row_loss);
  } else if (prec == FAX_PREC_BF16)
    fax_launch(ctx, xent_kernel<bf16>, dim3(rows), dim3(512), 0, rows, vocab, (bf16*)logits, ld, targets, inv_n, row_loss);
  else
    fax_launch(ctx, xent_kernel<float>, dim3(rows), dim3(512), 0, rows, vocab, (float*)logits, ld, targets, inv_n, row_loss);
  return fax_after_launch(ctx);
}

fax_status fax_loss_mean(fax_ctx* ctx, int n, const float* row_loss, float* loss) {
  fax_launch(ctx, loss_mean_kernel, dim3(1), dim3(1024), 0, n, row_loss, loss);
  return fax_after_launch(ctx);
}
