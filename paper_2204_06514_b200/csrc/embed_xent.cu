// Embedding lookup / scatter and softmax cross-entropy of the LM step
// (steps LM-E, LM-H loss part, LM-B).  All HBM-bound.
#include "tc_common.cuh"

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

// bf16 rows of which two fit in shared memory: a row is read from HBM once.  Pass 1 takes the
// maximum; pass 2 replaces each logit by exp(logit - max) (bf16) while summing the unrounded
// exponentials; pass 3 writes (e / sum - onehot) * inv_n.  A persistent kernel (one block per SM)
// that keeps HBM busy while it computes: an extra warp moves rows with bulk
// asynchronous copies, global -> shared into one of two row buffers ahead of the compute warps and
// shared -> global behind them, so the load of row i+1 and the store of row i-1 run under the
// passes over row i.  Hand-offs are mbarriers (full[b]: the row has landed; done[b]: all 16
// compute warps have finished it); every wait is bounded.
constexpr int XS_COMPUTE_THREADS = 512;
constexpr int XS_THREADS = XS_COMPUTE_THREADS + 32;

__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store_row(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(XS_THREADS, 1)
xent_stream_kernel(int rows, int vocab, bf16* __restrict__ logits, int64_t ld, const int32_t* __restrict__ targets,
                   float inv_n, float* __restrict__ row_loss, int32_t* status) {
  using namespace tc;
  extern __shared__ uint4 xs_raw[];                  // [2][vocab / 8] vectors, then barriers
  __shared__ float red[32];
  __shared__ uint64_t bars_mem[4];
  __shared__ int abort_mem;
  const uint32_t row_bytes = (uint32_t)vocab * 2u;
  const int nvec = vocab >> 3;
  const uint32_t bars = smem_u32(bars_mem);
  auto full_bar = [&](int b) { return bars + 8u * b; };
  auto done_bar = [&](int b) { return bars + 8u * (2 + b); };
  volatile int* abort_flag = &abort_mem;
  if (threadIdx.x == 0) {
    mbar_init(full_bar(0), 1); mbar_init(full_bar(1), 1);
    mbar_init(done_bar(0), XS_COMPUTE_THREADS / 32); mbar_init(done_bar(1), XS_COMPUTE_THREADS / 32);
    abort_mem = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  fax_grid_dependency_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_mine = (rows - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;      // rows blockIdx.x + k * gridDim.x

  if (warp == XS_COMPUTE_THREADS / 32) {
    // ---------------- copy warp ----------------
    if (lane == 0) {
      bool ok = true;
      for (int k = 0; k < n_mine && k < 2; ++k) {
        mbar_expect_tx(full_bar(k), row_bytes);
        bulk_load_row(smem_u32(xs_raw) + (uint32_t)k * row_bytes, logits + (size_t)(blockIdx.x + k * gridDim.x) * ld,
                      row_bytes, full_bar(k));
      }
      for (int k = 0; k < n_mine && ok; ++k) {
        const int b = k & 1;
        if (!mbar_wait(done_bar(b), (uint32_t)(k >> 1) & 1u, abort_flag, status, 401)) { ok = false; break; }
        const size_t r = (size_t)blockIdx.x + (size_t)k * gridDim.x;
        bulk_store_row(logits + r * ld, smem_u32(xs_raw) + (uint32_t)b * row_bytes, row_bytes);
        bulk_commit_group();
        if (k + 2 < n_mine) {
          bulk_wait_read_all();                     // the store has read the buffer: it may be refilled
          mbar_expect_tx(full_bar(b), row_bytes);
          bulk_load_row(smem_u32(xs_raw) + (uint32_t)b * row_bytes, logits + (r + 2 * (size_t)gridDim.x) * ld, row_bytes,
                        full_bar(b));
        }
      }
      bulk_wait_all();                              // all stores have landed before the block exits
    }
  } else {
    // ---------------- compute warps ----------------
    bool ok = true;
    for (int k = 0; k < n_mine && ok; ++k) {
      const int b = k & 1;
      const int r = (int)blockIdx.x + k * (int)gridDim.x;
      uint4* xrow = xs_raw + (size_t)b * nvec;
      if (!mbar_wait_warp(full_bar(b), (uint32_t)(k >> 1) & 1u, abort_flag, status, 402)) { ok = false; break; }
      const int tg = targets[r];
      // maximum in packed bf16 pairs (exact: the values are bf16)
      __nv_bfloat162 m2 = __float2bfloat162_rn(-INFINITY);
      for (int i = threadIdx.x; i < nvec; i += XS_COMPUTE_THREADS) {
        const uint4 u = xrow[i];
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
        m2 = __hmax2(__hmax2(m2, h[0]), __hmax2(h[1], __hmax2(h[2], h[3])));
      }
      float mx = fmaxf(__low2float(m2), __high2float(m2));
      float lt = 0.f;
      if (threadIdx.x == 0 && tg >= 0 && tg < vocab) lt = __bfloat162float(reinterpret_cast<const bf16*>(xrow)[tg]);
      // block-wide reductions among the compute warps only (named barrier 1)
      auto reduce = [&](float v, bool is_max) {
        v = is_max ? warp_max(v) : warp_sum(v);
        named_barrier_sync(1, XS_COMPUTE_THREADS);
        if (lane == 0) red[warp] = v;
        named_barrier_sync(1, XS_COMPUTE_THREADS);
        float t = lane < XS_COMPUTE_THREADS / 32 ? red[lane] : (is_max ? -INFINITY : 0.f);
        return is_max ? warp_max(t) : warp_sum(t);
      };
      mx = reduce(mx, true);
      float s = 0.f;
      for (int i = threadIdx.x; i < nvec; i += XS_COMPUTE_THREADS) {
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
      s = reduce(s, false);
      if (threadIdx.x == 0) {
        const float lse = mx + logf(s);
        row_loss[r] = (tg >= 0 && tg < vocab) ? lse - lt : 0.f;
      }
      const float kk = inv_n / s;
      const int tgv = (tg >= 0 && tg < vocab) ? (tg >> 3) : -1;       // the one vector that holds the target column
      for (int i = threadIdx.x; i < nvec; i += XS_COMPUTE_THREADS) {
        uint4 u = xrow[i];
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
        if (i != tgv) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            h[e] = __floats2bfloat162_rn(f.x * kk, f.y * kk);
          }
        } else {
          const int c0 = i << 3;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            float p0 = f.x * kk, p1 = f.y * kk;
            if (c0 + 2 * e == tg) p0 -= inv_n;
            if (c0 + 2 * e + 1 == tg) p1 -= inv_n;
            h[e] = __floats2bfloat162_rn(p0, p1);
          }
        }
        xrow[i] = u;
      }
      fence_proxy_async();                          // this thread's shared-memory writes, for the bulk store
      __syncwarp();
      if (lane == 0) mbar_arrive(done_bar(b));
    }
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
  const bool vec_ok = prec == FAX_PREC_BF16 && vocab % 8 == 0 && ld % 8 == 0 && fax_aligned(logits, 16);
  if (vec_ok && 2 * row_bytes <= 220 * 1024) {
    // two rows fit: persistent kernel, rows streamed through shared memory by bulk copies
    static bool attr_set[FAX_MAX_DEVICES] = {};
    FAX_TRY(fax_opt_in_shared_memory(ctx, xent_stream_kernel, 220 * 1024, attr_set));
    const int grid = rows < ctx->sm_count ? rows : ctx->sm_count;
    fax_launch(ctx, xent_stream_kernel, dim3(grid), dim3(XS_THREADS), 2 * row_bytes, rows, vocab, (bf16*)logits,
               ld, targets, inv_n, row_loss, ctx->dev_status);
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
