// Causal multi-head attention on the tcgen05 tensor cores (steps F3 / B5).
//
// Forward: one CTA per (batch, head, 128-query tile).  Q stays in shared memory;
// K and V tiles of 128 keys stream through a double-buffered TMA ring.  One
// elected thread issues S = Q K^T into tensor memory; four warps (one query row
// per thread) run the online softmax on S read from tensor memory, write
// P (bf16) to shared memory in the swizzled K-major operand layout, and the
// elected thread issues O_j = P V_j; the row threads fold O_j into their
// register accumulators.  S_{j+1} is issued before O_j is consumed so the
// tensor core works while the row threads rescale.  log-sum-exp is saved.
//
// All shared-memory operand tiles are 128-byte swizzled: Q, K, P are K-major
// (blocks of 64 columns, 128 rows x 128 B each); V is MN-major (its rows are
// the contraction index).  Every wait is bounded.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int TQ = 128;            // queries per CTA
constexpr int TK = 128;            // keys per tile
constexpr int FWD_THREADS = 160;   // 4 row warps + 1 driver warp

struct AttnFwdParams {
  int B, T, H;
  bf16* o; float* lse;
  float scale_log2;
  int32_t* status;
};

template <int HD> struct FwdCfg {
  static constexpr int TILE_BYTES = TQ * HD * 2;        // Q, K or V tile
  static constexpr int P_BYTES = TQ * TK * 2;
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = TILE_BYTES;              // 2 buffers
  static constexpr int V_OFF = 3 * TILE_BYTES;          // 2 buffers
  static constexpr int P_OFF = 5 * TILE_BYTES;
  static constexpr int BAR_OFF = P_OFF + P_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 128 + 1024;
  static constexpr int TMEM_COLS = 256;                 // S: 128 columns, O: HD columns
};

// Load a 128-row x HD-column tile as HD/64 boxes of 64 columns (16 KB each).
template <int HD>
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int col, int row) {
  mbar_expect_tx(bar, TQ * HD * 2);
#pragma unroll
  for (int i = 0; i < HD / 64; ++i) tma_load_2d(dst + i * 16384, map, bar, col + 64 * i, row);
}

template <int HD>
__global__ void __launch_bounds__(FWD_THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap, const AttnFwdParams p) {
  using C_ = FwdCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  // barriers: 0 Q, 1-2 K[2], 3-4 V[2], 5 S, 6 P, 7 O
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + 64);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + 68);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / TQ;
  const int bh_count = p.B * p.H;
  const int qi = nq - 1 - (int)(blockIdx.x / bh_count);     // heaviest tiles first
  const int bh = blockIdx.x % bh_count;
  const int b = bh / p.H, h = bh % p.H;
  const int d = p.H * HD;
  const int nkv = qi + 1;
  const int row0 = b * p.T;                                 // first token row of this sequence
  const int qcol = h * HD, kcol = d + h * HD, vcol = 2 * d + h * HD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) mbar_init(bar(i), i == 6 ? 4u : 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
  }
  if (warp == 4) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_s = tmem, tmem_o = tmem + 128;

  if (warp == 4) {
    if (lane == 0) {
      const uint32_t q_s = base + C_::Q_OFF, p_s = base + C_::P_OFF;
      auto k_s = [&](int i) { return base + C_::K_OFF + i * C_::TILE_BYTES; };
      auto v_s = [&](int i) { return base + C_::V_OFF + i * C_::TILE_BYTES; };
      const uint32_t idesc_s = idesc_bf16(TK, false, false);
      const uint32_t idesc_o = idesc_bf16(HD, false, true);
      auto mma_s = [&](int buf) {
#pragma unroll
        for (int s = 0; s < HD / 16; ++s) {
          const uint32_t off = (s / 4) * 16384 + (s % 4) * 32;
          tc_mma_bf16(tmem_s, smem_desc(q_s + off, 16, 1024), smem_desc(k_s(buf) + off, 16, 1024), idesc_s, s ? 1u : 0u);
        }
        tc_commit(bar(5));
      };
      load_tile<HD>(q_s, &tmap, bar(0), qcol, row0 + qi * TQ);
      load_tile<HD>(k_s(0), &tmap, bar(1), kcol, row0);
      load_tile<HD>(v_s(0), &tmap, bar(3), vcol, row0);
      if (nkv > 1) {
        load_tile<HD>(k_s(1), &tmap, bar(2), kcol, row0 + TK);
        load_tile<HD>(v_s(1), &tmap, bar(4), vcol, row0 + TK);
      }
      bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 201) && mbar_wait(bar(1), 0, abort_flag, p.status, 202);
      if (ok) { tc_fence_after(); mma_s(0); }
      for (int j = 0; j < nkv && ok; ++j) {
        const int buf = j & 1;
        const uint32_t ring_phase = (uint32_t)((j >> 1) & 1);
        if (!mbar_wait(bar(6), j & 1, abort_flag, p.status, 203)) { ok = false; break; }       // P_j ready
        if (!mbar_wait(bar(3 + buf), ring_phase, abort_flag, p.status, 204)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < TK / 16; ++s) {
          const uint64_t ad = smem_desc(p_s + (s / 4) * 16384 + (s % 4) * 32, 16, 1024);
          const uint64_t bd = smem_desc(v_s(buf) + s * 2048, 16384, 1024);
          tc_mma_bf16(tmem_o, ad, bd, idesc_o, s ? 1u : 0u);
        }
        tc_commit(bar(7));
        if (j + 1 < nkv) {
          if (!mbar_wait(bar(1 + (buf ^ 1)), (uint32_t)(((j + 1) >> 1) & 1), abort_flag, p.status, 205)) { ok = false; break; }
          tc_fence_after();
          mma_s(buf ^ 1);
        }
        if (j + 2 < nkv) {
          // K[buf] was consumed by S_j (complete before P_j was signalled); V[buf] is free once O_j is done
          load_tile<HD>(k_s(buf), &tmap, bar(1 + buf), kcol, row0 + (j + 2) * TK);
          if (!mbar_wait(bar(7), j & 1, abort_flag, p.status, 206)) { ok = false; break; }
          load_tile<HD>(v_s(buf), &tmap, bar(3 + buf), vcol, row0 + (j + 2) * TK);
        }
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else {
    // ---- row threads: online softmax, one query row each ----
    const int r = 32 * warp + lane;
    const uint32_t lane_base = (uint32_t)(32 * warp) << 16;
    uint8_t* p_row = gbase + C_::P_OFF + r * 128;
    float m = -INFINITY, l = 0.f;
    float o[HD];
#pragma unroll
    for (int c = 0; c < HD; ++c) o[c] = 0.f;
    bool ok = true;
    for (int j = 0; j < nkv; ++j) {
      if (!mbar_wait(bar(5), j & 1, abort_flag, p.status, 207)) { ok = false; break; }
      tc_fence_after();
      const bool diag = (j == qi);
      float mx = -INFINITY;
#pragma unroll 1
      for (int c0 = 0; c0 < TK; c0 += 32) {
        uint32_t v[32];
        tc_ld32(tmem_s + lane_base + c0, v);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          float s = __uint_as_float(v[c]);
          if (diag && (c0 + c > r)) s = -INFINITY;
          mx = fmaxf(mx, s);
        }
      }
      const float m_new = fmaxf(m, mx * p.scale_log2);
      const float corr = exp2f(m - m_new);
      float rowsum = 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < TK; c0 += 32) {
        uint32_t v[32];
        tc_ld32(tmem_s + lane_base + c0, v);
        tc_wait_ld();
        uint32_t packed[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float p0 = exp2f(__uint_as_float(v[c]) * p.scale_log2 - m_new);
          float p1 = exp2f(__uint_as_float(v[c + 1]) * p.scale_log2 - m_new);
          if (diag) { if (c0 + c > r) p0 = 0.f; if (c0 + c + 1 > r) p1 = 0.f; }
          rowsum += p0 + p1;
          __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          packed[c >> 1] = *reinterpret_cast<uint32_t*>(&h2);
        }
        uint8_t* blk = p_row + (c0 >> 6) * 16384;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int chunk = ((c0 & 63) >> 3) + k;
          *reinterpret_cast<uint4*>(blk + ((chunk ^ (r & 7)) << 4)) =
              make_uint4(packed[4 * k], packed[4 * k + 1], packed[4 * k + 2], packed[4 * k + 3]);
        }
      }
      l = l * corr + rowsum;
      m = m_new;
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(6));
      if (!mbar_wait(bar(7), j & 1, abort_flag, p.status, 208)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t v[32];
        tc_ld32(tmem_o + lane_base + c0, v);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) o[c0 + c] = o[c0 + c] * corr + __uint_as_float(v[c]);
      }
      tc_fence_before();
    }
    if (ok) {
      const float inv = 1.f / l;
      const long long tok = (long long)row0 + qi * TQ + r;
      bf16* orow = p.o + tok * d + h * HD;
#pragma unroll
      for (int c = 0; c < HD; c += 8) {
        uint4 u;
        __nv_bfloat162* hh = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) hh[e] = __floats2bfloat162_rn(o[c + 2 * e] * inv, o[c + 2 * e + 1] * inv);
        *reinterpret_cast<uint4*>(orow + c) = u;
      }
      p.lse[((long long)b * p.H + h) * p.T + qi * TQ + r] = (m + log2f(l)) * 0.6931471805599453f;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

template <int HD>
fax_status launch_fwd(fax_ctx* ctx, int B, int T, int H, const void* qkv, void* o, float* lse) {
  CUtensorMap map;
  const uint64_t d = (uint64_t)H * HD;
  if (!make_map(ctx, &map, qkv, 3 * d, (uint64_t)B * T, 3 * d, 64, 128)) return FAX_ERR_INVALID_ARG;
  AttnFwdParams p;
  p.B = B; p.T = T; p.H = H; p.o = (bf16*)o; p.lse = lse;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  p.status = ctx->dev_status;
  static bool attr_set = false;
  if (!attr_set) {
    FAX_CUDA_TRY(ctx, cudaFuncSetAttribute(attn_fwd_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           FwdCfg<HD>::SMEM_BYTES));
    attr_set = true;
  }
  const int grid = B * H * (T / TQ);
  attn_fwd_tc_kernel<HD><<<grid, FWD_THREADS, FwdCfg<HD>::SMEM_BYTES, ctx->stream>>>(map, p);
  return fax_after_launch(ctx);
}

}  // namespace

bool fax_attention_tc_supported(int B, int T, int H, int hd) {
  return (hd == 64 || hd == 128) && T % 128 == 0 && B > 0 && H > 0;
}

fax_status fax_attention_fwd_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, void* o, float* lse) {
  if (!fax_attention_tc_supported(B, T, H, hd) || !fax_aligned(qkv, 16) || !fax_aligned(o, 16))
    return FAX_ERR_UNSUPPORTED_SHAPE;
  return hd == 64 ? launch_fwd<64>(ctx, B, T, H, qkv, o, lse) : launch_fwd<128>(ctx, B, T, H, qkv, o, lse);
}
