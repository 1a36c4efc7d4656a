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
constexpr int FWD_THREADS = 192;   // 4 row warps + MMA warp + TMA warp

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
  static constexpr int SMEM_BYTES = BAR_OFF + 256 + 1024;
  static constexpr int TMEM_COLS = 512;                 // S0 [0,128), S1 [128,256), O [256, 256+HD)
};

// Load a 128-row x HD-column tile as HD/64 boxes of 64 columns (16 KB each).
template <int HD>
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int col, int row) {
  mbar_expect_tx(bar, TQ * HD * 2);
#pragma unroll
  for (int i = 0; i < HD / 64; ++i) tma_load_2d(dst + i * 16384, map, bar, col + 64 * i, row);
}

// Forward.  S for tile j+1 and j+2 is issued ahead, so the row threads always find
// their next scores ready while the tensor core runs P V of the tile before; O
// accumulates in tensor memory and is rescaled only when a row maximum has grown by
// more than 2^8 since the value the accumulator is expressed in (the decision is
// taken per warp, because tensor-memory loads and stores are warp-collective).
template <int HD>
__global__ void __launch_bounds__(FWD_THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap, const AttnFwdParams p) {
  using C_ = FwdCfg<HD>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  // barriers: 0 Q | 1,2 K full | 3,4 K empty | 5,6 V full | 7,8 V empty | 9,10 S full | 11 P ready | 12 O done
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + 128);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + 132);

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
    for (int i = 0; i < 13; ++i) mbar_init(bar(i), i == 11 ? 4u : 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
  }
  if (warp == 4) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 256;
  const uint32_t q_s = base + C_::Q_OFF, p_s = base + C_::P_OFF;
  auto k_s = [&](int i) { return base + C_::K_OFF + i * C_::TILE_BYTES; };
  auto v_s = [&](int i) { return base + C_::V_OFF + i * C_::TILE_BYTES; };

  if (warp == 5) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      load_tile<HD>(q_s, &tmap, bar(0), qcol, row0 + qi * TQ);
      bool ok = true;
      for (int j = 0; j < nkv && ok; ++j) {
        const int s = j & 1;
        const uint32_t ph = (uint32_t)((j >> 1) & 1);
        if (!mbar_wait(bar(3 + s), ph ^ 1u, abort_flag, p.status, 201)) { ok = false; break; }
        load_tile<HD>(k_s(s), &tmap, bar(1 + s), kcol, row0 + j * TK);
        if (!mbar_wait(bar(7 + s), ph ^ 1u, abort_flag, p.status, 202)) { ok = false; break; }
        load_tile<HD>(v_s(s), &tmap, bar(5 + s), vcol, row0 + j * TK);
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else if (warp == 4) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(TK, false, false);
      const uint32_t idesc_o = idesc_bf16(HD, false, true);
      bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 203);
      auto issue_s = [&](int j) -> bool {
        const int s = j & 1;
        if (!mbar_wait(bar(1 + s), (uint32_t)((j >> 1) & 1), abort_flag, p.status, 204)) return false;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
          tc_mma_bf16(tmem + (uint32_t)(s * 128), smem_desc(q_s + off, 16, 1024), smem_desc(k_s(s) + off, 16, 1024),
                      idesc_s, k ? 1u : 0u);
        }
        tc_commit(bar(3 + s));      // K buffer free
        tc_commit(bar(9 + s));      // S ready
        return true;
      };
      if (ok) ok = issue_s(0);
      if (ok && nkv > 1) ok = issue_s(1);
      for (int j = 0; j < nkv && ok; ++j) {
        const int s = j & 1;
        if (!mbar_wait(bar(11), (uint32_t)(j & 1), abort_flag, p.status, 205)) { ok = false; break; }
        if (!mbar_wait(bar(5 + s), (uint32_t)((j >> 1) & 1), abort_flag, p.status, 206)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < TK / 16; ++k) {
          const uint64_t ad = smem_desc(p_s + (k / 4) * 16384 + (k % 4) * 32, 16, 1024);
          const uint64_t bd = smem_desc(v_s(s) + k * 2048, 16384, 1024);
          tc_mma_bf16(tmem_o, ad, bd, idesc_o, (j | k) ? 1u : 0u);
        }
        tc_commit(bar(7 + s));      // V buffer free
        tc_commit(bar(12));         // O_j accumulated, P buffer free
        if (j + 2 < nkv) ok = issue_s(j + 2);   // S buffer s was consumed before P_j was signalled
      }
    }
  } else {
    // ---- row threads: online softmax, one query row each ----
    const int r = 32 * warp + lane;
    const uint32_t lane_base = (uint32_t)(32 * warp) << 16;
    uint8_t* p_row = gbase + C_::P_OFF + r * 128;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nkv; ++j) {
      const int sb = j & 1;
      if (!mbar_wait_warp(bar(9 + sb), (uint32_t)((j >> 1) & 1), abort_flag, p.status, 207)) { ok = false; break; }
      tc_fence_after();
      uint32_t sv[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tc_ld32(tmem + lane_base + (uint32_t)(sb * 128 + 32 * c), sv[c]);
      tc_wait_ld();
      const bool diag = (j == qi);
      if (diag) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (32 * c + e > r) sv[c][e] = 0xff800000u;      // -inf
      }
      // three-input max, four independent chains (the two-input form is the slowest part of the tile)
      float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 32; e += 2)
          mxa[(e >> 1) & 3] = max3(mxa[(e >> 1) & 3], __uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1]));
      const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
      const float m_new = fmaxf(m_used, mx * p.scale_log2);
      bool odone_waited = false;
      if (__any_sync(0xffffffffu, m_new > m_used + 8.0f)) {
        if (j > 0) {
          if (!mbar_wait_warp(bar(12), (uint32_t)((j - 1) & 1), abort_flag, p.status, 208)) { ok = false; break; }
          odone_waited = true;
          tc_fence_after();
          const float factor = ex2_approx(m_used - m_new);
          l *= factor;
#pragma unroll 1
          for (int c0 = 0; c0 < HD; c0 += 32) {
            uint32_t ov[32];
            tc_ld32(tmem_o + lane_base + c0, ov);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * factor);
            tc_st32(tmem_o + lane_base + c0, ov);
          }
          tc_wait_st();
        }
        m_used = m_new;
      }
      float rowsum = 0.f;
      uint32_t packed[64];
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float p0 = ex2_approx(__uint_as_float(sv[c][e]) * p.scale_log2 - m_used);
          const float p1 = ex2_approx(__uint_as_float(sv[c][e + 1]) * p.scale_log2 - m_used);
          rowsum += p0 + p1;
          __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          packed[16 * c + (e >> 1)] = *reinterpret_cast<uint32_t*>(&h2);
        }
      l += rowsum;
      if (j > 0 && !odone_waited) {      // P buffer is free once P V of the previous tile is complete
        if (!mbar_wait_warp(bar(12), (uint32_t)((j - 1) & 1), abort_flag, p.status, 209)) { ok = false; break; }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint8_t* blk = p_row + (c >> 1) * 16384;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int chunk = ((c & 1) << 2) + k;
          *reinterpret_cast<uint4*>(blk + ((chunk ^ (r & 7)) << 4)) =
              make_uint4(packed[16 * c + 4 * k], packed[16 * c + 4 * k + 1], packed[16 * c + 4 * k + 2],
                         packed[16 * c + 4 * k + 3]);
        }
      }
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(11));
    }
    if (ok && mbar_wait_warp(bar(12), (uint32_t)((nkv - 1) & 1), abort_flag, p.status, 210)) {
      tc_fence_after();
      const float inv = 1.f / l;
      const long long tok = (long long)row0 + qi * TQ + r;
      bf16* orow = p.o + tok * d + h * HD;
#pragma unroll 1
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t ov[32];
        tc_ld32(tmem_o + lane_base + c0, ov);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 u;
          __nv_bfloat162* hh = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e)
            hh[e] = __floats2bfloat162_rn(__uint_as_float(ov[c + 2 * e]) * inv, __uint_as_float(ov[c + 2 * e + 1]) * inv);
          *reinterpret_cast<uint4*>(orow + c0 + c) = u;
        }
      }
      p.lse[((long long)b * p.H + h) * p.T + qi * TQ + r] = (m_used + log2f(l)) * 0.6931471805599453f;
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


// ---------------------------------------------------------------------------
// Backward.  One CTA per (batch, head, 128-key tile j); it keeps K_j and V_j in
// shared memory and walks the query tiles i >= j.  Per step the elected thread
// issues S = Q_i K_j^T and dP = dO_i V_j^T; the row threads (one query row
// each) form P = exp(S/sqrt(hd) - LSE) and dS = P * (dP - D) and write both as
// bf16 operand tiles; the elected thread then issues dV_j += P^T dO_i and
// dK_j += dS^T Q_i (accumulating in tensor memory over the whole walk) and
// dQ_i = dS K_j, which the row threads stage in shared memory and one thread adds
// into a float32 dQ buffer with a bulk tensor reduction (per-thread vector reductions
// from registers into global memory were measured a third slower).  Eight row warps:
// nothing in the backward pass reduces along a row, so two warps share each quarter
// of the tensor-memory lanes and take one half of the columns each.  The P / dS / Q / dO / K tiles are each used both as a K-major and as
// an MN-major operand: the bytes are the same, only the descriptor differs.
// Tensor memory: [0,128) S, [128,256) dP then dQ, [256,256+HD) dV, [384,384+HD) dK.  P is signalled
// before dS so that dV runs while the row threads still work on dS; dK is issued before dQ so the Q
// tile can be reloaded while dQ is computed and read out.
// ---------------------------------------------------------------------------
constexpr int BWD_THREADS = 320;   // 8 row warps (4 lane quarters x 2 column halves) + MMA warp + TMA warp

struct AttnBwdParams {
  int B, T, H;
  const float* lse; const float* Dv;
  float* dq_acc; bf16* dqkv;
  float scale, scale_log2;
  int32_t* status;
};

template <int HD> struct BwdCfg {
  static constexpr int NQ = (HD == 64) ? 2 : 1;          // Q / dO stages (shared memory allows 2 only at hd 64)
  static constexpr int TILE_BYTES = 128 * HD * 2;
  static constexpr int PS_BYTES = 128 * 128 * 2;
  static constexpr int K_OFF = 0, V_OFF = TILE_BYTES;
  static constexpr int Q_OFF = 2 * TILE_BYTES, DO_OFF = Q_OFF + NQ * TILE_BYTES;
  static constexpr int P_OFF = DO_OFF + NQ * TILE_BYTES, DS_OFF = P_OFF + PS_BYTES;
  static constexpr int BAR_OFF = DS_OFF + PS_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 256 + 1024;
  static constexpr int TMEM_COLS = 512;                  // S [0,128) | dP then dQ [128,256) | dV [256,..) | dK [384,..)
};

template <int HD>
__global__ void __launch_bounds__(BWD_THREADS, 1)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const __grid_constant__ CUtensorMap tmap_do,
                   const __grid_constant__ CUtensorMap tmap_dq, const AttnBwdParams p) {
  using C_ = BwdCfg<HD>;
  constexpr int NQ = C_::NQ;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  // barriers: 0 K/V full | 1,2 Q full | 3,4 dO full | 5,6 Q free | 7,8 dO free | 9 S full | 10 dP full |
  //           11 P ready (8) | 12 dS ready (8) | 13 dQ full | 14 dQ read out (8)
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + 128);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + 132);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / 128;
  const int bh_count = p.B * p.H;
  const int kj = (int)(blockIdx.x / bh_count);             // heaviest key tiles (small j) first
  const int bh = blockIdx.x % bh_count;
  const int b = bh / p.H, h = bh % p.H;
  const int d = p.H * HD;
  const int row0 = b * p.T;
  const int qcol = h * HD, kcol = d + h * HD, vcol = 2 * d + h * HD;
  const int nsteps = nq - kj;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 15; ++i) mbar_init(bar(i), (i == 11 || i == 12 || i == 14) ? 8u : 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_do) : "memory");
  }
  if (warp == 8) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s = tmem, tm_dp = tmem + 128, tm_dv = tmem + 256, tm_dk = tmem + 384;
  const uint32_t k_s = base + C_::K_OFF, v_s = base + C_::V_OFF;
  const uint32_t p_s = base + C_::P_OFF, ds_s = base + C_::DS_OFF;
  auto q_s = [&](int i) { return base + C_::Q_OFF + i * C_::TILE_BYTES; };
  auto do_s = [&](int i) { return base + C_::DO_OFF + i * C_::TILE_BYTES; };

  if (warp == 9) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      mbar_expect_tx(bar(0), 2 * C_::TILE_BYTES);
#pragma unroll
      for (int i = 0; i < HD / 64; ++i) {
        tma_load_2d(k_s + i * 16384, &tmap_qkv, bar(0), kcol + 64 * i, row0 + kj * 128);
        tma_load_2d(v_s + i * 16384, &tmap_qkv, bar(0), vcol + 64 * i, row0 + kj * 128);
      }
      bool ok = true;
      for (int it = 0; it < nsteps && ok; ++it) {
        const int st = it % NQ;
        const uint32_t ph = (uint32_t)((it / NQ) & 1);
        const int qrow = row0 + (kj + it) * 128;
        if (!mbar_wait(bar(5 + st), ph ^ 1u, abort_flag, p.status, 301)) { ok = false; break; }
        mbar_expect_tx(bar(1 + st), C_::TILE_BYTES);
#pragma unroll
        for (int i = 0; i < HD / 64; ++i) tma_load_2d(q_s(st) + i * 16384, &tmap_qkv, bar(1 + st), qcol + 64 * i, qrow);
        if (!mbar_wait(bar(7 + st), ph ^ 1u, abort_flag, p.status, 302)) { ok = false; break; }
        mbar_expect_tx(bar(3 + st), C_::TILE_BYTES);
#pragma unroll
        for (int i = 0; i < HD / 64; ++i) tma_load_2d(do_s(st) + i * 16384, &tmap_do, bar(3 + st), qcol + 64 * i, qrow);
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, false, false);
      const uint32_t idesc_kv = idesc_bf16(HD, true, true);
      const uint32_t idesc_q = idesc_bf16(HD, false, true);
      auto koff = [](int s) { return (uint32_t)((s / 4) * 16384 + (s % 4) * 32); };   // K-major k-step
      bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 303);
      for (int it = 0; it < nsteps && ok; ++it) {
        const int st = it % NQ;
        const uint32_t sph = (uint32_t)((it / NQ) & 1), ph = (uint32_t)(it & 1);
        // S = Q K^T  (the S columns were read out before P of the previous step was signalled)
        if (!mbar_wait(bar(1 + st), sph, abort_flag, p.status, 304)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < HD / 16; ++s)
          tc_mma_bf16(tm_s, smem_desc(q_s(st) + koff(s), 16, 1024), smem_desc(k_s + koff(s), 16, 1024), idesc_s, s ? 1u : 0u);
        tc_commit(bar(9));
        // dP = dO V^T  (its columns double as dQ: wait until the previous dQ has been read out)
        if (!mbar_wait(bar(3 + st), sph, abort_flag, p.status, 305)) { ok = false; break; }
        if (it > 0 && !mbar_wait(bar(14), ph ^ 1u, abort_flag, p.status, 306)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < HD / 16; ++s)
          tc_mma_bf16(tm_dp, smem_desc(do_s(st) + koff(s), 16, 1024), smem_desc(v_s + koff(s), 16, 1024), idesc_s, s ? 1u : 0u);
        tc_commit(bar(10));
        // dV += P^T dO
        if (!mbar_wait(bar(11), ph, abort_flag, p.status, 307)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 8; ++s)
          tc_mma_bf16(tm_dv, smem_desc(p_s + s * 2048, 16384, 1024), smem_desc(do_s(st) + s * 2048, 16384, 1024),
                      idesc_kv, (it | s) ? 1u : 0u);
        tc_commit(bar(7 + st));          // dO stage free
        // dK += dS^T Q, then dQ = dS K
        if (!mbar_wait(bar(12), ph, abort_flag, p.status, 308)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 8; ++s)
          tc_mma_bf16(tm_dk, smem_desc(ds_s + s * 2048, 16384, 1024), smem_desc(q_s(st) + s * 2048, 16384, 1024),
                      idesc_kv, (it | s) ? 1u : 0u);
        tc_commit(bar(5 + st));          // Q stage free
#pragma unroll
        for (int s = 0; s < 8; ++s)
          tc_mma_bf16(tm_dp, smem_desc(ds_s + koff(s), 16, 1024), smem_desc(k_s + s * 2048, 16384, 1024),
                      idesc_q, s ? 1u : 0u);
        tc_commit(bar(13));              // dQ ready; also: every MMA issued so far is complete
      }
    }
  } else {
    // Row threads: warp w serves query rows 32*(w&3).. (its quarter of the tensor-memory lanes) and
    // the column half w>>2 of every tile: nothing here reduces along a row, so the halves are
    // independent and each scheduler has two warps to interleave.
    const int hc = warp >> 2;
    const int r = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    uint8_t* p_row = gbase + C_::P_OFF + r * 128;
    uint8_t* ds_row = gbase + C_::DS_OFF + r * 128;
    bool ok = true;
    for (int it = 0; it < nsteps; ++it) {
      const uint32_t ph = (uint32_t)(it & 1);
      const int qi = kj + it;
      const long long stat = ((long long)b * p.H + h) * p.T + qi * 128 + r;
      const float lse2 = p.lse[stat] * 1.4426950408889634f;
      const float Dr = p.Dv[stat];
      const bool diag = (it == 0);
      uint32_t pp[32];
      // P = exp(S / sqrt(hd) - LSE): the P tile is also needed (as bf16) by dS below
      if (!mbar_wait_warp(bar(9), ph, abort_flag, p.status, 309)) { ok = false; break; }
      tc_fence_after();
      {
        uint32_t sv[2][32];
#pragma unroll
        for (int c = 0; c < 2; ++c) tc_ld32(tm_s + lane_base + 64 * hc + 32 * c, sv[c]);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float p0 = ex2_approx(__uint_as_float(sv[c][e]) * p.scale_log2 - lse2);
            float p1 = ex2_approx(__uint_as_float(sv[c][e + 1]) * p.scale_log2 - lse2);
            if (diag) { if (64 * hc + 32 * c + e > r) p0 = 0.f; if (64 * hc + 32 * c + e + 1 > r) p1 = 0.f; }
            __nv_bfloat162 hp = __floats2bfloat162_rn(p0, p1);
            pp[16 * c + (e >> 1)] = *reinterpret_cast<uint32_t*>(&hp);
          }
      }
      if (it > 0) {
        // the P / dS buffers staged the previous dQ tile: its bulk reduction must have read them
        if (threadIdx.x == 0) bulk_wait_read_all();
        named_barrier_sync(1, 256);
      }
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int off = hc * 16384 + ((((c << 2) + k) ^ (r & 7)) << 4);
          *reinterpret_cast<uint4*>(p_row + off) =
              make_uint4(pp[16 * c + 4 * k], pp[16 * c + 4 * k + 1], pp[16 * c + 4 * k + 2], pp[16 * c + 4 * k + 3]);
        }
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(11));
      // dS = P * (dP - D), from the bf16 P that the products use
      if (!mbar_wait_warp(bar(10), ph, abort_flag, p.status, 310)) { ok = false; break; }
      tc_fence_after();
      {
        uint32_t dv[2][32];
        tc_ld32(tm_dp + lane_base + 64 * hc, dv[0]);
        tc_ld32(tm_dp + lane_base + 64 * hc + 32, dv[1]);
        tc_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int c = cc;
          uint32_t dd[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 pf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pp[16 * c + (e >> 1)]));
            __nv_bfloat162 hd2 = __floats2bfloat162_rn(pf.x * (__uint_as_float(dv[cc][e]) - Dr),
                                                       pf.y * (__uint_as_float(dv[cc][e + 1]) - Dr));
            dd[e >> 1] = *reinterpret_cast<uint32_t*>(&hd2);
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int off = hc * 16384 + ((((c << 2) + k) ^ (r & 7)) << 4);
            *reinterpret_cast<uint4*>(ds_row + off) = make_uint4(dd[4 * k], dd[4 * k + 1], dd[4 * k + 2], dd[4 * k + 3]);
          }
        }
      }
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(12));
      // dQ tile of this step: tensor memory -> shared memory (the P / dS buffers, free by now, as
      // 32-column boxes in the 128-byte-swizzled layout) -> one bulk add-reduction into the
      // float32 dQ accumulator in global memory
      if (!mbar_wait_warp(bar(13), ph, abort_flag, p.status, 311)) { ok = false; break; }
      tc_fence_after();
      {
        // this warp's half of the head's columns: HD/2 = 64 (two boxes) or 32 (one box)
        constexpr int NB = HD / 64;
        const int c0 = hc * (HD / 2);
        uint32_t v[NB][32];
#pragma unroll
        for (int cc = 0; cc < NB; ++cc) tc_ld32(tm_dp + lane_base + c0 + 32 * cc, v[cc]);
        tc_wait_ld();
#pragma unroll
        for (int cc = 0; cc < NB; ++cc) {
          uint8_t* box = gbase + C_::P_OFF + ((c0 >> 5) + cc) * 16384 + r * 128;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            *reinterpret_cast<uint4*>(box + ((k ^ (r & 7)) << 4)) =
                make_uint4(v[cc][4 * k], v[cc][4 * k + 1], v[cc][4 * k + 2], v[cc][4 * k + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(14));
      fence_proxy_async();
      named_barrier_sync(1, 256);
      if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < HD / 32; ++i)
          tma_reduce_add_2d(&tmap_dq, base + C_::P_OFF + i * 16384, h * HD + 32 * i, (int)(row0 + qi * 128));
        bulk_commit_group();
      }
    }
    if (threadIdx.x == 0) bulk_wait_all();
    if (ok) {
      // the last wait on the dQ barrier covered every MMA: dV and dK of this key tile are final
      const long long tok = (long long)row0 + kj * 128 + r;
      bf16* dk_row = p.dqkv + tok * 3 * d + d + h * HD;
      bf16* dv_row = p.dqkv + tok * 3 * d + 2 * d + h * HD;
#pragma unroll 1
      for (int c0 = hc * (HD / 2); c0 < (hc + 1) * (HD / 2); c0 += 32) {
        uint32_t kv[32], vv[32];
        tc_ld32(tm_dk + lane_base + c0, kv);
        tc_ld32(tm_dv + lane_base + c0, vv);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 uk, uv;
          __nv_bfloat162* hk = reinterpret_cast<__nv_bfloat162*>(&uk);
          __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&uv);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            hk[e] = __floats2bfloat162_rn(__uint_as_float(kv[c + 2 * e]) * p.scale, __uint_as_float(kv[c + 2 * e + 1]) * p.scale);
            hv[e] = __floats2bfloat162_rn(__uint_as_float(vv[c + 2 * e]), __uint_as_float(vv[c + 2 * e + 1]));
          }
          *reinterpret_cast<uint4*>(dk_row + c0 + c) = uk;
          *reinterpret_cast<uint4*>(dv_row + c0 + c) = uv;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

// D[b,h,t] = sum_c dO[t,c] * O[t,c] over the head's columns; one warp per (token, head)
__global__ void attn_rowdot_bf16_kernel(int n_tok, int T, int H, int hd, const bf16* __restrict__ d_o,
                                        const bf16* __restrict__ o, float* __restrict__ Dv) {
  const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (gw >= n_tok * H) return;
  const int tok = gw / H, h = gw % H;
  const long long off = (long long)tok * H * hd + h * hd;
  float s = 0.f;
  for (int c = lane * 2; c < hd; c += 64) {
    float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(d_o + off + c));
    float2 bq = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(o + off + c));
    s += a.x * bq.x + a.y * bq.y;
  }
  s = warp_sum(s);
  if (lane == 0) Dv[((long long)(tok / T) * H + h) * T + (tok % T)] = s;
}

// dqkv[n, 0:d] = bf16(dq_acc[n, :] * scale)
__global__ void attn_dq_convert_kernel(long long n_tok, int d, const float* __restrict__ dq_acc, float scale,
                                       bf16* __restrict__ dqkv) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // one per 4 elements
  const long long total = n_tok * d / 4;
  if (idx >= total) return;
  const long long e = idx * 4;
  const long long n = e / d; const int c = (int)(e % d);
  float4 v = *reinterpret_cast<const float4*>(dq_acc + e);
  uint2 u;
  *reinterpret_cast<__nv_bfloat162*>(&u.x) = __floats2bfloat162_rn(v.x * scale, v.y * scale);
  *reinterpret_cast<__nv_bfloat162*>(&u.y) = __floats2bfloat162_rn(v.z * scale, v.w * scale);
  *reinterpret_cast<uint2*>(dqkv + n * 3 * d + c) = u;
}

template <int HD>
fax_status launch_bwd(fax_ctx* ctx, int B, int T, int H, const void* qkv, const void* o, const float* lse,
                      const void* d_o, void* dqkv, float* Dv, float* dq_acc) {
  CUtensorMap mq, md, mdq;
  const uint64_t d = (uint64_t)H * HD;
  const long long n_tok = (long long)B * T;
  if (!make_map(ctx, &mq, qkv, 3 * d, (uint64_t)n_tok, 3 * d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map(ctx, &md, d_o, d, (uint64_t)n_tok, d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map_f32(ctx, &mdq, dq_acc, d, (uint64_t)n_tok, d, 32, 128)) return FAX_ERR_INVALID_ARG;
  FAX_CUDA_TRY(ctx, cudaMemsetAsync(dq_acc, 0, (size_t)n_tok * d * sizeof(float), ctx->stream));
  {
    const long long warps = n_tok * H;
    const int threads = 256;
    const long long blocks = (warps * 32 + threads - 1) / threads;
    attn_rowdot_bf16_kernel<<<(unsigned)blocks, threads, 0, ctx->stream>>>((int)n_tok, T, H, HD, (const bf16*)d_o,
                                                                          (const bf16*)o, Dv);
    FAX_TRY(fax_after_launch(ctx));
  }
  AttnBwdParams p;
  p.B = B; p.T = T; p.H = H; p.lse = lse; p.Dv = Dv; p.dq_acc = dq_acc; p.dqkv = (bf16*)dqkv;
  p.scale = 1.0f / sqrtf((float)HD);
  p.scale_log2 = 1.4426950408889634f * p.scale;
  p.status = ctx->dev_status;
  static bool attr_set = false;
  if (!attr_set) {
    FAX_CUDA_TRY(ctx, cudaFuncSetAttribute(attn_bwd_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           BwdCfg<HD>::SMEM_BYTES));
    attr_set = true;
  }
  const int grid = B * H * (T / 128);
  attn_bwd_tc_kernel<HD><<<grid, BWD_THREADS, BwdCfg<HD>::SMEM_BYTES, ctx->stream>>>(mq, md, mdq, p);
  FAX_TRY(fax_after_launch(ctx));
  const long long quads = n_tok * (long long)d / 4;
  attn_dq_convert_kernel<<<(unsigned)((quads + 255) / 256), 256, 0, ctx->stream>>>(n_tok, (int)d, dq_acc, p.scale,
                                                                                  (bf16*)dqkv);
  return fax_after_launch(ctx);
}

}  // namespace

bool fax_attention_tc_supported(int B, int T, int H, int hd) {
  return (hd == 64 || hd == 128) && T % 128 == 0 && B > 0 && H > 0;
}

fax_status fax_attention_fwd_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, void* o, float* lse) {
  if (!fax_attention_tc_supported(B, T, H, hd) || !fax_aligned(qkv, 16) || !fax_aligned(o, 16))
    return FAX_ERR_UNSUPPORTED_SHAPE;
  // sequences of a whole number of query-tile pairs take the two-tile persistent kernel
  if (fax_attention_fwd2_supported(B, T, H, hd)) return fax_attention_fwd2_tc(ctx, B, T, H, hd, qkv, o, lse);
  return hd == 64 ? launch_fwd<64>(ctx, B, T, H, qkv, o, lse) : launch_fwd<128>(ctx, B, T, H, qkv, o, lse);
}

size_t fax_attention_bwd_tc_scratch_bytes(int B, int T, int H, int hd) {
  return fax_round_up((size_t)B * H * T * sizeof(float), 256) + (size_t)B * T * H * hd * sizeof(float);
}

fax_status fax_attention_bwd_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const void* o,
                                const float* lse, const void* d_o, void* dqkv, void* scratch, size_t scratch_bytes) {
  if (!fax_attention_tc_supported(B, T, H, hd) || !fax_aligned(qkv, 16) || !fax_aligned(o, 16) ||
      !fax_aligned(d_o, 16) || !fax_aligned(dqkv, 16) || !fax_aligned(scratch, 256))
    return FAX_ERR_UNSUPPORTED_SHAPE;
  if (scratch_bytes < fax_attention_bwd_tc_scratch_bytes(B, T, H, hd)) return FAX_ERR_WORKSPACE_TOO_SMALL;
  float* Dv = (float*)scratch;
  float* dq_acc = (float*)((char*)scratch + fax_round_up((size_t)B * H * T * sizeof(float), 256));
  return hd == 64 ? launch_bwd<64>(ctx, B, T, H, qkv, o, lse, d_o, dqkv, Dv, dq_acc)
                  : launch_bwd<128>(ctx, B, T, H, qkv, o, lse, d_o, dqkv, Dv, dq_acc);
}
