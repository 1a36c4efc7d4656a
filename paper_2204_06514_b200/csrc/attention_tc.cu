// Causal multi-head attention on the tcgen05 tensor cores (steps F3 / B5).
//
// Forward (sequence lengths that are not a multiple of 256; the others take the two-tile kernel
// of attention_fwd2_tc.cu): one CTA per (batch, head, 128-query tile).  Q stays in shared memory;
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
  fax_grid_dependency_wait();    // set-up above may run under the previous kernel's tail; global memory only from here
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
  static bool attr_set[FAX_MAX_DEVICES] = {};
  FAX_TRY(fax_opt_in_shared_memory(ctx, attn_fwd_tc_kernel<HD>, FwdCfg<HD>::SMEM_BYTES, attr_set));
  const int grid = B * H * (T / TQ);
  fax_launch(ctx, attn_fwd_tc_kernel<HD>, dim3(grid), dim3(FWD_THREADS), FwdCfg<HD>::SMEM_BYTES, map, p);
  return fax_after_launch(ctx);
}


constexpr int BWD_THREADS = 320;   // 8 row warps (4 lane quarters x 2 column halves) + MMA warp + TMA warp

struct AttnBwdParams {
  int B, T, H;
  const float* lse; const float* Dv;
  float* dq_acc; bf16* dqkv;
  float scale, scale_log2;
  int32_t* status;
};

// ---------------------------------------------------------------------------
// Backward (step B5), persistent.  A CTA owns a 128-key tile j (K_j, V_j resident in shared memory) and
// walks the query tiles i >= j; the score tiles are formed transposed (keys in the tensor-memory lanes):
//   S^T = K_j Q_i^T, dP^T = V_j dO_i^T, so P^T and dS^T (bf16, written back over their own
// accumulators by the row threads) are the A operands of dV_j += P^T dO_i and dK_j += dS^T Q_i
// straight from tensor memory; only dS also goes to shared memory, as the MN-major A operand of
// dQ_i = dS K_j.  After dS the MMA thread issues dQ first, then dK and (Q is double-buffered) S^T of
// the next step, so these run while the row threads read dQ out.  A row thread owns one key row and
// one half of the tile's 128 queries; the per-query statistics (LSE, D) of the tile sit in shared
// memory.  A CTA loops over its share of the (batch, head, key tile) list, longest walks first;
// the next tile's K, V, Q, dO loads overlap the read-out of dK and dV.
// Tensor memory: [0,128) S^T, then P^T at +64h+[0,32) and dS^T at +64h+[32,64) | [128,256) dP^T, then dQ |
// [256,256+HD) dV | [384,384+HD) dK.
// ---------------------------------------------------------------------------
template <int HD> struct Bwd2Cfg {
  static constexpr int NQ = 2;                             // Q stages
  static constexpr int NDO = (HD == 64) ? 2 : 1;           // dO stages
  static constexpr int TILE_BYTES = 128 * HD * 2;
  static constexpr int K_OFF = 0, V_OFF = TILE_BYTES;
  static constexpr int Q_OFF = 2 * TILE_BYTES, DO_OFF = Q_OFF + NQ * TILE_BYTES;
  static constexpr int DS_OFF = DO_OFF + NDO * TILE_BYTES;  // dS tile (32 KB); the dQ staging boxes start here too
  static constexpr int STG_BYTES = 128 * HD * 4;            // dQ tile in float32
  static constexpr int DS_BYTES = (STG_BYTES > 32768) ? STG_BYTES : 32768;
  // head_dim 64 leaves room for dQ staging buffers of their own, two of them: the write of dS and the
  // staging of a dQ tile then never wait for the bulk reduction of the step before (only for the one
  // two steps back).  At head_dim 128 the staging boxes share the dS tile's bytes.
  static constexpr int NSTG = (HD == 64) ? 2 : 1;
  static constexpr int STG_OFF = (HD == 64) ? DS_OFF + DS_BYTES : DS_OFF;
  static constexpr int STAT_OFF = (HD == 64) ? STG_OFF + NSTG * STG_BYTES : DS_OFF + DS_BYTES;   // [2][2][128] floats: log2e*LSE and D of the query tile
  static constexpr int BAR_OFF = STAT_OFF + 2048;
  static constexpr int LAYOUT_BYTES = BAR_OFF + 256;
  // 768 bytes of slack for aligning the tiles to 1024 bytes (at hd 128 this is exactly the 227 KB a CTA
  // may have); the kernel checks that the aligned layout fits before it touches anything
  static constexpr int SMEM_BYTES = LAYOUT_BYTES + 768;
  static constexpr int TMEM_COLS = 512;
  // barriers
  static constexpr int KVFULL = 0, KVFREE = 1, QFULL = 2, QFREE = 4, DOFULL = 6, DOFREE = 8, SFULL = 10, DPFULL = 11,
                       PREADY = 12, DSREADY = 13, DQFULL = 14, DQREAD = 15, DKVREAD = 16, STGFREE = 17, STGFULL = 18,
                       STATFULL = 19, ALLDONE = 20, STGFREE2 = 21, NBARS = 22;
};

template <int HD>
__global__ void __launch_bounds__(BWD_THREADS, 1)
attn_bwd2_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const __grid_constant__ CUtensorMap tmap_do,
                    const __grid_constant__ CUtensorMap tmap_dq, const AttnBwdParams p) {
  using C_ = Bwd2Cfg<HD>;
  constexpr int NQ = C_::NQ, NDO = C_::NDO;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + 192);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + 196);
  if ((base - raw) + (uint32_t)C_::LAYOUT_BYTES > (uint32_t)C_::SMEM_BYTES) {
    // the dynamic shared memory window starts less aligned than assumed: report, touch nothing
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, 1) == 0) p.status[1] = 320;
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / 128;
  const int bh_count = p.B * p.H;
  const int n_items = nq * bh_count;
  const int d = p.H * HD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C_::NBARS; ++i) {
      const bool eight = (i == C_::PREADY || i == C_::DSREADY || i == C_::DQREAD || i == C_::DKVREAD ||
                          i == C_::STGFULL || i == C_::STATFULL);
      mbar_init(bar(i), eight ? 8u : 1u);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_do) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_dq) : "memory");
  }
  if (warp == 8) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  fax_grid_dependency_wait();    // set-up above may run under the previous kernel's tail; global memory only from here
  const uint32_t tm_st = tmem, tm_dp = tmem + 128, tm_dv = tmem + 256, tm_dk = tmem + 384;
  const uint32_t k_s = base + C_::K_OFF, v_s = base + C_::V_OFF, ds_s = base + C_::DS_OFF;
  auto q_s = [&](int i) { return base + C_::Q_OFF + i * C_::TILE_BYTES; };
  auto do_s = [&](int i) { return base + C_::DO_OFF + i * C_::TILE_BYTES; };

  if (warp == 9) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t gs = 0;              // steps requested so far (all items)
      bool ok = true;
      int it_n = 0;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
        const int kj = t / bh_count, bh = t % bh_count;
        const int b = bh / p.H, h = bh % p.H;
        const int row0 = b * p.T;
        const int qcol = h * HD, kcol = d + h * HD, vcol = 2 * d + h * HD;
        if (!mbar_wait(bar(C_::KVFREE), (uint32_t)(it_n & 1) ^ 1u, abort_flag, p.status, 321)) { ok = false; break; }
        mbar_expect_tx(bar(C_::KVFULL), 2 * C_::TILE_BYTES);
#pragma unroll
        for (int i = 0; i < HD / 64; ++i) {
          tma_load_2d(k_s + i * 16384, &tmap_qkv, bar(C_::KVFULL), kcol + 64 * i, row0 + kj * 128);
          tma_load_2d(v_s + i * 16384, &tmap_qkv, bar(C_::KVFULL), vcol + 64 * i, row0 + kj * 128);
        }
        const int nsteps = nq - kj;
        for (int it = 0; it < nsteps && ok; ++it, ++gs) {
          const int qrow = row0 + (kj + it) * 128;
          const int sq = (int)(gs % NQ), sd = (int)(gs % NDO);
          if (!mbar_wait(bar(C_::QFREE + sq), ((gs / NQ) & 1u) ^ 1u, abort_flag, p.status, 322)) { ok = false; break; }
          mbar_expect_tx(bar(C_::QFULL + sq), C_::TILE_BYTES);
#pragma unroll
          for (int i = 0; i < HD / 64; ++i) tma_load_2d(q_s(sq) + i * 16384, &tmap_qkv, bar(C_::QFULL + sq), qcol + 64 * i, qrow);
          if (!mbar_wait(bar(C_::DOFREE + sd), ((gs / NDO) & 1u) ^ 1u, abort_flag, p.status, 323)) { ok = false; break; }
          mbar_expect_tx(bar(C_::DOFULL + sd), C_::TILE_BYTES);
#pragma unroll
          for (int i = 0; i < HD / 64; ++i) tma_load_2d(do_s(sd) + i * 16384, &tmap_do, bar(C_::DOFULL + sd), qcol + 64 * i, qrow);
        }
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, false, false);     // S^T, dP^T: both operands K-major
      const uint32_t idesc_acc = idesc_bf16(HD, false, true);      // dV, dK: A in tensor memory, B MN-major
      const uint32_t idesc_dq = idesc_bf16(HD, true, true);        // dQ: dS and K both MN-major
      auto koff = [](int s) { return (uint32_t)((s / 4) * 16384 + (s % 4) * 32); };   // K-major k-step
      auto acol = [](int k) { return (uint32_t)(64 * (k / 4) + 8 * (k % 4)); };       // A k-step in tensor memory
      uint32_t gs = 0;
      bool ok = true;
      int it_n = 0;
      auto issue_s = [&](uint32_t g) -> bool {
        const int sq = (int)(g % NQ);
        if (!mbar_wait(bar(C_::QFULL + sq), (g / NQ) & 1u, abort_flag, p.status, 324)) return false;
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < HD / 16; ++s)
          tc_mma_bf16(tm_st, smem_desc(k_s + koff(s), 16, 1024), smem_desc(q_s(sq) + koff(s), 16, 1024), idesc_s, s ? 1u : 0u);
        tc_commit(bar(C_::SFULL));
        return true;
      };
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
        const int kj = t / bh_count;
        const int nsteps = nq - kj;
        if (!mbar_wait(bar(C_::KVFULL), (uint32_t)(it_n & 1), abort_flag, p.status, 325)) { ok = false; break; }
        if (!issue_s(gs)) { ok = false; break; }
        for (int it = 0; it < nsteps && ok; ++it, ++gs) {
          const int sq = (int)(gs % NQ), sd = (int)(gs % NDO);
          // dP^T = V dO^T (its columns held the previous step's dQ: wait until that was read out)
          if (!mbar_wait(bar(C_::DOFULL + sd), (gs / NDO) & 1u, abort_flag, p.status, 326)) { ok = false; break; }
          if (gs > 0 && !mbar_wait(bar(C_::DQREAD), (gs - 1) & 1u, abort_flag, p.status, 327)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int s = 0; s < HD / 16; ++s)
            tc_mma_bf16(tm_dp, smem_desc(v_s + koff(s), 16, 1024), smem_desc(do_s(sd) + koff(s), 16, 1024), idesc_s, s ? 1u : 0u);
          tc_commit(bar(C_::DPFULL));
          // dV += P^T dO (the first one of a key tile overwrites: dV and dK of the tile before must have been read out)
          if (!mbar_wait(bar(C_::PREADY), gs & 1u, abort_flag, p.status, 328)) { ok = false; break; }
          if (it == 0 && !mbar_wait(bar(C_::DKVREAD), (uint32_t)(it_n & 1) ^ 1u, abort_flag, p.status, 329)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)
            tc_mma_bf16_ts(tm_dv, tm_st + acol(k), smem_desc(do_s(sd) + k * 2048, 16384, 1024), idesc_acc, (it | k) ? 1u : 0u);
          tc_commit(bar(C_::DOFREE + sd));
          // dQ = dS K over the dP^T columns (all read by now), then dK += dS^T Q with dS^T from the spare
          // columns of the S^T accumulator, then S^T of the next step over that accumulator
          if (!mbar_wait(bar(C_::DSREADY), gs & 1u, abort_flag, p.status, 330)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)
            tc_mma_bf16(tm_dp, smem_desc(ds_s + k * 2048, 16384, 1024), smem_desc(k_s + k * 2048, 16384, 1024), idesc_dq,
                        k ? 1u : 0u);
          tc_commit(bar(C_::DQFULL));
#pragma unroll
          for (int k = 0; k < 8; ++k)
            tc_mma_bf16_ts(tm_dk, tm_st + 32u + acol(k), smem_desc(q_s(sq) + k * 2048, 16384, 1024), idesc_acc, (it | k) ? 1u : 0u);
          tc_commit(bar(C_::QFREE + sq));
          if (it + 1 == nsteps) {
            tc_commit(bar(C_::KVFREE));
            tc_commit(bar(C_::ALLDONE));         // every MMA of this key tile is complete: dV and dK are final
          } else if (!issue_s(gs + 1)) { ok = false; break; }
        }
      }
    }
  } else {
    // ---- row threads: key row kr (dQ read-out: query row kr), query / column half hc ----
    const int hc = warp >> 2;
    const int kr = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    uint8_t* ds_row = gbase + C_::DS_OFF + hc * 16384 + kr * 128;
    float* stat = reinterpret_cast<float*>(gbase + C_::STAT_OFF);      // [buf][0: lse2, 1: D][128]
    const int tid = threadIdx.x;                                       // 0..255
    uint32_t gs = 0;
    bool ok = true;
    int it_n = 0;
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
      const int kj = t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int row0 = b * p.T;
      const int nsteps = nq - kj;
      const long long stat0 = ((long long)b * p.H + h) * p.T;
      auto load_stats = [&](int qi, uint32_t buf) {
        const long long idx = stat0 + qi * 128 + (tid & 127);
        stat[buf * 256 + tid] = (tid < 128) ? p.lse[idx] * 1.4426950408889634f : p.Dv[idx];
      };
      // statistics of a step are published through a barrier of eight warp arrivals: one phase per step
      load_stats(kj, gs & 1u);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::STATFULL));
      for (int it = 0; it < nsteps; ++it, ++gs) {
        const uint32_t ph = gs & 1u;
        const int qi = kj + it;
        const float* st_l = stat + ph * 256 + 64 * hc;
        const float* st_d = st_l + 128;
        if (!mbar_wait_warp(bar(C_::STATFULL), ph, abort_flag, p.status, 335)) { ok = false; break; }
        if (it + 1 < nsteps) {
          // the other buffer was last read in the step before this one, which every warp has left
          // (this step's S^T needed the previous dS of all of them)
          load_stats(qi + 1, ph ^ 1u);
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::STATFULL));
        }
        uint32_t pp[32];
        // P^T = exp(S^T / sqrt(hd) - LSE[q])
        if (!mbar_wait_warp(bar(C_::SFULL), ph, abort_flag, p.status, 331)) { ok = false; break; }
        tc_fence_after();
        {
          uint32_t sv[2][32];
          tc_ld32(tm_st + lane_base + 64 * hc, sv[0]);
          tc_ld32(tm_st + lane_base + 64 * hc + 32, sv[1]);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 l4 = *reinterpret_cast<const float4*>(st_l + 32 * c + e);
              float p0 = ex2_approx(__uint_as_float(sv[c][e]) * p.scale_log2 - l4.x);
              float p1 = ex2_approx(__uint_as_float(sv[c][e + 1]) * p.scale_log2 - l4.y);
              float p2 = ex2_approx(__uint_as_float(sv[c][e + 2]) * p.scale_log2 - l4.z);
              float p3 = ex2_approx(__uint_as_float(sv[c][e + 3]) * p.scale_log2 - l4.w);
              if (it == 0) {        // diagonal tile: query index below key index is masked
                const int q0 = 64 * hc + 32 * c + e;
                if (q0 < kr) p0 = 0.f;
                if (q0 + 1 < kr) p1 = 0.f;
                if (q0 + 2 < kr) p2 = 0.f;
                if (q0 + 3 < kr) p3 = 0.f;
              }
              __nv_bfloat162 h0 = __floats2bfloat162_rn(p0, p1), h1 = __floats2bfloat162_rn(p2, p3);
              pp[16 * c + (e >> 1)] = *reinterpret_cast<uint32_t*>(&h0);
              pp[16 * c + (e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h1);
            }
        }
        tc_st32(tm_st + lane_base + 64 * hc, pp);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::PREADY));
        // dS^T = P^T * (dP^T - D[q]), from the bf16 P that the products use
        if (!mbar_wait_warp(bar(C_::DPFULL), ph, abort_flag, p.status, 332)) { ok = false; break; }
        tc_fence_after();
        uint32_t dd[32];
        {
          uint32_t dv[2][32];
          tc_ld32(tm_dp + lane_base + 64 * hc, dv[0]);
          tc_ld32(tm_dp + lane_base + 64 * hc + 32, dv[1]);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 d4 = *reinterpret_cast<const float4*>(st_d + 32 * c + e);
              const float2 pa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pp[16 * c + (e >> 1)]));
              const float2 pb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pp[16 * c + (e >> 1) + 1]));
              __nv_bfloat162 h0 = __floats2bfloat162_rn(pa.x * (__uint_as_float(dv[c][e]) - d4.x),
                                                        pa.y * (__uint_as_float(dv[c][e + 1]) - d4.y));
              __nv_bfloat162 h1 = __floats2bfloat162_rn(pb.x * (__uint_as_float(dv[c][e + 2]) - d4.z),
                                                        pb.y * (__uint_as_float(dv[c][e + 3]) - d4.w));
              dd[16 * c + (e >> 1)] = *reinterpret_cast<uint32_t*>(&h0);
              dd[16 * c + (e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h1);
            }
        }
        tc_st32(tm_st + lane_base + 64 * hc + 32, dd);
        if (HD == 128 && gs > 0) {
          // the dS buffer staged the first 32 KB of the previous dQ tile: the bulk reductions of those
          // boxes (the older of the step's two groups) must have read it
          if (tid == 0) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            mbar_arrive(bar(C_::STGFREE));
          }
          if (!mbar_wait_warp(bar(C_::STGFREE), (gs - 1) & 1u, abort_flag, p.status, 333)) { ok = false; break; }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<uint4*>(ds_row + ((k ^ (kr & 7)) << 4)) = make_uint4(dd[4 * k], dd[4 * k + 1], dd[4 * k + 2], dd[4 * k + 3]);
        fence_proxy_async();
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::DSREADY));
        // dQ tile: tensor memory -> shared memory (32-column float boxes, 128-byte swizzled) -> one bulk
        // add-reduction per box into the float32 dQ accumulator
        if (!mbar_wait_warp(bar(C_::DQFULL), ph, abort_flag, p.status, 334)) { ok = false; break; }
        tc_fence_after();
        if (HD == 128 && gs > 0) {
          // boxes 2 and 3 (the column half of warps 4..7) lie behind the dS tile: their reductions of the step before
          if (tid == 0) { bulk_wait_read_all(); mbar_arrive(bar(C_::STGFREE2)); }
          if (hc == 1 && !mbar_wait_warp(bar(C_::STGFREE2), (gs - 1) & 1u, abort_flag, p.status, 337)) { ok = false; break; }
        }
        if (HD == 64 && gs > 1) {
          // staging buffer gs & 1 was last the source of the reduction issued two steps ago (one bulk
          // group per step): all but the newest group must have read their boxes
          if (tid == 0) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            mbar_arrive(bar(C_::STGFREE));
          }
          if (!mbar_wait_warp(bar(C_::STGFREE), gs & 1u, abort_flag, p.status, 333)) { ok = false; break; }
        }
        const uint32_t stg_off = (uint32_t)C_::STG_OFF + (HD == 64 ? (gs & 1u) * (uint32_t)C_::STG_BYTES : 0u);
        {
          constexpr int NB = HD / 64;          // this warp's half of the head's columns: two boxes or one
          const int c0 = hc * (HD / 2);
          uint32_t v[NB][32];
#pragma unroll
          for (int cc = 0; cc < NB; ++cc) tc_ld32(tm_dp + lane_base + c0 + 32 * cc, v[cc]);
          tc_wait_ld();
#pragma unroll
          for (int cc = 0; cc < NB; ++cc) {
            uint8_t* box = gbase + stg_off + ((c0 >> 5) + cc) * 16384 + kr * 128;
#pragma unroll
            for (int k = 0; k < 8; ++k)
              *reinterpret_cast<uint4*>(box + ((k ^ (kr & 7)) << 4)) =
                  make_uint4(v[cc][4 * k], v[cc][4 * k + 1], v[cc][4 * k + 2], v[cc][4 * k + 3]);
          }
        }
        tc_fence_before();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) { mbar_arrive(bar(C_::DQREAD)); mbar_arrive(bar(C_::STGFULL)); }
        if (tid == 0 && mbar_wait(bar(C_::STGFULL), ph, abort_flag, p.status, 336)) {
#pragma unroll
          for (int i = 0; i < HD / 32; ++i) {
            tma_reduce_add_2d(&tmap_dq, base + stg_off + i * 16384, h * HD + 32 * i, (int)(row0 + qi * 128));
            if (HD == 128 && i == 1) bulk_commit_group();     // boxes 0, 1 (the dS tile's bytes) as a group of their own
          }
          bulk_commit_group();
        }
      }
      if (!ok) break;
      if (!mbar_wait_warp(bar(C_::ALLDONE), (uint32_t)(it_n & 1), abort_flag, p.status, 338)) { ok = false; break; }
      tc_fence_after();
      {
        const long long tok = (long long)row0 + kj * 128 + kr;
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
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::DKVREAD));
      }
    }
    if (tid == 0) bulk_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

// D[b,h,t] = sum_c dO[t,c] * O[t,c] over the head's columns.  A thread takes 8 columns (one 16-byte
// vector of each operand), hd / 8 neighbouring lanes share a (token, head) and add up with shuffles.
// The same thread also clears its 8 elements of the float32 dQ accumulator [n_tok, H * hd], which
// the backward kernel's bulk reductions add into (no separate memset).
__global__ void __launch_bounds__(256)
attn_rowdot_bf16_kernel(int n_tok, int T, int H, int hd, const bf16* __restrict__ d_o,
                        const bf16* __restrict__ o, float* __restrict__ Dv, float* __restrict__ dq_acc) {
  fax_grid_dependency_wait();
  const int lanes = hd >> 3;                                   // 8 (hd 64) or 16 (hd 128): divides the warp
  const long long vec = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = (long long)n_tok * H * lanes;
  const bool in = vec < total;
  float s = 0.f;
  if (in) {
    const uint4 a = reinterpret_cast<const uint4*>(d_o)[vec];  // rows are dense: vector index = element / 8
    const uint4 b = reinterpret_cast<const uint4*>(o)[vec];
    reinterpret_cast<float4*>(dq_acc)[2 * vec] = make_float4(0.f, 0.f, 0.f, 0.f);
    reinterpret_cast<float4*>(dq_acc)[2 * vec + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
    const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 fa = __bfloat1622float2(ha[e]), fb = __bfloat1622float2(hb[e]);
      s += fa.x * fb.x + fa.y * fb.y;
    }
  }
  for (int off = lanes >> 1; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (in && (vec % lanes) == 0) {
    const long long th = vec / lanes;                          // token * H + head
    const int tok = (int)(th / H), h = (int)(th % H);
    Dv[((long long)(tok / T) * H + h) * T + (tok % T)] = s;
  }
}

// dqkv[n, 0:d] = bf16(dq_acc[n, :] * scale)
__global__ void attn_dq_convert_kernel(long long n_tok, int d, const float* __restrict__ dq_acc, float scale,
                                       bf16* __restrict__ dqkv) {
  fax_grid_dependency_wait();
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
  {
    const long long vecs = n_tok * H * (HD / 8);
    const int threads = 256;
    const long long blocks = (vecs + threads - 1) / threads;
    fax_launch(ctx, attn_rowdot_bf16_kernel, dim3((unsigned)blocks), dim3(threads), 0, (int)n_tok, T, H, HD,
               (const bf16*)d_o, (const bf16*)o, Dv, dq_acc);
    FAX_TRY(fax_after_launch(ctx));
  }
  AttnBwdParams p;
  p.B = B; p.T = T; p.H = H; p.lse = lse; p.Dv = Dv; p.dq_acc = dq_acc; p.dqkv = (bf16*)dqkv;
  p.scale = 1.0f / sqrtf((float)HD);
  p.scale_log2 = 1.4426950408889634f * p.scale;
  p.status = ctx->dev_status;
  if (ctx->attn_bwd_mode >= 2 && fax_attention_bwd4_supported(B, T, H, HD)) {
    FAX_TRY(fax_attention_bwd4_tc(ctx, B, T, H, HD, qkv, lse, d_o, dqkv, Dv, dq_acc));
  } else if (ctx->attn_bwd_mode >= 1 && fax_attention_bwd3_supported(B, T, H, HD)) {
    FAX_TRY(fax_attention_bwd3_tc(ctx, B, T, H, HD, qkv, lse, d_o, dqkv, Dv, dq_acc));
  } else {
    static bool attr_set[FAX_MAX_DEVICES] = {};
    FAX_TRY(fax_opt_in_shared_memory(ctx, attn_bwd2_tc_kernel<HD>, Bwd2Cfg<HD>::SMEM_BYTES, attr_set));
    const long long items = (long long)B * H * (T / 128);
    const int grid = (int)(items < ctx->sm_count ? items : ctx->sm_count);
    fax_launch(ctx, attn_bwd2_tc_kernel<HD>, dim3(grid), dim3(BWD_THREADS), Bwd2Cfg<HD>::SMEM_BYTES, mq, md, mdq, p);
    FAX_TRY(fax_after_launch(ctx));
  }
  const long long quads = n_tok * (long long)d / 4;
  fax_launch(ctx, attn_dq_convert_kernel, dim3((unsigned)((quads + 255) / 256)), dim3(256), 0, n_tok, (int)d, dq_acc,
             p.scale, (bf16*)dqkv);
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
