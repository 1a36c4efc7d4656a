// Causal attention forward (step F3), two query tiles per CTA, persistent.
//
// A CTA owns pairs of neighbouring 128-query tiles (A = 2m, B = 2m+1) of one (batch, head) and
// walks the key tiles 0..2m+1 once for both, so K and V are loaded once per pair.  Each query
// tile has its own group of four softmax warps (one row per thread), its own S accumulator and
// its own O accumulator in tensor memory; the elected MMA thread alternates between the tiles
// (P_A V, S_A of the next key tile, P_B V, S_B of the next key tile), so one group's softmax runs
// under the other group's products.  P never touches shared memory: the softmax threads write
// it as bf16 over the first 64 columns of their S accumulator and the P V product takes its A
// operand from tensor memory.  The CTA loops over its share of the work list (heaviest pairs
// first); the next pair's Q, K and V tiles are requested as soon as their buffers are free, so
// the set-up of one pair hides under the tail of the one before.  Every wait is bounded.
//
// head_dim 64 leaves 128 tensor-memory columns free, which hold P beside S (EARLY_S): a group's softmax
// threads signal "S read" as soon as the scores are in registers, the MMA thread issues the NEXT key
// tile's S product right then, and the group goes from one tile's softmax straight into the next
// without waiting for a product.  With that the exponentials (1024 clocks of the special-function
// units per 128 x 128 tile, more than the tile's 876 tensor-core clocks at head_dim 64) are the bound;
// before, each group's loop was softmax + both products + the hand-offs, about 2900 clocks per tile.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int F2_THREADS = 320;    // 2 x 4 softmax warps + MMA warp + TMA warp

struct AttnFwd2Params {
  int B, T, H;
  bf16* o; float* lse;
  float scale_log2;
  int32_t* status;
};

template <int HD> struct Fwd2Cfg {
  static constexpr int TILE_BYTES = 128 * HD * 2;        // Q, K or V tile
  static constexpr int NS = (HD == 64) ? 4 : 2;          // K and V ring depth
  static constexpr int Q_OFF = 0;                        // two query tiles
  static constexpr int K_OFF = 2 * TILE_BYTES;
  static constexpr int V_OFF = K_OFF + NS * TILE_BYTES;
  static constexpr int BAR_OFF = V_OFF + NS * TILE_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 512 + 1024;
  static constexpr int TMEM_COLS = 512;                  // S_A [0,128) S_B [128,256) O_A [256,..) O_B [384,..)
  static constexpr bool EARLY_S = (HD == 64);            // then O_A [256,320) O_B [320,384) P_A [384,448) P_B [448,512)
  static constexpr int O_STRIDE = EARLY_S ? 64 : 128;
  // barriers
  static constexpr int QFULL = 0, QFREE = 2, SFULL = 4, PREADY = 6, OFULL = 8, OFREE = 10, SREAD = 12, PFREE = 14;
  static constexpr int KFULL = 16, KFREE = KFULL + NS, VFULL = KFREE + NS, VFREE = VFULL + NS;
  static constexpr int NBARS = VFREE + NS;
  static_assert(NBARS <= 32, "barrier area");
};

template <int HD>
__device__ __forceinline__ void load_tile2(uint32_t dst, const CUtensorMap* map, uint32_t bar, int col, int row) {
  mbar_expect_tx(bar, 128 * HD * 2);
#pragma unroll
  for (int i = 0; i < HD / 64; ++i) tma_load_2d(dst + i * 16384, map, bar, col + 64 * i, row);
}

template <int HD>
__global__ void __launch_bounds__(F2_THREADS, 1)
attn_fwd2_tc_kernel(const __grid_constant__ CUtensorMap tmap, const AttnFwd2Params p) {
  using C_ = Fwd2Cfg<HD>;
  constexpr int NS = C_::NS;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + 256);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + 260);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int npairs = p.T / 256;
  const int bh_count = p.B * p.H;
  const int n_items = npairs * bh_count;
  const int d = p.H * HD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C_::NBARS; ++i) {
      const bool four = (i == C_::PREADY || i == C_::PREADY + 1 || i == C_::OFREE || i == C_::OFREE + 1 ||
                         i == C_::SREAD || i == C_::SREAD + 1);
      mbar_init(bar(i), four ? 4u : 1u);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
  }
  if (warp == 8) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  fax_grid_dependency_wait();    // set-up above may run under the previous kernel's tail; global memory only from here
  auto q_s = [&](int x) { return base + C_::Q_OFF + x * C_::TILE_BYTES; };
  auto k_s = [&](int i) { return base + C_::K_OFF + i * C_::TILE_BYTES; };
  auto v_s = [&](int i) { return base + C_::V_OFF + i * C_::TILE_BYTES; };

  if (warp == 9) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t kc = 0;          // K / V tiles requested so far
      bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it) {
        const int m = npairs - 1 - t / bh_count, bh = t % bh_count;
        const int b = bh / p.H, h = bh % p.H;
        const int row0 = b * p.T;
        const uint32_t iph = (uint32_t)(it & 1);
        for (int x = 0; x < 2 && ok; ++x) {
          if (!mbar_wait(bar(C_::QFREE + x), iph ^ 1u, abort_flag, p.status, 221)) { ok = false; break; }
          load_tile2<HD>(q_s(x), &tmap, bar(C_::QFULL + x), h * HD, row0 + (2 * m + x) * 128);
        }
        const int nkv = 2 * m + 2;
        for (int j = 0; j < nkv && ok; ++j, ++kc) {
          const int s = (int)(kc % NS);
          const uint32_t ph = (kc / NS) & 1u;
          if (!mbar_wait(bar(C_::KFREE + s), ph ^ 1u, abort_flag, p.status, 222)) { ok = false; break; }
          load_tile2<HD>(k_s(s), &tmap, bar(C_::KFULL + s), d + h * HD, row0 + j * 128);
          if (!mbar_wait(bar(C_::VFREE + s), ph ^ 1u, abort_flag, p.status, 223)) { ok = false; break; }
          load_tile2<HD>(v_s(s), &tmap, bar(C_::VFULL + s), 2 * d + h * HD, row0 + j * 128);
        }
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, false, false);
      const uint32_t idesc_o = idesc_bf16(HD, false, true);
      // descriptors = {low word, high word}; only the start-address field (16-byte units) of the low word
      // differs between tiles and k-steps, so each product adds a constant to a precomputed word (the
      // instructions of this one thread between two products are on the critical path)
      const uint32_t d_hi = (uint32_t)(smem_desc(0, 16, 1024) >> 32);
      const uint32_t q_lo0 = (uint32_t)smem_desc(q_s(0), 16, 1024), k_lo0 = (uint32_t)smem_desc(k_s(0), 16, 1024);
      const uint32_t v_lo0 = (uint32_t)smem_desc(v_s(0), 16384, 1024);
      constexpr uint32_t TILE16 = C_::TILE_BYTES >> 4;
      auto mk = [&](uint32_t lo) -> uint64_t { return ((uint64_t)d_hi << 32) | lo; };
      uint32_t kc0 = 0;                 // K / V tiles of the pairs before this one
      uint32_t pc[2] = {0u, 0u};        // P tiles consumed per query tile
      uint32_t ns[2] = {0u, 0u};        // S tiles issued per query tile
      bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it) {
        const int m = npairs - 1 - t / bh_count;
        const int nkv = 2 * m + 2, lastA = nkv - 2, lastB = nkv - 1;
        const uint32_t iph = (uint32_t)(it & 1);
        // S_x = Q_x K_j^T into the S accumulator of query tile x
        auto issue_s = [&](int x, int j) -> bool {
          const uint32_t c = kc0 + (uint32_t)j;
          const int s = (int)(c % NS);
          if (C_::EARLY_S && ns[x] > 0 &&
              !mbar_wait(bar(C_::SREAD + x), (ns[x] - 1u) & 1u, abort_flag, p.status, 232)) return false;
          ++ns[x];
          if (!mbar_wait(bar(C_::KFULL + s), (c / NS) & 1u, abort_flag, p.status, 224)) return false;
          tc_fence_after();
          const uint32_t qlo = q_lo0 + (uint32_t)x * TILE16, klo = k_lo0 + (uint32_t)s * TILE16;
          const uint32_t dst = tmem + (uint32_t)(x * 128);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint32_t off = (k / 4) * 1024 + (k % 4) * 2;
            tc_mma_bf16(dst, mk(qlo + off), mk(klo + off), idesc_s, k ? 1u : 0u);
          }
          tc_commit(bar(C_::SFULL + x));
          return true;
        };
        // O_x += P_x V_j, P_x read from the first 64 columns of the S accumulator
        auto issue_pv = [&](int x, int j) -> bool {
          if (!mbar_wait(bar(C_::PREADY + x), pc[x] & 1u, abort_flag, p.status, 225)) return false;
          ++pc[x];
          if (j == 0 && !mbar_wait(bar(C_::OFREE + x), iph ^ 1u, abort_flag, p.status, 226)) return false;
          tc_fence_after();
          const int s = (int)((kc0 + (uint32_t)j) % NS);
          const uint32_t vlo = v_lo0 + (uint32_t)s * TILE16;
          const uint32_t dst = tmem + 256u + (uint32_t)(x * C_::O_STRIDE);
          const uint32_t src = C_::EARLY_S ? tmem + 384u + (uint32_t)(x * 64) : tmem + (uint32_t)(x * 128);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            tc_mma_bf16_ts(dst, src + 8 * k, mk(vlo + k * 128), idesc_o, (j | k) ? 1u : 0u);
          if (C_::EARLY_S) tc_commit(bar(C_::PFREE + x));
          return true;
        };
        if (!mbar_wait(bar(C_::QFULL), iph, abort_flag, p.status, 227)) { ok = false; break; }
        if (!mbar_wait(bar(C_::QFULL + 1), iph, abort_flag, p.status, 228)) { ok = false; break; }
        if (!issue_s(0, 0)) { ok = false; break; }
        if (lastA == 0) tc_commit(bar(C_::QFREE));
        if (!issue_s(1, 0)) { ok = false; break; }
        tc_commit(bar(C_::KFREE + (int)(kc0 % NS)));
        for (int j = 0; j < nkv && ok; ++j) {
          const uint32_t c = kc0 + (uint32_t)j;
          const int s = (int)(c % NS);
          if (C_::EARLY_S) {
            // the next key tile's scores first (they wait only for "S read"), then this tile's P V products
            if (j + 1 <= lastA) {
              if (!issue_s(0, j + 1)) { ok = false; break; }
              if (j + 1 == lastA) tc_commit(bar(C_::QFREE));
            }
            if (j + 1 <= lastB) {
              if (!issue_s(1, j + 1)) { ok = false; break; }
              tc_commit(bar(C_::KFREE + (int)((c + 1) % NS)));
              if (j + 1 == lastB) tc_commit(bar(C_::QFREE + 1));
            }
            if (!mbar_wait(bar(C_::VFULL + s), (c / NS) & 1u, abort_flag, p.status, 229)) { ok = false; break; }
            if (j <= lastA) {
              if (!issue_pv(0, j)) { ok = false; break; }
              if (j == lastA) tc_commit(bar(C_::OFULL));
            }
            if (!issue_pv(1, j)) { ok = false; break; }
            tc_commit(bar(C_::VFREE + s));
            if (j == lastB) tc_commit(bar(C_::OFULL + 1));
            continue;
          }
          if (!mbar_wait(bar(C_::VFULL + s), (c / NS) & 1u, abort_flag, p.status, 229)) { ok = false; break; }
          if (j <= lastA) {
            if (!issue_pv(0, j)) { ok = false; break; }
            if (j == lastA) tc_commit(bar(C_::OFULL));
            if (j + 1 <= lastA) {
              if (!issue_s(0, j + 1)) { ok = false; break; }
              if (j + 1 == lastA) tc_commit(bar(C_::QFREE));
            }
          }
          if (!issue_pv(1, j)) { ok = false; break; }
          tc_commit(bar(C_::VFREE + s));
          if (j == lastB) tc_commit(bar(C_::OFULL + 1));
          if (j + 1 <= lastB) {
            if (!issue_s(1, j + 1)) { ok = false; break; }
            tc_commit(bar(C_::KFREE + (int)((c + 1) % NS)));      // tile B is the last reader of every K tile
            if (j + 1 == lastB) tc_commit(bar(C_::QFREE + 1));
          }
        }
        kc0 += (uint32_t)nkv;
      }
    }
  } else {
    // ---- softmax threads: group x = warp / 4 serves query tile x, one row per thread ----
    const int x = warp >> 2, wq = warp & 3;
    const int r = 32 * wq + lane;
    const uint32_t lane_base = (uint32_t)(32 * wq) << 16;
    const uint32_t tm_s = tmem + (uint32_t)(x * 128) + lane_base;
    const uint32_t tm_o = tmem + 256u + (uint32_t)(x * C_::O_STRIDE) + lane_base;
    const uint32_t tm_p = C_::EARLY_S ? tmem + 384u + (uint32_t)(x * 64) + lane_base : tm_s;
    uint32_t sc = 0;                  // S tiles consumed
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it) {
      const int m = npairs - 1 - t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int qx = 2 * m + x;       // this group's query tile = its last (diagonal) key tile
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j <= qx; ++j, ++sc) {
        if (!mbar_wait_warp(bar(C_::SFULL + x), sc & 1u, abort_flag, p.status, 230)) { ok = false; break; }
        tc_fence_after();
        uint32_t sv[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tc_ld32(tm_s + (uint32_t)(32 * c), sv[c]);
        tc_wait_ld();
        if (C_::EARLY_S) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::SREAD + x));       // the next key tile's scores may overwrite S
        }
        // EARLY_S: P V of the tile before (global count sc - 1) must be complete before O is rescaled or P overwritten
        bool pv_done = !C_::EARLY_S || sc == 0;
        if (j == qx) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (32 * c + e > r) sv[c][e] = 0xff800000u;      // -inf
        }
        float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            mxa[(e >> 1) & 3] = max3(mxa[(e >> 1) & 3], __uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1]));
        const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
        const float m_new = fmaxf(m_used, mx * p.scale_log2);
        // O is rescaled only when a row maximum of the warp has grown by more than 2^8.  Without EARLY_S,
        // S_j complete implies P V of tile j-1 complete (the MMA thread issues them in that order)
        if (__any_sync(0xffffffffu, m_new > m_used + 8.0f)) {
          if (j > 0) {
            if (!pv_done) {
              if (!mbar_wait_warp(bar(C_::PFREE + x), (sc - 1u) & 1u, abort_flag, p.status, 233)) { ok = false; break; }
              tc_fence_after();
              pv_done = true;
            }
            const float factor = ex2_approx(m_used - m_new);
            l *= factor;
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
              uint32_t ov[32];
              tc_ld32(tm_o + (uint32_t)c0, ov);
              tc_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * factor);
              tc_st32(tm_o + (uint32_t)c0, ov);
            }
          }
          m_used = m_new;
        }
        float rowsum = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t packed[32];
#pragma unroll
          for (int cc = 0; cc < 2; ++cc)
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float p0 = ex2_approx(__uint_as_float(sv[2 * half + cc][e]) * p.scale_log2 - m_used);
              const float p1 = ex2_approx(__uint_as_float(sv[2 * half + cc][e + 1]) * p.scale_log2 - m_used);
              rowsum += p0 + p1;
              __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
              packed[16 * cc + (e >> 1)] = *reinterpret_cast<uint32_t*>(&h2);
            }
          if (half == 0 && !pv_done) {
            if (!mbar_wait_warp(bar(C_::PFREE + x), (sc - 1u) & 1u, abort_flag, p.status, 233)) { ok = false; break; }
            tc_fence_after();
            pv_done = true;
          }
          tc_st32(tm_p + (uint32_t)(32 * half), packed);
        }
        if (!ok) break;
        l += rowsum;
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::PREADY + x));
      }
      if (!ok) break;
      if (!mbar_wait_warp(bar(C_::OFULL + x), (uint32_t)(it & 1), abort_flag, p.status, 231)) { ok = false; break; }
      tc_fence_after();
      const float inv = 1.f / l;
      const long long tok = (long long)b * p.T + qx * 128 + r;
      bf16* orow = p.o + tok * d + h * HD;
#pragma unroll 1
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t ov[32];
        tc_ld32(tm_o + (uint32_t)c0, ov);
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
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::OFREE + x));
      p.lse[((long long)b * p.H + h) * p.T + qx * 128 + r] = (m_used + log2f(l)) * 0.6931471805599453f;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

template <int HD>
fax_status launch_fwd2(fax_ctx* ctx, int B, int T, int H, const void* qkv, void* o, float* lse) {
  CUtensorMap map;
  const uint64_t d = (uint64_t)H * HD;
  if (!make_map(ctx, &map, qkv, 3 * d, (uint64_t)B * T, 3 * d, 64, 128)) return FAX_ERR_INVALID_ARG;
  AttnFwd2Params p;
  p.B = B; p.T = T; p.H = H; p.o = (bf16*)o; p.lse = lse;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  p.status = ctx->dev_status;
  static bool attr_set[FAX_MAX_DEVICES] = {};
  FAX_TRY(fax_opt_in_shared_memory(ctx, attn_fwd2_tc_kernel<HD>, Fwd2Cfg<HD>::SMEM_BYTES, attr_set));
  const long long items = (long long)B * H * (T / 256);
  const int grid = (int)(items < ctx->sm_count ? items : ctx->sm_count);
  fax_launch(ctx, attn_fwd2_tc_kernel<HD>, dim3(grid), dim3(F2_THREADS), Fwd2Cfg<HD>::SMEM_BYTES, map, p);
  return fax_after_launch(ctx);
}

}  // namespace

bool fax_attention_fwd2_supported(int B, int T, int H, int hd) {
  return (hd == 64 || hd == 128) && T % 256 == 0 && B > 0 && H > 0;
}

fax_status fax_attention_fwd2_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, void* o, float* lse) {
  if (!fax_attention_fwd2_supported(B, T, H, hd)) return FAX_ERR_UNSUPPORTED_SHAPE;
  return hd == 64 ? launch_fwd2<64>(ctx, B, T, H, qkv, o, lse) : launch_fwd2<128>(ctx, B, T, H, qkv, o, lse);
}
