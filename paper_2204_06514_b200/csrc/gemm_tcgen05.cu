// bf16 GEMM on the 5th-generation tensor cores: TMA-fed multi-stage shared
// memory ring, tcgen05.mma issued by one thread with float accumulators in
// tensor memory, double-buffered so the epilogue of one tile overlaps the main
// loop of the next, persistent over output tiles.
//
//   warp 0      : TMA producer (one elected lane)
//   warp 1      : tensor-memory allocation, MMA issue (one elected lane)
//   warps 2..9  : epilogue; warp w reads TMEM lanes 32*(w%4) .. +31, columns half (w-2)/4
//
// Operand layouts (both for A and B, chosen at run time):
//   K-major  : [rows, K] row-major; one TMA box of 64 k x rows, 128-byte swizzle;
//              8-row groups 1024 B apart (SBO); a K step of 16 elements is +32 B.
//   MN-major : [K, rows] row-major; TMA boxes of 64 rows x 64 k (one per 64 rows,
//              8192 B apart = LBO); 8-k groups 1024 B apart (SBO); a K step of 16
//              is +2048 B.
// Every device-side wait is bounded; on expiry the kernel records an error in
// the context's status word, drains and returns.
#include "gemm_common.cuh"

#include <cstddef>

namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int NUM_EPI_WARPS = 8;      // two per tensor-memory lane quarter, each storing half of the columns
constexpr int NUM_THREADS = 32 * (2 + NUM_EPI_WARPS);
template <int BN> struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                    const GemmParams p) {
  using C_ = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (tiles_base - raw);
  uint8_t* bar_mem = gen_base + C_::STAGES * C_::STAGE_BYTES;
  const uint32_t bars = tiles_base + C_::STAGES * C_::STAGE_BYTES;
  // barrier layout: full[S], empty[S], tmem_full[2], tmem_empty[2], then tmem base word + abort flag
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (C_::STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * C_::STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * C_::STAGES + 2 + a); };
  volatile uint32_t* tmem_base_slot = (volatile uint32_t*)(bar_mem + 8 * (2 * C_::STAGES + 4));
  volatile int* abort_flag = (volatile int*)(bar_mem + 8 * (2 * C_::STAGES + 4) + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = p.M / BM, tiles_n = p.N / BN;
  const int out_tiles = tiles_m * tiles_n;
  const int num_tiles = out_tiles * p.splits;          // work items: (output tile, K slice)
  const int kb_total = p.K / BK;
  const int kb_per = (kb_total + p.splits - 1) / p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C_::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), NUM_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_base_slot)), "r"((uint32_t)C_::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  fax_grid_dependency_wait();    // set-up above may run under the previous kernel's tail; global memory only from here

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tm, tn;
        tile_coords(tile % out_tiles, tiles_m, tiles_n, p.group_m, p.group_along_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        const int kb0 = (tile / out_tiles) * kb_per, kb1 = min(kb_total, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 101)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * C_::STAGE_BYTES;
          const uint32_t b_dst = a_dst + C_::A_BYTES;
          mbar_expect_tx(full_bar(stage), C_::STAGE_BYTES);
          const int k0 = kb * BK;
          if (!p.a_mn) {
            tma_load_2d(a_dst, &tmap_a, full_bar(stage), k0, m0);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d(a_dst + i * 8192, &tmap_a, full_bar(stage), m0 + 64 * i, k0);
          }
          if (!p.b_mn) {
            tma_load_2d(b_dst, &tmap_b, full_bar(stage), k0, n0);
          } else {
#pragma unroll
            for (int i = 0; i < BN / 64; ++i) tma_load_2d(b_dst + i * 8192, &tmap_b, full_bar(stage), n0 + 64 * i, k0);
          }
          if (++stage == C_::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let copies already in flight land before the block can exit
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      const uint32_t a_kstep = p.a_mn ? 2048u : 32u, b_kstep = p.b_mn ? 2048u : 32u;
      const uint32_t a_lbo = p.a_mn ? 8192u : 16u, b_lbo = p.b_mn ? 8192u : 16u;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 102)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        const int kb0 = (tile / out_tiles) * kb_per, kb1 = min(kb_total, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 103)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * C_::STAGE_BYTES;
          const uint32_t b_src = a_src + C_::A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t ad = smem_desc(a_src + k * a_kstep, a_lbo, 1024u);
            const uint64_t bd = smem_desc(b_src + k * b_kstep, b_lbo, 1024u);
            tc_mma_bf16(d_tmem, ad, bd, idesc, ((kb - kb0) | k) ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));          // frees the smem stage once these MMAs have read it
          if (++stage == C_::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));              // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue ----------------
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;            // which half of the tile's columns this warp stores
    constexpr int NCH = BN / 64;                 // 32-column chunks per warp
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int tm, tn;
      tile_coords(tile % out_tiles, tiles_m, tiles_n, p.group_m, p.group_along_n, tm, tn);
      const int m0 = tm * BM, n0 = tn * BN;
      const long long row = m0 + 32 * q + lane;
      U8 x0[2];
      gemm_epilogue_fetch<-1>(p, row, n0 + half * (BN / 2), x0);      // in flight while the accumulator fills
      if (!mbar_wait_warp(tfull_bar(acc), acc_phase, abort_flag, p.status, 104)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_base = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * BN + half * (BN / 2));
      gemm_epilogue_warp<NCH, -1>(p, t_base, row, n0 + half * (BN / 2), x0, [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_relaxed(tempty_bar(acc));
      });
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C_::TMEM_COLS) : "memory");
  }
}

int pick_bn(int N) { return (N % 256 == 0) ? 256 : (N % 128 == 0 ? 128 : (N % 64 == 0 ? 64 : 0)); }

template <int BN>
fax_status launch(fax_ctx* ctx, const FaxGemm& g) {
  CUtensorMap ma, mb;
  bool ok = g.a_mn_major ? make_map(ctx, &ma, g.A, g.M, g.K, g.lda, 64, BK)
                         : make_map(ctx, &ma, g.A, g.K, g.M, g.lda, BK, BM);
  ok = ok && (g.b_mn_major ? make_map(ctx, &mb, g.B, g.N, g.K, g.ldb, 64, BK)
                           : make_map(ctx, &mb, g.B, g.K, g.N, g.ldb, BK, BN));
  if (!ok) return FAX_ERR_INVALID_ARG;
  GemmParams p;
  fill_gemm_params(p, g, ctx->dev_status);
  static bool attr_set[FAX_MAX_DEVICES] = {};
  FAX_TRY(fax_opt_in_shared_memory(ctx, gemm_tcgen05_kernel<BN>, Cfg<BN>::SMEM_BYTES, attr_set));
  const int tiles = (g.M / BM) * (g.N / BN);
  // Few output tiles and a long K (the weight-gradient shapes of narrow models): slice K so that
  // the machine is filled; partial tiles are added into the float output with vector atomics.
  p.splits = gemm_split_count(g, tiles, ctx->sm_count, BK);
  if (p.splits == 1 && ctx->gemm_l2_budget > 0) gemm_choose_raster(p, BM, BN, ctx->sm_count, ctx->gemm_l2_budget);
  if (p.splits > 1 && !g.accumulate)
    FAX_CUDA_TRY(ctx, cudaMemset2DAsync(g.C, (size_t)g.ldc * 4, 0, (size_t)g.N * 4, (size_t)g.M, ctx->stream));
  const int items = tiles * p.splits;
  const int grid = items < ctx->sm_count ? items : ctx->sm_count;
  fax_launch(ctx, gemm_tcgen05_kernel<BN>, dim3(grid), dim3(NUM_THREADS), Cfg<BN>::SMEM_BYTES, ma, mb, p);
  return fax_after_launch(ctx);
}

}  // namespace

bool fax_gemm_patch_info_1cta(const void* func, const void* param, size_t* size, size_t* sc_offset) {
  if (func != (const void*)gemm_tcgen05_kernel<256> && func != (const void*)gemm_tcgen05_kernel<128> &&
      func != (const void*)gemm_tcgen05_kernel<64>)
    return false;
  if (((const GemmParams*)param)->epi != EPI_ADAMW) return false;
  *size = sizeof(GemmParams);
  *sc_offset = offsetof(GemmParams, ad_sc);
  return true;
}

bool fax_gemm_can_fuse_adam(fax_ctx* ctx, const FaxGemm& g) {
  if (!fax_gemm_tc_supported(g) || !g.c_f32 || g.epi != EPI_NONE || g.accumulate || g.alpha != 1.f) return false;
  if (g.ldc != g.N) return false;                       // w, m, v share C's dense layout
  FaxGemm plain = g;
  plain.adam = nullptr;
  if (ctx->use_2cta && fax_gemm_tc2_supported(g))
    return gemm_split_count(plain, (g.M / 256) * (g.N / 256), ctx->sm_count / 2, BK) == 1;
  return gemm_split_count(plain, (g.M / BM) * (g.N / pick_bn(g.N)), ctx->sm_count, BK) == 1;
}

bool fax_gemm_tc_supported(const FaxGemm& g) {
  if (g.M % BM || g.K % BK || pick_bn(g.N) == 0) return false;
  if (g.lda % 8 || g.ldb % 8) return false;
  if (!fax_aligned(g.A, 16) || !fax_aligned(g.B, 16) || !fax_aligned(g.C, 32)) return false;
  if (g.ldc % (g.c_f32 ? 8 : 16)) return false;             // the epilogue stores whole 32-byte sectors
  if (g.bias && !fax_aligned(g.bias, 16)) return false;
  if (g.resid && (!fax_aligned(g.resid, 32) || g.ldr % 16)) return false;
  if (g.aux && (!fax_aligned(g.aux, 32) || g.ldaux % 16)) return false;
  return true;
}

// A dimension that is 128 past a multiple of 256 (the vocabulary of the LM head): the two-CTA
// kernel takes the multiple-of-256 part, the one-CTA kernel the last 128 rows or columns.
static bool split_for_two_cta(fax_ctx* ctx, const FaxGemm& g, FaxGemm* main_part, FaxGemm* tail) {
  if (!ctx->use_2cta || g.adam || g.K % 64) return false;
  const size_t es = 2, cs = g.c_f32 ? 4 : 2;
  if (g.M % 256 == 0 && g.N % 256 == 128 && g.N > 1024) {
    const int n1 = g.N - 128;
    *main_part = g; *tail = g;
    main_part->N = n1; tail->N = 128;
    tail->B = (const char*)g.B + (g.b_mn_major ? (size_t)n1 : (size_t)n1 * g.ldb) * es;
    tail->C = (char*)g.C + (size_t)n1 * cs;
    if (g.bias) tail->bias = (const char*)g.bias + (size_t)n1 * es;
    if (g.resid) tail->resid = (const char*)g.resid + (size_t)n1 * es;
    if (g.aux) tail->aux = (char*)g.aux + (size_t)n1 * es;
    return true;
  }
  if (g.N % 256 == 0 && g.M % 256 == 128 && g.M > 1024) {
    const int m1 = g.M - 128;
    *main_part = g; *tail = g;
    main_part->M = m1; tail->M = 128;
    tail->A = (const char*)g.A + (g.a_mn_major ? (size_t)m1 : (size_t)m1 * g.lda) * es;
    tail->C = (char*)g.C + (size_t)m1 * g.ldc * cs;
    if (g.resid) tail->resid = (const char*)g.resid + (size_t)m1 * g.ldr * es;
    if (g.aux) tail->aux = (char*)g.aux + (size_t)m1 * g.ldaux * es;
    return true;
  }
  return false;
}

fax_status fax_gemm_tc(fax_ctx* ctx, const FaxGemm& g) {
  if (!fax_gemm_tc_supported(g)) return FAX_ERR_UNSUPPORTED_SHAPE;
  FaxProfScope prof(ctx, KC_GEMM_TC, 2.0 * g.M * g.N * g.K, 0.0);
  if (ctx->use_2cta && fax_gemm_tc2_supported(g)) return fax_gemm_tc2(ctx, g);
  FaxGemm part, tail;
  if (split_for_two_cta(ctx, g, &part, &tail) && fax_gemm_tc_supported(part) && fax_gemm_tc_supported(tail)) {
    FAX_TRY(fax_gemm_tc2(ctx, part));
    return launch<128>(ctx, tail);
  }
  switch (pick_bn(g.N)) {
    case 256: return launch<256>(ctx, g);
    case 128: return launch<128>(ctx, g);
    default: return launch<64>(ctx, g);
  }
}
