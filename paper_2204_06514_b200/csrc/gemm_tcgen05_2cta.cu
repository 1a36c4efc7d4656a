// bf16 GEMM with the tensor cores of two SMs working on one 256 x 256 output tile
// (tcgen05.mma.cta_group::2).  A cluster of two CTAs; CTA r of the pair holds rows
// 128 r .. 128 r + 127 of the A tile and rows 128 r .. of the B tile (its half of N) in
// its own shared memory and its half of the accumulator (128 lanes x 256 columns) in
// its own tensor memory.  Per 64-wide K block each SM therefore stages 32 KB instead of
// 48 KB and its tensor core reads 8 KB instead of 12 KB of operands per MMA: the
// shared-memory and L2 traffic per FLOP drop by a third against the one-CTA kernel.
//
//   warp 0      : TMA producer (both CTAs; each loads its own halves and signals the
//                 even CTA's "full" barrier)
//   warp 1      : tensor-memory allocation (both CTAs); MMA issue (even CTA only);
//                 tcgen05.commit multicasts "stage empty" / "accumulator full" to both
//   warps 2..9  : epilogue of the CTA's own 128 x 256 half; "accumulator empty" is
//                 signalled to the even CTA's barrier.  Outputs are stored from registers; the
//                 partial tiles of a K-sliced float GEMM are staged in shared memory and added
//                 into C by bulk tensor reductions.
// Every TMA load is a plain load into the issuing CTA's own shared memory.  Every wait is bounded.
#include "gemm_common.cuh"

#include <cstddef>

namespace {

using namespace tc;

constexpr int BM = 128;            // rows per CTA (256 per pair)
constexpr int BN = 256;            // columns per pair; each CTA stages 128 of B's rows
constexpr int BNH = 128;
constexpr int BK = 64;
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = 32 * (2 + NUM_EPI_WARPS);
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BNH * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int STAGES = 6;
constexpr int TMEM_COLS = 512;
constexpr int STAGING_BYTES = NUM_EPI_WARPS * EPI_STAGING_BYTES;
constexpr int BAR_BYTES = 256;
// Only a K-sliced float output stages partial tiles; every other launch leaves that shared memory to L1 (which
// the epilogue's residual / pre-activation loads go through) and to the blocks of the kernels that run beside
// or right behind this one (the AdamW stream, the next kernel's blocks under programmatic dependent launch:
// with the staging in every float-output launch a block step of hidden 5120 took 4.9 instead of 4.5 ms).
constexpr int smem_bytes(bool staged) { return STAGES * STAGE_BYTES + (staged ? STAGING_BYTES : 0) + 1024 + BAR_BYTES; }
static_assert(smem_bytes(true) <= 227 * 1024, "shared memory per CTA");
static_assert(8 * (2 * STAGES + 4) + 8 <= BAR_BYTES, "barrier area");

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The same shared-memory offset in the even CTA (rank 0) of the pair, as a shared::cluster address.
__device__ __forceinline__ uint32_t leader_addr(uint32_t a) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(0u));
  return r;
}

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// Arrival on a barrier of the pair's even CTA.  Relaxed: what it orders is this warp's
// tensor-memory reads, which tcgen05.wait::ld and the tcgen05 fence have already completed; a
// release at cluster scope would also wait until the warp's global stores have drained.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tcgen05_2cta_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const GemmParams p, const __grid_constant__ CUtensorMap tmap_c) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (tiles_base - raw);
  const uint32_t staging = tiles_base + STAGES * STAGE_BYTES;
  const int stg_bytes = (EPI == EPI_STATIC_F32 && p.splits > 1) ? STAGING_BYTES : 0;      // as the launcher sized it
  uint8_t* bar_mem = gen_base + STAGES * STAGE_BYTES + stg_bytes;
  const uint32_t bars = staging + (uint32_t)stg_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };                         // used in the even CTA
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };             // one per CTA
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };         // one per CTA
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };    // used in the even CTA
  volatile uint32_t* tmem_base_slot = (volatile uint32_t*)(bar_mem + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = (volatile int*)(bar_mem + 8 * (2 * STAGES + 4) + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = (rank == 0);
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int tiles_m = p.M / (2 * BM), tiles_n = p.N / BN;
  const int out_tiles = tiles_m * tiles_n;
  const int num_tiles = out_tiles * p.splits;
  const int kb_total = p.K / BK;
  const int kb_per = (kb_total + p.splits - 1) / p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * NUM_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    if (EPI == EPI_STATIC_F32) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_c) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_base_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  fax_grid_dependency_wait();    // set-up above may run under the previous kernel's tail; global memory only from here

  if (warp == 0) {
    // ---------------- TMA producer (each CTA loads its own halves) ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        int tm, tn;
        tile_coords(tile % out_tiles, tiles_m, tiles_n, p.group_m, p.group_along_n, tm, tn);
        const int m0 = tm * 2 * BM + (int)rank * BM, n0 = tn * BN + (int)rank * BNH;
        const int kb0 = (tile / out_tiles) * kb_per, kb1 = min(kb_total, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 111)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const uint32_t fbar = leader_addr(full_bar(stage));
          if (leader) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);       // both CTAs' bytes
          const int k0 = kb * BK;
          if (!p.a_mn) {
            tma_load_2d_pair(a_dst, &tmap_a, fbar, k0, m0);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(a_dst + i * 8192, &tmap_a, fbar, m0 + 64 * i, k0);
          }
          if (!p.b_mn) {
            tma_load_2d_pair(b_dst, &tmap_b, fbar, k0, n0);
          } else {
#pragma unroll
            for (int i = 0; i < BNH / 64; ++i) tma_load_2d_pair(b_dst + i * 8192, &tmap_b, fbar, n0 + 64 * i, k0);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (even CTA of the pair) ----------------
    if (leader && lane == 0) {
      // D = f32, A = B = bf16, majors, N = 256, M = 256 over the pair
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)((2 * BM) >> 4) << 24);
      const uint32_t a_kstep = p.a_mn ? 2048u : 32u, b_kstep = p.b_mn ? 2048u : 32u;
      const uint32_t a_lbo = p.a_mn ? 8192u : 16u, b_lbo = p.b_mn ? 8192u : 16u;
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 112)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        const int kb0 = (tile / out_tiles) * kb_per, kb1 = min(kb_total, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 113)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t ad = smem_desc(a_src + k * a_kstep, a_lbo, 1024u);
            const uint64_t bd = smem_desc(b_src + k * b_kstep, b_lbo, 1024u);
            tc_mma_bf16_pair(d_tmem, ad, bd, idesc, ((kb - kb0) | k) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(stage));      // frees this stage in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar(acc));          // accumulator complete, both halves
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue: this CTA's 128 rows of the tile ----------------
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    constexpr int NCH = BN / 64;
    static_assert(NCH == EPI_TMA_CHUNKS, "a warp's share is four chunks");
    int acc = 0; uint32_t acc_phase = 0;
    const uint32_t stg = staging + (uint32_t)(warp - 2) * EPI_STAGING_BYTES;
    const bool reduce_out = EPI == EPI_STATIC_F32 && p.splits > 1;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
      int tm, tn;
      tile_coords(tile % out_tiles, tiles_m, tiles_n, p.group_m, p.group_along_n, tm, tn);
      const int m0 = tm * 2 * BM + (int)rank * BM, n0 = tn * BN;
      const long long row = m0 + 32 * q + lane;
      const int col0 = n0 + half * (BN / 2);
      U8 x0[2];
      gemm_epilogue_fetch<EPI>(p, row, col0, x0);     // in flight while the accumulator fills
      if (!mbar_wait_warp(tfull_bar(acc), acc_phase, abort_flag, p.status, 114)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_base = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * BN + half * (BN / 2));
      auto drained = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_addr(tempty_bar(acc)));
      };
      if (reduce_out) gemm_epilogue_warp_reduce(p, &tmap_c, t_base, m0 + 32 * q, col0, lane, stg, drained);
      else gemm_epilogue_warp<NCH, EPI>(p, t_base, row, col0, x0, drained);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (reduce_out && lane == 0) bulk_wait_all();     // the staging buffers have been read and the additions are complete
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // neither CTA leaves (or frees tensor memory) while the other may still signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

bool fax_gemm_patch_info_2cta(const void* func, const void* param, size_t* size, size_t* sc_offset) {
  if (func != (const void*)gemm_tcgen05_2cta_kernel<-1>) return false;
  if (((const GemmParams*)param)->epi != EPI_ADAMW) return false;
  *size = sizeof(GemmParams);
  *sc_offset = offsetof(GemmParams, ad_sc);
  return true;
}

bool fax_gemm_tc2_supported(const FaxGemm& g) { return g.M % 256 == 0 && g.N % 256 == 0 && g.K % BK == 0; }

// Caller has already checked fax_gemm_tc_supported (alignment, strides).
fax_status fax_gemm_tc2(fax_ctx* ctx, const FaxGemm& g) {
  CUtensorMap ma, mb;
  bool ok = g.a_mn_major ? make_map(ctx, &ma, g.A, g.M, g.K, g.lda, 64, BK)
                         : make_map(ctx, &ma, g.A, g.K, g.M, g.lda, BK, BM);
  ok = ok && (g.b_mn_major ? make_map(ctx, &mb, g.B, g.N, g.K, g.ldb, 64, BK)
                           : make_map(ctx, &mb, g.B, g.K, g.N, g.ldb, BK, BNH));
  if (!ok) return FAX_ERR_INVALID_ARG;
  CUtensorMap mc = ma;                                   // read only by the K-sliced float epilogue
  if (g.c_f32 && !make_map_f32(ctx, &mc, g.C, g.N, g.M, g.ldc, 32, 32)) return FAX_ERR_INVALID_ARG;
  GemmParams p;
  fill_gemm_params(p, g, ctx->dev_status);
  {
    static bool attr_set[7][FAX_MAX_DEVICES] = {};
#define FAX_SET_SMEM(I, E) FAX_TRY(fax_opt_in_shared_memory(ctx, gemm_tcgen05_2cta_kernel<E>, smem_bytes(E == EPI_STATIC_F32), attr_set[I]))
    FAX_SET_SMEM(0, -1); FAX_SET_SMEM(1, 0); FAX_SET_SMEM(2, 1); FAX_SET_SMEM(3, 2); FAX_SET_SMEM(4, 3); FAX_SET_SMEM(5, 4);
    FAX_SET_SMEM(6, EPI_STATIC_F32);
#undef FAX_SET_SMEM
  }
  const int tiles = (g.M / 256) * (g.N / 256);
  const int max_pairs = ctx->sm_count / 2;
  p.splits = gemm_split_count(g, tiles, max_pairs, BK);
  if (p.splits == 1 && ctx->gemm_l2_budget > 0) gemm_choose_raster(p, 256, 256, max_pairs, ctx->gemm_l2_budget);
  if (p.splits > 1 && !g.accumulate)
    FAX_CUDA_TRY(ctx, cudaMemset2DAsync(g.C, (size_t)g.ldc * 4, 0, (size_t)g.N * 4, (size_t)g.M, ctx->stream));
  const int items = tiles * p.splits;
  const int pairs = items < max_pairs ? items : max_pairs;
  switch (gemm_static_epi(g)) {
#define FAX_LAUNCH(E) case E: fax_launch(ctx, gemm_tcgen05_2cta_kernel<E>, dim3(2 * pairs), dim3(NUM_THREADS), smem_bytes(E == EPI_STATIC_F32 && p.splits > 1), ma, mb, p, mc); break
    FAX_LAUNCH(0); FAX_LAUNCH(1); FAX_LAUNCH(2); FAX_LAUNCH(3); FAX_LAUNCH(4); FAX_LAUNCH(EPI_STATIC_F32);
    default: fax_launch(ctx, gemm_tcgen05_2cta_kernel<-1>, dim3(2 * pairs), dim3(NUM_THREADS), smem_bytes(false), ma, mb, p, mc); break;
#undef FAX_LAUNCH
  }
  return fax_after_launch(ctx);
}
