// Causal attention backward (step B5), head_dim 128 and 64: sixteen row warps, half-tile hand-offs.
// (Written for head_dim 128 below; at head_dim 64 the operand tiles are one 64-column panel, dV and dK
// take 64 tensor-memory columns each, and dQ is formed untransposed, dQ = dS K with the queries in the
// lanes, because the transposed form would have only 64 rows; its staging is by query rows.)
//
// A CTA owns a 128-key tile j (K_j, V_j resident in shared memory) and walks the 128-query tiles
// i >= j.  Everything is formed transposed (keys in the tensor-memory lanes): S^T = K_j Q_i^T and
// dP^T = V_j dO_i^T are 128 x 128 accumulators; P^T and dS^T (bf16) are written back over spare
// columns of the S^T accumulator and are the tensor-memory A operands of dV_j += P^T dO_i and
// dK_j += dS^T Q_i; dS^T also goes to shared memory as the B operand of dQ_i^T = K_j^T dS^T (head
// dimension in the lanes), which lands on the columns of dP^T.  Tensor memory (512 columns):
//   [0,128)   S^T; query quarter r then holds P^T at 32 r + [0,16) and dS^T at 32 r + [16,32)
//   [128,256) dP^T, then dQ^T        [256,384) dV        [384,512) dK
// Every product is 128 wide (a 128 x N x 16 MMA takes the same ~70 clocks for any N <= 128, so
// narrower tiles waste the tensor pipe).  With one score tile in flight the overlap comes from
// finer hand-offs: sixteen row warps (one key row per thread, a quarter of the tile's queries each,
// four warps per scheduler so that tensor-memory and special-function latencies hide each other)
// publish P^T and dS^T per query half, and the MMA thread issues the matching half of the dV and dK
// contractions as soon as a half is there; after the second dS^T half it issues dQ^T first, then
// the rest of dK and S^T of the next query tile, which run under the dQ^T read-out.  The dQ^T tile
// goes tensor memory -> shared memory (transposed back to query rows) -> bulk tensor add-reductions
// into the float32 dQ accumulator, issued by a warp of its own.  The reduction engine drains a 64 KB
// tile in about 2500 clocks, so nothing on the critical path may wait for it: the second query half
// is staged in the bytes of the dS^T tile (dead once dQ^T is done; its reduction goes first and has
// the whole P phase of the next tile to finish), the first half in the bytes of this tile's dO stage
// (dead once dV is done; the TMA producer waits for that reduction before it refills the stage, two
// tiles later).  Staging in the Q stage instead delayed the next Q tile and with it S^T.
// Per-query statistics (log2e * LSE, D) travel with the Q stage they belong to.  The MMA thread
// builds every shared-memory descriptor from precomputed words with one addition.  Every wait is bounded.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int B3_ROW_WARPS = 16;
constexpr int B3_THREADS = 32 * (B3_ROW_WARPS + 3);   // + MMA warp, TMA / statistics warp, dQ reduction warp

struct Bwd3Params {
  int B, T, H;
  const float* lse; const float* Dv;
  bf16* dqkv;
  float scale, scale_log2;
  int32_t* status;
};

template <int HD_> struct B3 {
  static constexpr int HD = HD_;
  static constexpr int TILE_BYTES = 128 * HD * 2;         // HD / 64 panels of 128 rows x 128 B
  static constexpr int K_OFF = 0, V_OFF = TILE_BYTES;
  static constexpr int Q_OFF = 2 * TILE_BYTES;            // two stages
  static constexpr int DO_OFF = 4 * TILE_BYTES;           // two stages
  static constexpr int DS_OFF = 6 * TILE_BYTES;           // dS^T: two panels (query halves) of 128 key rows x 128 B
  static constexpr int STAT_OFF = DS_OFF + 32768;         // [2 stages][0: log2e * lse, 1: D][128] floats
  static constexpr int BAR_OFF = STAT_OFF + 2 * 1024;
  // a dQ tile is staged as 2 x 4 boxes of 64 rows x 32 floats (32 KB per query half): first half in the tile's
  // dO stage, second half in the dS^T tile
  static constexpr int KVFULL = 0, KVFREE = 1, QFULL = 2, QFREE = 4, DOFULL = 6, DOFREE = 8, SFULL = 10, DPFULL = 11,
                       PREADY = 12, DSREADY = 14, DQFULL = 16, DQREAD = 17, STGFULL = 18 /* per half */,
                       STGFREE_DO = 20 /* per stage */, STGFREE_DS = 22, ALLDONE = 23, DKVREAD = 24, NBARS = 25;
  static constexpr int LAYOUT_BYTES = BAR_OFF + NBARS * 8 + 16;
  // the layout plus slack for aligning it to 1024 bytes, capped at the 227 KB a block may have (head_dim 128)
  static constexpr int SMEM_BYTES = (LAYOUT_BYTES + 1024 < 227 * 1024) ? LAYOUT_BYTES + 1024 : 227 * 1024;
  static constexpr int TMEM_COLS = 512;
};
static_assert(B3<128>::LAYOUT_BYTES + 512 <= B3<128>::SMEM_BYTES, "shared-memory layout does not fit");

template <int HD>
__global__ void __launch_bounds__(B3_THREADS, 1)
attn_bwd3_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const __grid_constant__ CUtensorMap tmap_do,
                    const __grid_constant__ CUtensorMap tmap_dq, const Bwd3Params p) {
  using C_ = B3<HD>;
  constexpr uint32_t HALF_WARPS = B3_ROW_WARPS / 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + C_::NBARS * 8);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + C_::NBARS * 8 + 4);
  if ((base - raw) + (uint32_t)C_::LAYOUT_BYTES > (uint32_t)C_::SMEM_BYTES) {
    if (threadIdx.x == 0 && atomicCAS(p.status, 0, 1) == 0) p.status[1] = 340;
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / 128;
  const int bh_count = p.B * p.H;
  const int n_items = nq * bh_count;
  const int d = p.H * HD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C_::NBARS; ++i) {
      uint32_t count = 1;
      if (i == C_::PREADY || i == C_::PREADY + 1 || i == C_::DSREADY || i == C_::DSREADY + 1) count = HALF_WARPS;
      if (i == C_::DQREAD || i == C_::DKVREAD) count = B3_ROW_WARPS;
      if (i == C_::STGFULL || i == C_::STGFULL + 1) count = HALF_WARPS;
      if (i == C_::QFULL || i == C_::QFULL + 1) count = 2;       // the tile's bytes and its statistics
      mbar_init(bar(i), count);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_do) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_dq) : "memory");
  }
  if (warp == B3_ROW_WARPS) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  fax_grid_dependency_wait();
  const uint32_t tm_s = tmem, tm_dp = tmem + 128, tm_dv = tmem + 256, tm_dk = tmem + 384;
  const uint32_t k_s = base + C_::K_OFF, v_s = base + C_::V_OFF, ds_s = base + C_::DS_OFF;
  auto q_s = [&](uint32_t i) { return base + C_::Q_OFF + i * C_::TILE_BYTES; };
  auto do_s = [&](uint32_t i) { return base + C_::DO_OFF + i * C_::TILE_BYTES; };
  float* stat = reinterpret_cast<float*>(gbase + C_::STAT_OFF);

  if (warp == B3_ROW_WARPS + 1) {
    // ---------------- TMA producer (lane 0) and statistics loader (all lanes) ----------------
    // Statistics of a tile are requested one tile ahead, so the global-memory latency is not in the loop.
    auto stat_ptr = [&](const float* src, int t, int it) -> const float4* {
      const int kj = t / bh_count, bh = t % bh_count;
      return reinterpret_cast<const float4*>(src + (long long)bh * p.T + (kj + it) * 128) + lane;
    };
    uint32_t gs = 0;
    bool ok = true;
    int it_n = 0;
    float4 l_next = make_float4(0.f, 0.f, 0.f, 0.f), d_next = l_next;
    if ((int)blockIdx.x < n_items) { l_next = *stat_ptr(p.lse, blockIdx.x, 0); d_next = *stat_ptr(p.Dv, blockIdx.x, 0); }
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
      const int kj = t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int row0 = b * p.T;
      const int qcol = h * HD, kcol = d + h * HD, vcol = 2 * d + h * HD;
      const int nsteps = nq - kj;
      for (int it = 0; it < nsteps; ++it, ++gs) {
        const int qrow = row0 + (kj + it) * 128;
        const uint32_t sq = gs & 1u;
        float4 l_cur = l_next;
        const float4 d_cur = d_next;
        if (it + 1 < nsteps) { l_next = *stat_ptr(p.lse, t, it + 1); d_next = *stat_ptr(p.Dv, t, it + 1); }
        else if (t + (int)gridDim.x < n_items) { l_next = *stat_ptr(p.lse, t + gridDim.x, 0); d_next = *stat_ptr(p.Dv, t + gridDim.x, 0); }
        if (!mbar_wait_warp(bar(C_::QFREE + sq), ((gs >> 1) & 1u) ^ 1u, abort_flag, p.status, 342)) { ok = false; break; }
        if (lane == 0) {
          mbar_expect_tx(bar(C_::QFULL + sq), C_::TILE_BYTES);
#pragma unroll
          for (int i = 0; i < HD / 64; ++i) tma_load_2d(q_s(sq) + i * 16384, &tmap_qkv, bar(C_::QFULL + sq), qcol + 64 * i, qrow);
        }
        l_cur.x *= 1.4426950408889634f; l_cur.y *= 1.4426950408889634f; l_cur.z *= 1.4426950408889634f; l_cur.w *= 1.4426950408889634f;
        *reinterpret_cast<float4*>(stat + sq * 256 + 4 * lane) = l_cur;
        *reinterpret_cast<float4*>(stat + sq * 256 + 128 + 4 * lane) = d_cur;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::QFULL + sq));
        if (it == 0) {
          if (!mbar_wait_warp(bar(C_::KVFREE), (uint32_t)(it_n & 1) ^ 1u, abort_flag, p.status, 341)) { ok = false; break; }
          if (lane == 0) {
            mbar_expect_tx(bar(C_::KVFULL), 2 * C_::TILE_BYTES);
#pragma unroll
            for (int i = 0; i < HD / 64; ++i) {
              tma_load_2d(k_s + i * 16384, &tmap_qkv, bar(C_::KVFULL), kcol + 64 * i, row0 + kj * 128);
              tma_load_2d(v_s + i * 16384, &tmap_qkv, bar(C_::KVFULL), vcol + 64 * i, row0 + kj * 128);
            }
          }
        }
        // the dO stage of this parity staged half of the dQ tile two tiles back: its reduction must have read it
        if (!mbar_wait_warp(bar(C_::STGFREE_DO + sq), ((gs >> 1) & 1u) ^ 1u, abort_flag, p.status, 356)) { ok = false; break; }
        if (!mbar_wait_warp(bar(C_::DOFREE + sq), ((gs >> 1) & 1u) ^ 1u, abort_flag, p.status, 343)) { ok = false; break; }
        if (lane == 0) {
          mbar_expect_tx(bar(C_::DOFULL + sq), C_::TILE_BYTES);
#pragma unroll
          for (int i = 0; i < HD / 64; ++i) tma_load_2d(do_s(sq) + i * 16384, &tmap_do, bar(C_::DOFULL + sq), qcol + 64 * i, qrow);
        }
      }
    }
    if (!ok && lane == 0) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
  } else if (warp == B3_ROW_WARPS) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, false, false);      // S^T, dP^T: both operands K-major
      const uint32_t idesc_acc = idesc_bf16(HD, false, true);      // dV, dK: A in tensor memory, B MN-major
      // dQ^T = K^T dS^T (128 x 128) at head_dim 128; dQ = dS K (128 queries x 64) at head_dim 64, where the
      // transposed form would have only 64 rows: both operands MN-major either way
      const uint32_t idesc_dq = idesc_bf16(HD == 128 ? 128 : 64, true, true);
      // A descriptor = {low word, high word}; only the 14-bit start-address field (16-byte units) of the
      // low word changes between stages and k-steps.  K-major tiles: a k-step is 32 bytes inside a
      // 64-column panel (panels 16 KB apart); MN-major: a k-step is 16 rows (2048 bytes).
      const uint32_t hi = (uint32_t)(smem_desc(0, 16, 1024) >> 32);
      const uint32_t k_kmaj = (uint32_t)smem_desc(k_s, 16, 1024), v_kmaj = (uint32_t)smem_desc(v_s, 16, 1024);
      const uint32_t k_mn = (uint32_t)smem_desc(k_s, 16384, 1024), ds_mn = (uint32_t)smem_desc(ds_s, 16384, 1024);
      const uint32_t q_kmaj0 = (uint32_t)smem_desc(q_s(0), 16, 1024), q_mn0 = (uint32_t)smem_desc(q_s(0), 16384, 1024);
      const uint32_t do_kmaj0 = (uint32_t)smem_desc(do_s(0), 16, 1024), do_mn0 = (uint32_t)smem_desc(do_s(0), 16384, 1024);
      auto mk = [&](uint32_t lo) -> uint64_t { return ((uint64_t)hi << 32) | lo; };
      constexpr uint32_t TILE16 = C_::TILE_BYTES >> 4;
      bool ok = true;
      auto issue_s = [&](uint32_t g) -> bool {
        const uint32_t sq = g & 1u;
        if (!mbar_wait(bar(C_::QFULL + sq), (g >> 1) & 1u, abort_flag, p.status, 344)) return false;
        tc_fence_after();
        const uint32_t bq = q_kmaj0 + sq * TILE16;
#pragma unroll
        for (int s = 0; s < HD / 16; ++s)
          tc_mma_bf16(tm_s, mk(k_kmaj + (s / 4) * 1024 + (s % 4) * 2), mk(bq + (s / 4) * 1024 + (s % 4) * 2), idesc_s, s ? 1u : 0u);
        tc_commit(bar(C_::SFULL));
        return true;
      };
      // A k-step of P^T / dS^T in tensor memory: 16 queries = 8 columns inside the quarter's 32
      auto acol = [](int k) { return (uint32_t)(32 * (k / 2) + 8 * (k % 2)); };
      uint32_t gs = 0;
      int it_n = 0;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
        const int kj = t / bh_count;
        const uint32_t nsteps = (uint32_t)(nq - kj);
        if (!mbar_wait(bar(C_::KVFULL), (uint32_t)(it_n & 1), abort_flag, p.status, 349)) { ok = false; break; }
        if (!issue_s(gs)) { ok = false; break; }
        for (uint32_t it = 0; it < nsteps; ++it, ++gs) {
          const uint32_t ph = gs & 1u, sq = gs & 1u;
          // dP^T = V dO^T (its columns held the dQ^T of the tile before: wait until that was read out)
          const uint32_t do_kmaj = do_kmaj0 + sq * TILE16, do_mn = do_mn0 + sq * TILE16;
          if (!mbar_wait(bar(C_::DOFULL + sq), (gs >> 1) & 1u, abort_flag, p.status, 345)) { ok = false; break; }
          if (gs > 0 && !mbar_wait(bar(C_::DQREAD), ph ^ 1u, abort_flag, p.status, 348)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int s = 0; s < HD / 16; ++s)
            tc_mma_bf16(tm_dp, mk(v_kmaj + (s / 4) * 1024 + (s % 4) * 2), mk(do_kmaj + (s / 4) * 1024 + (s % 4) * 2), idesc_s,
                        s ? 1u : 0u);
          tc_commit(bar(C_::DPFULL));
          // dV += P^T dO, a query half at a time (the first product of a key tile overwrites: dV and dK of
          // the tile before must have been read out)
          if (!mbar_wait(bar(C_::PREADY), ph, abort_flag, p.status, 346)) { ok = false; break; }
          if (it == 0 && !mbar_wait(bar(C_::DKVREAD), (uint32_t)(it_n & 1) ^ 1u, abort_flag, p.status, 350)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_bf16_ts(tm_dv, tm_s + acol(k), mk(do_mn + k * 128), idesc_acc, (it | (uint32_t)k) ? 1u : 0u);
          if (!mbar_wait(bar(C_::PREADY + 1), ph, abort_flag, p.status, 346)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 4; k < 8; ++k) tc_mma_bf16_ts(tm_dv, tm_s + acol(k), mk(do_mn + k * 128), idesc_acc, 1u);
          tc_commit(bar(C_::DOFREE + sq));
          // dK += dS^T Q, first query half
          const uint32_t bq = q_mn0 + sq * TILE16;
          if (!mbar_wait(bar(C_::DSREADY), ph, abort_flag, p.status, 347)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_bf16_ts(tm_dk, tm_s + 16u + acol(k), mk(bq + k * 128), idesc_acc, (it | (uint32_t)k) ? 1u : 0u);
          // all of dS^T is there: dQ^T = K^T dS^T over the dP^T columns (read by now), then the rest of dK
          if (!mbar_wait(bar(C_::DSREADY + 1), ph, abort_flag, p.status, 347)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (HD == 128) tc_mma_bf16(tm_dp, mk(k_mn + k * 128), mk(ds_mn + k * 128), idesc_dq, k ? 1u : 0u);
            else tc_mma_bf16(tm_dp, mk(ds_mn + k * 128), mk(k_mn + k * 128), idesc_dq, k ? 1u : 0u);
          }
          tc_commit(bar(C_::DQFULL));
#pragma unroll
          for (int k = 4; k < 8; ++k) tc_mma_bf16_ts(tm_dk, tm_s + 16u + acol(k), mk(bq + k * 128), idesc_acc, 1u);
          tc_commit(bar(C_::QFREE + sq));
          if (it + 1 == nsteps) {
            tc_commit(bar(C_::KVFREE));
            tc_commit(bar(C_::ALLDONE));         // every product of this key tile is complete: dV and dK are final
          } else if (!issue_s(gs + 1)) { ok = false; break; }
        }
      }
    }
  } else if (warp == B3_ROW_WARPS + 2) {
    // ---------------- dQ reduction issuer ----------------
    if (lane == 0) {
      uint32_t gs = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x) {
        const int kj = t / bh_count, bh = t % bh_count;
        const int b = bh / p.H, h = bh % p.H;
        const int nsteps = nq - kj;
        for (int it = 0; it < nsteps; ++it, ++gs) {
          const int qrow = b * p.T + (kj + it) * 128;
          const uint32_t sq = gs & 1u;
          // second query half first: its staging bytes (the dS^T tile) are needed again soonest
          if (!mbar_wait(bar(C_::STGFULL + 1), gs & 1u, abort_flag, p.status, 351)) { ok = false; break; }
#pragma unroll
          for (int i = 0; i < HD / 32; ++i) tma_reduce_add_2d(&tmap_dq, ds_s + i * 8192, h * HD + 32 * i, qrow + 64);   // boxes of 64 rows x 32 floats
          bulk_commit_group();
          if (!mbar_wait(bar(C_::STGFULL), gs & 1u, abort_flag, p.status, 351)) { ok = false; break; }
#pragma unroll
          for (int i = 0; i < HD / 32; ++i) tma_reduce_add_2d(&tmap_dq, do_s(sq) + i * 8192, h * HD + 32 * i, qrow);
          bulk_commit_group();
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          mbar_arrive(bar(C_::STGFREE_DS));
          bulk_wait_read_all();
          mbar_arrive(bar(C_::STGFREE_DO + sq));
        }
      }
      bulk_wait_all();
    }
  } else {
    // ---- row threads: key row kr (dQ^T read-out: head column kr), query quarter qr ----
    const uint32_t qr = (uint32_t)warp >> 2;              // queries 32 qr .. 32 qr + 31 of the tile
    const uint32_t half = qr >> 1;
    const int kr = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    // dS^T row of this key in the query half's panel; the 64 bytes of this quarter are chunks 4 (qr & 1) ..
    uint8_t* ds_row = gbase + C_::DS_OFF + half * 16384 + kr * 128;
    // dQ staging: the box of this warp's 32 head columns, in the buffer that takes this thread's query half
    // (dO stage 0, or the dS^T tile)
    uint8_t* stg_box = gbase + (half ? C_::DS_OFF : C_::DO_OFF) + (warp & 3) * 8192 + (lane & 3) * 4;
    uint32_t gs = 0;
    bool ok = true;
    int it_n = 0;
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
      const int kj = t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int row0 = b * p.T;
      const int nsteps = nq - kj;
      for (int it = 0; it < nsteps; ++it, ++gs) {
        const uint32_t ph = gs & 1u, sq = gs & 1u;
        const float* st_l = stat + sq * 256 + 32 * qr;
        const float* st_d = st_l + 128;
        uint32_t pp[16];
        // ---- P^T = exp(S^T / sqrt(hd) - LSE[q]) ----
        if (!mbar_wait_warp(bar(C_::QFULL + sq), (gs >> 1) & 1u, abort_flag, p.status, 352)) { ok = false; break; }
        if (!mbar_wait_warp(bar(C_::SFULL), ph, abort_flag, p.status, 353)) { ok = false; break; }
        tc_fence_after();
        {
          uint32_t sv[32];
          tc_ld32(tm_s + lane_base + 32u * qr, sv);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(st_l + e);
            float p0 = ex2_approx(__uint_as_float(sv[e]) * p.scale_log2 - l4.x);
            float p1 = ex2_approx(__uint_as_float(sv[e + 1]) * p.scale_log2 - l4.y);
            float p2 = ex2_approx(__uint_as_float(sv[e + 2]) * p.scale_log2 - l4.z);
            float p3 = ex2_approx(__uint_as_float(sv[e + 3]) * p.scale_log2 - l4.w);
            if (it == 0) {                   // diagonal tile: a query before the key is masked
              const int q0 = 32 * (int)qr + e;
              if (q0 < kr) p0 = 0.f;
              if (q0 + 1 < kr) p1 = 0.f;
              if (q0 + 2 < kr) p2 = 0.f;
              if (q0 + 3 < kr) p3 = 0.f;
            }
            __nv_bfloat162 h0 = __floats2bfloat162_rn(p0, p1), h1 = __floats2bfloat162_rn(p2, p3);
            pp[e >> 1] = *reinterpret_cast<uint32_t*>(&h0);
            pp[(e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h1);
          }
        }
        tc_st16(tm_s + lane_base + 32u * qr, pp);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::PREADY + half));
        // ---- dS^T = P^T * (dP^T - D[q]), from the bf16 P^T that the products use ----
        if (!mbar_wait_warp(bar(C_::DPFULL), ph, abort_flag, p.status, 354)) { ok = false; break; }
        tc_fence_after();
        {
          uint32_t dv[32], dd[16];
          tc_ld32(tm_dp + lane_base + 32u * qr, dv);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 d4 = *reinterpret_cast<const float4*>(st_d + e);
            const float2 pa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pp[e >> 1]));
            const float2 pb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pp[(e >> 1) + 1]));
            __nv_bfloat162 h0 = __floats2bfloat162_rn(pa.x * (__uint_as_float(dv[e]) - d4.x),
                                                      pa.y * (__uint_as_float(dv[e + 1]) - d4.y));
            __nv_bfloat162 h1 = __floats2bfloat162_rn(pb.x * (__uint_as_float(dv[e + 2]) - d4.z),
                                                      pb.y * (__uint_as_float(dv[e + 3]) - d4.w));
            dd[e >> 1] = *reinterpret_cast<uint32_t*>(&h0);
            dd[(e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h1);
          }
          tc_st16(tm_s + lane_base + 32u * qr + 16u, dd);
          // the dS^T tile staged the second half of the dQ tile before: its reduction must have read it
          if (gs > 0 && !mbar_wait_warp(bar(C_::STGFREE_DS), ph ^ 1u, abort_flag, p.status, 358)) { ok = false; break; }
#pragma unroll
          for (int k = 0; k < 4; ++k)
            *reinterpret_cast<uint4*>(ds_row + (((4 * (int)(qr & 1u) + k) ^ (kr & 7)) << 4)) =
                make_uint4(dd[4 * k], dd[4 * k + 1], dd[4 * k + 2], dd[4 * k + 3]);
        }
        fence_proxy_async();
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::DSREADY + half));
        // ---- dQ^T (lane = head column kr, this quarter's 32 queries) -> staging boxes (row = query) ----
        if (!mbar_wait_warp(bar(C_::DQFULL), ph, abort_flag, p.status, 355)) { ok = false; break; }
        tc_fence_after();
        if (HD == 128) {
          uint32_t v[32];
          tc_ld32(tm_dp + lane_base + 32u * qr, v);
          tc_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::DQREAD));
          // first half -> this tile's dO stage (dV, issued before dQ^T, is complete); second half -> the dS^T
          // tile (the dQ^T product has read it)
          uint8_t* box = stg_box + (half ? 0u : sq * C_::TILE_BYTES);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int q = 32 * (int)(qr & 1u) + j;
            *reinterpret_cast<uint32_t*>(box + q * 128 + (((lane >> 2) ^ (q & 7)) << 4)) = v[j];
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::STGFULL + half));
        } else {
          // head_dim 64: dQ (lane = query row kr, 64 head columns); this thread takes columns 16 qr .. 16 qr + 15.
          // Query rows 0..63 (lane quarters 0, 1) are staged in the dO stage, rows 64..127 in the dS^T tile,
          // each as two boxes of 64 rows x 32 floats.
          uint32_t v[16];
          tc_ld16(tm_dp + lane_base + 16u * qr, v);
          tc_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::DQREAD));
          const uint32_t qhalf = (uint32_t)(warp & 3) >> 1;
          const int r = kr & 63;
          uint8_t* box = gbase + (qhalf ? (uint32_t)C_::DS_OFF : (uint32_t)C_::DO_OFF + sq * C_::TILE_BYTES) + (qr >> 1) * 8192 + r * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            *reinterpret_cast<uint4*>(box + (((4 * (int)(qr & 1u) + k) ^ (r & 7)) << 4)) =
                make_uint4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_::STGFULL + qhalf));
        }
      }
      if (!ok) break;
      if (!mbar_wait_warp(bar(C_::ALLDONE), (uint32_t)(it_n & 1), abort_flag, p.status, 357)) { ok = false; break; }
      tc_fence_after();
      {
        constexpr int CW = HD / 4;                 // head columns per thread: 32 or 16
        const long long tok = (long long)row0 + kj * 128 + kr;
        bf16* dk_row = p.dqkv + tok * 3 * d + d + h * HD + CW * qr;
        bf16* dv_row = p.dqkv + tok * 3 * d + 2 * d + h * HD + CW * qr;
        uint32_t kv[CW], vv[CW];
        if (HD == 128) {
          tc_ld32(tm_dk + lane_base + 32u * qr, reinterpret_cast<uint32_t(&)[32]>(kv));
          tc_ld32(tm_dv + lane_base + 32u * qr, reinterpret_cast<uint32_t(&)[32]>(vv));
        } else {
          tc_ld16(tm_dk + lane_base + 16u * qr, reinterpret_cast<uint32_t(&)[16]>(kv));
          tc_ld16(tm_dv + lane_base + 16u * qr, reinterpret_cast<uint32_t(&)[16]>(vv));
        }
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::DKVREAD));
#pragma unroll
        for (int c = 0; c < CW; c += 16) {        // 16 columns = one 32-byte sector per store
          U8 uk, uv;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            __nv_bfloat162 hk = __floats2bfloat162_rn(__uint_as_float(kv[c + 2 * e]) * p.scale, __uint_as_float(kv[c + 2 * e + 1]) * p.scale);
            __nv_bfloat162 hv = __floats2bfloat162_rn(__uint_as_float(vv[c + 2 * e]), __uint_as_float(vv[c + 2 * e + 1]));
            uk.w[e] = *reinterpret_cast<uint32_t*>(&hk);
            uv.w[e] = *reinterpret_cast<uint32_t*>(&hv);
          }
          st_global_v8(dk_row + c, uk);
          st_global_v8(dv_row + c, uv);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == B3_ROW_WARPS) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

}  // namespace

bool fax_attention_bwd3_supported(int B, int T, int H, int hd) {
  return (hd == 128 || hd == 64) && T % 128 == 0 && B > 0 && H > 0;
}

namespace {
template <int HD>
fax_status launch_bwd3(fax_ctx* ctx, int B, int T, int H, const void* qkv, const float* lse, const void* d_o,
                       void* dqkv, const float* Dv, float* dq_acc) {
  CUtensorMap mq, md, mdq;
  const uint64_t d = (uint64_t)H * HD;
  const uint64_t n_tok = (uint64_t)B * T;
  if (!make_map(ctx, &mq, qkv, 3 * d, n_tok, 3 * d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map(ctx, &md, d_o, d, n_tok, d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map_f32(ctx, &mdq, dq_acc, d, n_tok, d, 32, 64)) return FAX_ERR_INVALID_ARG;
  Bwd3Params p;
  p.B = B; p.T = T; p.H = H; p.lse = lse; p.Dv = Dv; p.dqkv = (bf16*)dqkv;
  p.scale = 1.0f / sqrtf((float)HD);
  p.scale_log2 = 1.4426950408889634f * p.scale;
  p.status = ctx->dev_status;
  static bool attr_set[FAX_MAX_DEVICES] = {};
  FAX_TRY(fax_opt_in_shared_memory(ctx, attn_bwd3_tc_kernel<HD>, B3<HD>::SMEM_BYTES, attr_set));
  const long long items = (long long)B * H * (T / 128);
  const int grid = (int)(items < ctx->sm_count ? items : ctx->sm_count);
  fax_launch(ctx, attn_bwd3_tc_kernel<HD>, dim3(grid), dim3(B3_THREADS), B3<HD>::SMEM_BYTES, mq, md, mdq, p);
  return fax_after_launch(ctx);
}
}  // namespace

// The main kernel only: D = rowsum(dO o O) must be in Dv and dq_acc cleared (both by the row-dot
// kernel), and dq_acc is converted to bf16 by the caller afterwards.
fax_status fax_attention_bwd3_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const float* lse,
                                 const void* d_o, void* dqkv, const float* Dv, float* dq_acc) {
  return hd == 128 ? launch_bwd3<128>(ctx, B, T, H, qkv, lse, d_o, dqkv, Dv, dq_acc)
                   : launch_bwd3<64>(ctx, B, T, H, qkv, lse, d_o, dqkv, Dv, dq_acc);
}
