// Causal attention backward (step B5), head_dim 64: two score tiles in flight.
//
// Same decomposition as the sixteen-row-warp kernel (a CTA owns a 128-key tile j with K_j, V_j resident
// and walks the 128-query tiles i >= j; S^T = K_j Q_i^T and dP^T = V_j dO_i^T with the keys in the
// tensor-memory lanes; P^T and dS^T written back as bf16 over the S^T columns as the A operands of
// dV_j += P^T dO_i and dK_j += dS^T Q_i; dQ_i = dS K_j with the queries in the lanes, added into a
// float32 accumulator by bulk tensor reductions).  At head_dim 64 dV and dK take 64 tensor-memory
// columns each, which leaves room for a SECOND S^T accumulator:
//   [0,128) S^T even tiles   [128,256) S^T odd tiles   [256,384) dP^T, then dQ (64 columns)
//   [384,448) dV             [448,512) dK
// so the row warps run the exponentials of a later tile while the tensor core works on tile g.  One
// iteration of the sixteen row warps (thread = key row, a quarter of the tile's queries):
//   C  dQ of tile g -> staging buffer in shared memory -> reduction warp   (waits for the dQ product only)
//   A  P^T of tile g + 2         (S^T(g+2) follows dQ(g) and dK(g), whose dS^T operand shares its buffer)
//   B  dS^T of tile g + 1        (needs dP^T(g+1), issued when C freed its columns; done while A ran)
// and of the MMA thread, after B of tile g:
//   dQ(g), dK(g), S^T(g+2) | dP^T(g+1) after C | dV(g+2) after A
// Each hand-off barrier completes once per tile and its waiter is never two phases behind (the producer
// of phase n + 1 depends, through another barrier, on the consumer having passed phase n); "P ready"
// alternates between two barriers because at the start of a key tile two S^T products are issued
// before the first of them is waited for.
// K and V of the next key tile are prefetched into a second buffer while the current one is walked, and
// the MMA thread issues the next key tile's first two S^T products right after the last products of the
// current one, so the row warps find their scores ready when they come back from the dV / dK read-out.
// Shared memory: two (K, V) buffers, three Q stages (a Q tile lives from S^T, two iterations ahead, to
// dK), two dO stages, the dS tile (B operand of dQ), a 32 KB dQ staging buffer, per-stage query
// statistics.  Every wait is bounded.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int B4_HD = 64;
constexpr int B4_ROW_WARPS = 16;
constexpr int B4_THREADS = 32 * (B4_ROW_WARPS + 3);   // + MMA warp, TMA / statistics warp, dQ reduction warp

struct Bwd4Params {
  int B, T, H;
  const float* lse; const float* Dv;
  bf16* dqkv;
  float scale, scale_log2;
  int32_t* status;
};

struct B4 {
  static constexpr int TILE_BYTES = 128 * B4_HD * 2;      // one panel of 128 rows x 128 B
  static constexpr int KV_OFF = 0;                        // two buffers of (K, V): the next key tile is prefetched
  static constexpr int Q_OFF = 4 * TILE_BYTES;            // three stages
  static constexpr int DO_OFF = 7 * TILE_BYTES;           // two stages
  static constexpr int DS_OFF = 9 * TILE_BYTES;           // dS^T: two panels (query halves) of 128 key rows x 128 B
  static constexpr int STG_OFF = DS_OFF + 32768;          // dQ staging: 4 boxes of 64 rows x 32 floats
  static constexpr int STAT_OFF = STG_OFF + 32768;        // [3 stages][0: log2e * lse, 1: D][128] floats
  static constexpr int BAR_OFF = STAT_OFF + 3 * 1024;
  static constexpr int KVFULL = 0 /* 2 */, KVFREE = 2 /* 2 */, QFULL = 4 /* 3 */, QFREE = 7 /* 3 */, DOFULL = 10 /* 2 */,
                       DOFREE = 12 /* 2 */, SFULL = 14 /* 2 */, DPFULL = 16, PREADY = 17 /* 2 */, DSREADY = 19, DQFULL = 20,
                       DQREAD = 21, STGFULL = 22, STGFREE = 23, ALLDONE = 24, DKVREAD = 25, NBARS = 26;
  static constexpr int LAYOUT_BYTES = BAR_OFF + NBARS * 8 + 16;
  static constexpr int SMEM_BYTES = LAYOUT_BYTES + 1024;
  static constexpr int TMEM_COLS = 512;
};
static_assert(B4::SMEM_BYTES <= 227 * 1024, "shared-memory layout does not fit");

__global__ void __launch_bounds__(B4_THREADS, 1)
attn_bwd4_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const __grid_constant__ CUtensorMap tmap_do,
                    const __grid_constant__ CUtensorMap tmap_dq, const Bwd4Params p) {
  using C_ = B4;
  constexpr int HD = B4_HD;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bars = base + C_::BAR_OFF;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(gbase + C_::BAR_OFF + C_::NBARS * 8);
  volatile int* abort_flag = (volatile int*)(gbase + C_::BAR_OFF + C_::NBARS * 8 + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / 128;
  const int bh_count = p.B * p.H;
  const int n_items = nq * bh_count;
  const int d = p.H * HD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C_::NBARS; ++i) {
      uint32_t count = 1;
      if (i == C_::PREADY || i == C_::PREADY + 1 || i == C_::DSREADY || i == C_::DQREAD || i == C_::DKVREAD || i == C_::STGFULL)
        count = B4_ROW_WARPS;
      if (i >= C_::QFULL && i < C_::QFULL + 3) count = 2;       // the tile's bytes and its statistics
      mbar_init(bar(i), count);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_do) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_dq) : "memory");
  }
  if (warp == B4_ROW_WARPS) tmem_alloc(smem_u32((const void*)tmem_slot), C_::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  fax_grid_dependency_wait();
  auto tm_s = [&](uint32_t g) { return tmem + 128u * (g & 1u); };
  const uint32_t tm_dp = tmem + 256, tm_dv = tmem + 384, tm_dk = tmem + 448;
  const uint32_t ds_s = base + C_::DS_OFF, stg_s = base + C_::STG_OFF;
  auto k_s = [&](uint32_t i) { return base + C_::KV_OFF + 2 * i * C_::TILE_BYTES; };
  auto v_s = [&](uint32_t i) { return base + C_::KV_OFF + (2 * i + 1) * C_::TILE_BYTES; };
  auto q_s = [&](uint32_t i) { return base + C_::Q_OFF + i * C_::TILE_BYTES; };
  auto do_s = [&](uint32_t i) { return base + C_::DO_OFF + i * C_::TILE_BYTES; };
  float* stat = reinterpret_cast<float*>(gbase + C_::STAT_OFF);

  if (warp == B4_ROW_WARPS + 1) {
    // ---------------- TMA producer (lane 0) and statistics loader (all lanes) ----------------
    // Statistics of a tile are requested one tile ahead, so the global-memory latency is not in the loop.
    auto stat_ptr = [&](const float* src, int t, int it) -> const float4* {
      const int kj = t / bh_count, bh = t % bh_count;
      return reinterpret_cast<const float4*>(src + (long long)bh * p.T + (kj + it) * 128) + lane;
    };
    // K, V of work item t (the CTA's item number n) into buffer n & 1, free once item n - 2 has finished
    auto load_kv = [&](int t, int n) -> bool {
      const uint32_t kb = (uint32_t)n & 1u;
      if (!mbar_wait_warp(bar(C_::KVFREE + kb), (((uint32_t)n >> 1) & 1u) ^ 1u, abort_flag, p.status, 441)) return false;
      if (lane == 0) {
        const int kj = t / bh_count, bh = t % bh_count;
        const int b = bh / p.H, h = bh % p.H;
        mbar_expect_tx(bar(C_::KVFULL + kb), 2 * C_::TILE_BYTES);
        tma_load_2d(k_s(kb), &tmap_qkv, bar(C_::KVFULL + kb), d + h * HD, b * p.T + kj * 128);
        tma_load_2d(v_s(kb), &tmap_qkv, bar(C_::KVFULL + kb), 2 * d + h * HD, b * p.T + kj * 128);
      }
      return true;
    };
    uint32_t gs = 0;
    bool ok = true;
    int it_n = 0;
    float4 l_next = make_float4(0.f, 0.f, 0.f, 0.f), d_next = l_next;
    if ((int)blockIdx.x < n_items) {
      l_next = *stat_ptr(p.lse, blockIdx.x, 0); d_next = *stat_ptr(p.Dv, blockIdx.x, 0);
      ok = load_kv(blockIdx.x, 0);
    }
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
      const int kj = t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int row0 = b * p.T;
      const int qcol = h * HD;
      const int nsteps = nq - kj;
      for (int it = 0; it < nsteps; ++it, ++gs) {
        const int qrow = row0 + (kj + it) * 128;
        const uint32_t s3 = gs % 3u, u3 = gs / 3u, s2 = gs & 1u, u2 = gs >> 1;
        float4 l_cur = l_next;
        const float4 d_cur = d_next;
        if (it + 1 < nsteps) { l_next = *stat_ptr(p.lse, t, it + 1); d_next = *stat_ptr(p.Dv, t, it + 1); }
        else if (t + (int)gridDim.x < n_items) { l_next = *stat_ptr(p.lse, t + gridDim.x, 0); d_next = *stat_ptr(p.Dv, t + gridDim.x, 0); }
        if (!mbar_wait_warp(bar(C_::QFREE + s3), (u3 & 1u) ^ 1u, abort_flag, p.status, 442)) { ok = false; break; }
        if (lane == 0) {
          mbar_expect_tx(bar(C_::QFULL + s3), C_::TILE_BYTES);
          tma_load_2d(q_s(s3), &tmap_qkv, bar(C_::QFULL + s3), qcol, qrow);
        }
        l_cur.x *= 1.4426950408889634f; l_cur.y *= 1.4426950408889634f; l_cur.z *= 1.4426950408889634f; l_cur.w *= 1.4426950408889634f;
        *reinterpret_cast<float4*>(stat + s3 * 256 + 4 * lane) = l_cur;
        *reinterpret_cast<float4*>(stat + s3 * 256 + 128 + 4 * lane) = d_cur;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::QFULL + s3));
        if (!mbar_wait_warp(bar(C_::DOFREE + s2), (u2 & 1u) ^ 1u, abort_flag, p.status, 443)) { ok = false; break; }
        if (lane == 0) {
          mbar_expect_tx(bar(C_::DOFULL + s2), C_::TILE_BYTES);
          tma_load_2d(do_s(s2), &tmap_do, bar(C_::DOFULL + s2), qcol, qrow);
        }
        // K, V of the next key tile, once this one's second query tile is requested (the first, if it has one)
        if (it == (nsteps > 1 ? 1 : 0) && t + (int)gridDim.x < n_items && !load_kv(t + gridDim.x, it_n + 1)) { ok = false; break; }
      }
    }
    if (!ok && lane == 0) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) { } }
  } else if (warp == B4_ROW_WARPS) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(128, false, false);      // S^T, dP^T: both operands K-major
      const uint32_t idesc_acc = idesc_bf16(HD, false, true);      // dV, dK: A in tensor memory, B MN-major
      const uint32_t idesc_dq = idesc_bf16(HD, true, true);        // dQ = dS K: both operands MN-major
      // A descriptor = {low word, high word}; only the start-address field (16-byte units) of the low word
      // changes between stages and k-steps.  K-major tiles: a k-step is 32 bytes inside the 64-column
      // panel; MN-major: a k-step is 16 rows (2048 bytes).
      const uint32_t hi = (uint32_t)(smem_desc(0, 16, 1024) >> 32);
      const uint32_t k_kmaj0 = (uint32_t)smem_desc(k_s(0), 16, 1024), v_kmaj0 = (uint32_t)smem_desc(v_s(0), 16, 1024);
      const uint32_t k_mn0 = (uint32_t)smem_desc(k_s(0), 16384, 1024), ds_mn = (uint32_t)smem_desc(ds_s, 16384, 1024);
      uint32_t k_kmaj = k_kmaj0, v_kmaj = v_kmaj0, k_mn = k_mn0;      // of the key tile being walked
      const uint32_t q_kmaj0 = (uint32_t)smem_desc(q_s(0), 16, 1024), q_mn0 = (uint32_t)smem_desc(q_s(0), 16384, 1024);
      const uint32_t do_kmaj0 = (uint32_t)smem_desc(do_s(0), 16, 1024), do_mn0 = (uint32_t)smem_desc(do_s(0), 16384, 1024);
      auto mk = [&](uint32_t lo) -> uint64_t { return ((uint64_t)hi << 32) | lo; };
      constexpr uint32_t TILE16 = C_::TILE_BYTES >> 4;
      // A k-step of P^T / dS^T in tensor memory: 16 queries = 8 columns inside the quarter's 32
      auto acol = [](int k) { return (uint32_t)(32 * (k / 2) + 8 * (k % 2)); };
      bool ok = true;
      auto issue_s = [&](uint32_t g, uint32_t kk) -> bool {         // kk: K (K-major words) of the key tile that tile g belongs to
        const uint32_t s3 = g % 3u;
        if (!mbar_wait(bar(C_::QFULL + s3), (g / 3u) & 1u, abort_flag, p.status, 444)) return false;
        tc_fence_after();
        const uint32_t bq = q_kmaj0 + s3 * TILE16;
#pragma unroll
        for (int s = 0; s < HD / 16; ++s) tc_mma_bf16(tm_s(g), mk(kk + s * 2), mk(bq + s * 2), idesc_s, s ? 1u : 0u);
        tc_commit(bar(C_::SFULL + (g & 1u)));
        return true;
      };
      auto issue_dv = [&](uint32_t g, bool first) -> bool {        // dV += P^T dO
        if (!mbar_wait(bar(C_::PREADY + (g & 1u)), (g >> 1) & 1u, abort_flag, p.status, 446)) return false;
        if (!mbar_wait(bar(C_::DOFULL + (g & 1u)), (g >> 1) & 1u, abort_flag, p.status, 445)) return false;
        tc_fence_after();
        const uint32_t do_mn = do_mn0 + (g & 1u) * TILE16;
#pragma unroll
        for (int k = 0; k < 8; ++k) tc_mma_bf16_ts(tm_dv, tm_s(g) + acol(k), mk(do_mn + k * 128), idesc_acc, (!first || k) ? 1u : 0u);
        return true;
      };
      auto issue_dp = [&](uint32_t g) -> bool {                    // dP^T = V dO^T over the columns dQ(g - 1) was read from
        if (g > 0 && !mbar_wait(bar(C_::DQREAD), (g - 1u) & 1u, abort_flag, p.status, 448)) return false;
        if (!mbar_wait(bar(C_::DOFULL + (g & 1u)), (g >> 1) & 1u, abort_flag, p.status, 445)) return false;
        tc_fence_after();
        const uint32_t do_kmaj = do_kmaj0 + (g & 1u) * TILE16;
#pragma unroll
        for (int s = 0; s < HD / 16; ++s) tc_mma_bf16(tm_dp, mk(v_kmaj + s * 2), mk(do_kmaj + s * 2), idesc_s, s ? 1u : 0u);
        tc_commit(bar(C_::DPFULL));
        tc_commit(bar(C_::DOFREE + (g & 1u)));                     // dV(g) was issued before: the dO stage is done with
        return true;
      };
      uint32_t gs = 0;
      int it_n = 0;
      // S^T of the first two query tiles of work item t (number n of this CTA, first tile g), K from buffer n & 1
      auto open_item = [&](int t, int n, uint32_t g) -> bool {
        const uint32_t kb = (uint32_t)n & 1u;
        if (!mbar_wait(bar(C_::KVFULL + kb), ((uint32_t)n >> 1) & 1u, abort_flag, p.status, 449)) return false;
        const uint32_t kk = k_kmaj0 + kb * 2 * TILE16;
        return issue_s(g, kk) && (nq - t / bh_count < 2 || issue_s(g + 1, kk));
      };
      if ((int)blockIdx.x < n_items && !open_item(blockIdx.x, 0, 0)) ok = false;
      for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
        const int kj = t / bh_count;
        const uint32_t nsteps = (uint32_t)(nq - kj);
        const uint32_t kb = (uint32_t)it_n & 1u;
        k_kmaj = k_kmaj0 + kb * 2 * TILE16; v_kmaj = v_kmaj0 + kb * 2 * TILE16; k_mn = k_mn0 + kb * 2 * TILE16;
        // the first dV product of a key tile overwrites: dV and dK of the tile before must have been read out
        if (!mbar_wait(bar(C_::DKVREAD), (uint32_t)(it_n & 1) ^ 1u, abort_flag, p.status, 450)) { ok = false; break; }
        if (!issue_dv(gs, true)) { ok = false; break; }
        if (!issue_dp(gs)) { ok = false; break; }
        if (nsteps > 1 && !issue_dv(gs + 1, false)) { ok = false; break; }
        for (uint32_t it = 0; it < nsteps; ++it, ++gs) {
          if (!mbar_wait(bar(C_::DSREADY), gs & 1u, abort_flag, p.status, 447)) { ok = false; break; }
          tc_fence_after();
          const uint32_t bq = q_mn0 + (gs % 3u) * TILE16;
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_bf16(tm_dp, mk(ds_mn + k * 128), mk(k_mn + k * 128), idesc_dq, k ? 1u : 0u);
          tc_commit(bar(C_::DQFULL));
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_bf16_ts(tm_dk, tm_s(gs) + 16u + acol(k), mk(bq + k * 128), idesc_acc, (it | (uint32_t)k) ? 1u : 0u);
          tc_commit(bar(C_::QFREE + gs % 3u));
          if (it + 1 == nsteps) {
            tc_commit(bar(C_::KVFREE + kb));
            tc_commit(bar(C_::ALLDONE));         // every product of this key tile is complete: dV and dK are final
            // the next key tile's first scores, ready when the row warps come back from the read-out
            if (t + (int)gridDim.x < n_items && !open_item(t + gridDim.x, it_n + 1, gs + 1)) { ok = false; break; }
            continue;
          }
          if (it + 2 < nsteps && !issue_s(gs + 2, k_kmaj)) { ok = false; break; }
          if (!issue_dp(gs + 1)) { ok = false; break; }
          if (it + 2 < nsteps && !issue_dv(gs + 2, false)) { ok = false; break; }
        }
      }
    }
  } else if (warp == B4_ROW_WARPS + 2) {
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
          if (!mbar_wait(bar(C_::STGFULL), gs & 1u, abort_flag, p.status, 451)) { ok = false; break; }
#pragma unroll
          for (int i = 0; i < 4; ++i)             // boxes of 64 rows x 32 floats: (row half i / 2, column half i % 2)
            tma_reduce_add_2d(&tmap_dq, stg_s + i * 8192, h * HD + 32 * (i & 1), qrow + 64 * (i >> 1));
          bulk_commit_group();
          bulk_wait_read_all();                   // the buffer has been read: the next tile may be staged
          mbar_arrive(bar(C_::STGFREE));
        }
      }
      bulk_wait_all();
    }
  } else {
    // ---- row threads: key row kr (dQ read-out: query row kr), query quarter qr ----
    const uint32_t qr = (uint32_t)warp >> 2;              // queries 32 qr .. 32 qr + 31 of the tile
    const uint32_t half = qr >> 1;
    const int kr = 32 * (warp & 3) + lane;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    // dS^T row of this key in the query half's panel; the 64 bytes of this quarter are chunks 4 (qr & 1) ..
    uint8_t* ds_row = gbase + C_::DS_OFF + half * 16384 + kr * 128;
    uint32_t gs = 0;
    bool ok = true;
    int it_n = 0;
    // A: P^T = exp(S^T / sqrt(hd) - LSE[q]) of tile g (diag: the key tile's own query tile, where a query
    // before the key is masked)
    auto phase_p = [&](uint32_t g, bool diag) -> bool {
      const uint32_t s3 = g % 3u;
      const float* st_l = stat + s3 * 256 + 32 * qr;
      if (!mbar_wait_warp(bar(C_::QFULL + s3), (g / 3u) & 1u, abort_flag, p.status, 452)) return false;
      if (!mbar_wait_warp(bar(C_::SFULL + (g & 1u)), (g >> 1) & 1u, abort_flag, p.status, 453)) return false;
      tc_fence_after();
      uint32_t sv[32], pp[16];
      tc_ld32(tm_s(g) + lane_base + 32u * qr, sv);
      tc_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; e += 4) {
        const float4 l4 = *reinterpret_cast<const float4*>(st_l + e);
        float p0 = ex2_approx(__uint_as_float(sv[e]) * p.scale_log2 - l4.x);
        float p1 = ex2_approx(__uint_as_float(sv[e + 1]) * p.scale_log2 - l4.y);
        float p2 = ex2_approx(__uint_as_float(sv[e + 2]) * p.scale_log2 - l4.z);
        float p3 = ex2_approx(__uint_as_float(sv[e + 3]) * p.scale_log2 - l4.w);
        if (diag) {
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
      tc_st16(tm_s(g) + lane_base + 32u * qr, pp);
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::PREADY + (g & 1u)));
      return true;
    };
    // C: dQ of tile g (lane = query row kr, columns 16 qr .. 16 qr + 15) -> the staging buffer as four boxes
    // of 64 rows x 32 floats (row half, column half)
    auto phase_dq = [&](uint32_t g) -> bool {
      if (!mbar_wait_warp(bar(C_::DQFULL), g & 1u, abort_flag, p.status, 455)) return false;
      tc_fence_after();
      uint32_t v[16];
      tc_ld16(tm_dp + lane_base + 16u * qr, v);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::DQREAD));
      // the reduction of the tile before has read the buffer
      if (g > 0 && !mbar_wait_warp(bar(C_::STGFREE), (g - 1u) & 1u, abort_flag, p.status, 456)) return false;
      const int r = kr & 63;
      uint8_t* box = gbase + C_::STG_OFF + (2u * ((uint32_t)kr >> 6) + (qr >> 1)) * 8192u + r * 128;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        *reinterpret_cast<uint4*>(box + (((4 * (int)(qr & 1u) + k) ^ (r & 7)) << 4)) =
            make_uint4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::STGFULL));
      return true;
    };
    // B: dS^T = P^T * (dP^T - D[q]) of tile g, from the bf16 P^T that the products use
    auto phase_ds = [&](uint32_t g) -> bool {
      const float* st_d = stat + (g % 3u) * 256 + 128 + 32 * qr;
      if (!mbar_wait_warp(bar(C_::DPFULL), g & 1u, abort_flag, p.status, 454)) return false;
      tc_fence_after();
      uint32_t dv[32], pp[16], dd[16];
      tc_ld32(tm_dp + lane_base + 32u * qr, dv);
      tc_ld16(tm_s(g) + lane_base + 32u * qr, pp);
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
      tc_st16(tm_s(g) + lane_base + 32u * qr + 16u, dd);
      // the dS tile in shared memory was the B operand of dQ(g - 1): complete, its read-out (C) came first
#pragma unroll
      for (int k = 0; k < 4; ++k)
        *reinterpret_cast<uint4*>(ds_row + (((4 * (int)(qr & 1u) + k) ^ (kr & 7)) << 4)) =
            make_uint4(dd[4 * k], dd[4 * k + 1], dd[4 * k + 2], dd[4 * k + 3]);
      fence_proxy_async();
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C_::DSREADY));
      return true;
    };
    for (int t = blockIdx.x; t < n_items && ok; t += gridDim.x, ++it_n) {
      const int kj = t / bh_count, bh = t % bh_count;
      const int b = bh / p.H, h = bh % p.H;
      const int row0 = b * p.T;
      const int nsteps = nq - kj;
      if (!phase_p(gs, true)) { ok = false; break; }
      if (nsteps > 1 && !phase_p(gs + 1, false)) { ok = false; break; }
      if (!phase_ds(gs)) { ok = false; break; }
      for (int it = 0; it < nsteps; ++it, ++gs) {
        if (!phase_dq(gs)) { ok = false; break; }
        if (it + 2 < nsteps && !phase_p(gs + 2, false)) { ok = false; break; }
        if (it + 1 < nsteps && !phase_ds(gs + 1)) { ok = false; break; }
      }
      if (!ok) break;
      if (!mbar_wait_warp(bar(C_::ALLDONE), (uint32_t)(it_n & 1), abort_flag, p.status, 457)) { ok = false; break; }
      tc_fence_after();
      {
        constexpr int CW = HD / 4;                 // head columns per thread
        const long long tok = (long long)row0 + kj * 128 + kr;
        bf16* dk_row = p.dqkv + tok * 3 * d + d + h * HD + CW * qr;
        bf16* dv_row = p.dqkv + tok * 3 * d + 2 * d + h * HD + CW * qr;
        uint32_t kv[CW], vv[CW];
        tc_ld16(tm_dk + lane_base + 16u * qr, kv);
        tc_ld16(tm_dv + lane_base + 16u * qr, vv);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_::DKVREAD));
        U8 uk, uv;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          __nv_bfloat162 hk = __floats2bfloat162_rn(__uint_as_float(kv[2 * e]) * p.scale, __uint_as_float(kv[2 * e + 1]) * p.scale);
          __nv_bfloat162 hv = __floats2bfloat162_rn(__uint_as_float(vv[2 * e]), __uint_as_float(vv[2 * e + 1]));
          uk.w[e] = *reinterpret_cast<uint32_t*>(&hk);
          uv.w[e] = *reinterpret_cast<uint32_t*>(&hv);
        }
        st_global_v8(dk_row, uk);
        st_global_v8(dv_row, uv);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == B4_ROW_WARPS) { tc_fence_after(); tmem_dealloc(tmem, C_::TMEM_COLS); }
}

}  // namespace

bool fax_attention_bwd4_supported(int B, int T, int H, int hd) { return hd == B4_HD && T % 128 == 0 && B > 0 && H > 0; }

// The main kernel only: D = rowsum(dO o O) must be in Dv and dq_acc cleared (both by the row-dot
// kernel), and dq_acc is converted to bf16 by the caller afterwards.
fax_status fax_attention_bwd4_tc(fax_ctx* ctx, int B, int T, int H, int hd, const void* qkv, const float* lse,
                                 const void* d_o, void* dqkv, const float* Dv, float* dq_acc) {
  if (!fax_attention_bwd4_supported(B, T, H, hd)) return FAX_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap mq, md, mdq;
  const uint64_t d = (uint64_t)H * B4_HD;
  const uint64_t n_tok = (uint64_t)B * T;
  if (!make_map(ctx, &mq, qkv, 3 * d, n_tok, 3 * d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map(ctx, &md, d_o, d, n_tok, d, 64, 128)) return FAX_ERR_INVALID_ARG;
  if (!make_map_f32(ctx, &mdq, dq_acc, d, n_tok, d, 32, 64)) return FAX_ERR_INVALID_ARG;
  Bwd4Params p;
  p.B = B; p.T = T; p.H = H; p.lse = lse; p.Dv = Dv; p.dqkv = (bf16*)dqkv;
  p.scale = 1.0f / sqrtf((float)B4_HD);
  p.scale_log2 = 1.4426950408889634f * p.scale;
  p.status = ctx->dev_status;
  static bool attr_set[FAX_MAX_DEVICES] = {};
  FAX_TRY(fax_opt_in_shared_memory(ctx, attn_bwd4_tc_kernel, B4::SMEM_BYTES, attr_set));
  const long long items = (long long)B * H * (T / 128);
  const int grid = (int)(items < ctx->sm_count ? items : ctx->sm_count);
  fax_launch(ctx, attn_bwd4_tc_kernel, dim3(grid), dim3(B4_THREADS), B4::SMEM_BYTES, mq, md, mdq, p);
  return fax_after_launch(ctx);
}
