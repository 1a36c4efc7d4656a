// Data parallelism over the batch: how the flat parameter buffers are cut into per-rank shards,
// and the AdamW launch over one shard (include/fax_dp.h).  The collectives belong to the caller.
#include "common.cuh"
#include "../../include/fax_dp.h"

#include <vector>

namespace {

bool dp_args_ok(const uint64_t* sizes, int n, int align, int world) {
  return sizes && n > 0 && align > 0 && (align & (align - 1)) == 0 && world >= 1;
}

uint64_t round_up64(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" fax_status fax_dp_layout(const uint64_t* sizes, int32_t n, int32_t align, int32_t world,
                                    uint64_t* offsets, uint64_t* padded_total) {
  if (!dp_args_ok(sizes, n, align, world) || !offsets || !padded_total) return FAX_ERR_INVALID_ARG;
  uint64_t off = 0;
  for (int i = 0; i < n; ++i) {
    offsets[i] = off;
    off = round_up64(off + sizes[i], (uint64_t)align);
  }
  *padded_total = round_up64(off, (uint64_t)align * (uint64_t)world);
  return FAX_OK;
}

extern "C" fax_status fax_dp_shard_map(const uint64_t* sizes, int32_t n, int32_t align, int32_t world, int32_t rank,
                                       uint64_t* shard_begin, uint64_t* shard_len,
                                       fax_dp_piece* pieces, int32_t max_pieces, int32_t* n_pieces) {
  if (!dp_args_ok(sizes, n, align, world) || rank < 0 || rank >= world || !shard_begin || !shard_len || !n_pieces ||
      (max_pieces > 0 && !pieces))
    return FAX_ERR_INVALID_ARG;
  std::vector<uint64_t> offsets((size_t)n);
  uint64_t total = 0;
  FAX_TRY(fax_dp_layout(sizes, n, align, world, offsets.data(), &total));
  const uint64_t len = total / (uint64_t)world;       // a multiple of align by construction
  const uint64_t lo = len * (uint64_t)rank, hi = lo + len;
  *shard_begin = lo; *shard_len = len;
  int count = 0;
  for (int i = 0; i < n; ++i) {
    const uint64_t t0 = offsets[i], t1 = offsets[i] + sizes[i];
    const uint64_t a = t0 > lo ? t0 : lo, b = t1 < hi ? t1 : hi;
    if (a >= b) continue;
    if (count >= max_pieces) return FAX_ERR_WORKSPACE_TOO_SMALL;
    pieces[count].tensor = i;
    pieces[count].begin = a - t0;
    pieces[count].end = b - t0;
    pieces[count].flat_begin = a;
    ++count;
  }
  *n_pieces = count;
  return FAX_OK;
}

extern "C" fax_status fax_dp_adamw_shard(fax_ctx* ctx, float* w, float* m, float* v, const float* g_shard,
                                         void* w_compute, const uint64_t* sizes, const float* weight_decay,
                                         int32_t n, int32_t align, int32_t world, int32_t rank,
                                         const fax_adamw_hparams* hp) {
  if (!ctx || !w || !m || !v || !g_shard || !weight_decay) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  // a piece starts on a tensor's first element (a multiple of align) or on a shard boundary (likewise):
  // with align >= 8 every slice below is 16-byte aligned in float32 and in bf16
  if (align < 8) return FAX_ERR_INVALID_ARG;
  std::vector<fax_dp_piece> pieces((size_t)n + 1);
  uint64_t lo = 0, len = 0;
  int32_t np = 0;
  FAX_TRY(fax_dp_shard_map(sizes, n, align, world, rank, &lo, &len, pieces.data(), n + 1, &np));
  std::vector<fax_adamw_tensor> t((size_t)np);
  for (int i = 0; i < np; ++i) {
    const fax_dp_piece& pc = pieces[i];
    t[i].w = w + pc.flat_begin;
    t[i].m = m + pc.flat_begin;
    t[i].v = v + pc.flat_begin;
    t[i].g = g_shard + (pc.flat_begin - lo);
    t[i].w_compute = w_compute ? (void*)((bf16*)w_compute + pc.flat_begin) : nullptr;
    t[i].n = pc.end - pc.begin;
    t[i].weight_decay = weight_decay[pc.tensor];
  }
  fax_adamw_hparams h = *hp;
  h.grad_is_bf16 = 0;
  return fax_adamw_launch(ctx, t.data(), np, &h);
}
