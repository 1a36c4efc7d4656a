// Graph replay of whole steps (see graph.cu).
#pragma once
#include "common.cuh"

#include <functional>

uint64_t fax_hash_bytes(uint64_t h, const void* data, size_t n);
template <typename T> static inline uint64_t fax_hash(uint64_t h, const T& v) { return fax_hash_bytes(h, &v, sizeof(T)); }
constexpr uint64_t FAX_HASH_SEED = 1469598103934665603ull;

// Field by field (the structs have padding bytes the caller need not have cleared).
static inline uint64_t fax_hash_param(uint64_t h, const fax_param& p) {
  h = fax_hash(h, p.w); h = fax_hash(h, p.w_compute); h = fax_hash(h, p.m); h = fax_hash(h, p.v);
  h = fax_hash(h, p.g); h = fax_hash(h, p.n); h = fax_hash(h, p.weight_decay);
  return h;
}
static inline uint64_t fax_hash_layer(uint64_t h, const fax_layer_state* L) {
  const fax_param* a = (const fax_param*)L;
  for (int i = 0; i < 12; ++i) h = fax_hash_param(h, a[i]);
  return h;
}

// Runs `enqueue` (which enqueues one whole step on the context's streams) directly, or
// captures / replays it as a graph identified by `key`.
fax_status fax_run_step(fax_ctx* ctx, uint64_t key, const fax_adamw_hparams* hp,
                        const std::function<fax_status()>& enqueue);
void fax_graph_clear(fax_ctx* ctx);
