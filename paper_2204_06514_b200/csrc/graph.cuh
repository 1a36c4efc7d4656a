// Graph replay of whole steps (see graph.cu).
#pragma once
#include "common.cuh"

#include <functional>

uint64_t fax_hash_bytes(uint64_t h, const void* data, size_t n);
constexpr uint64_t FAX_HASH_SEED = 1469598103934665603ull;

// What identifies a step for replay: configuration, every buffer address and size.  The bytes
// themselves are kept beside their hash, and a stored graph is replayed only when the bytes are
// equal (a 64-bit hash alone could replay another step's graph on a collision).
struct FaxStepKey {
  uint64_t hash = FAX_HASH_SEED;
  std::vector<unsigned char> material;
  template <typename T> void add(const T& v) {
    const unsigned char* p = (const unsigned char*)&v;
    material.insert(material.end(), p, p + sizeof(T));
    hash = fax_hash_bytes(hash, p, sizeof(T));
  }
  // Field by field (the structs have padding bytes the caller need not have cleared).
  void add_param(const fax_param& p) {
    add(p.w); add(p.w_compute); add(p.m); add(p.v); add(p.g); add(p.n); add(p.weight_decay);
  }
  void add_layer(const fax_layer_state* L) {
    const fax_param* a = (const fax_param*)L;
    for (int i = 0; i < 12; ++i) add_param(a[i]);
  }
};

// Runs `enqueue` (which enqueues one whole step on the context's streams) directly, or
// captures / replays it as a graph identified by `key`.
fax_status fax_run_step(fax_ctx* ctx, const FaxStepKey& key, const fax_adamw_hparams* hp,
                        const std::function<fax_status()>& enqueue);
void fax_graph_clear(fax_ctx* ctx);
