// Internal views of the block's saved-activation and scratch arenas.
#pragma once
#include "common.cuh"

struct BlockSaved {
  void *x, *a, *qkv, *o, *x1, *m, *h, *g;
  float *mu1, *rstd1, *mu2, *rstd2, *lse;
};
struct BlockScratch {
  void *bufF, *bufQ, *bufA, *bufB;
  float* partial; size_t partial_floats;
  void* attn; size_t attn_bytes;
};

void fax_block_carve_saved(const fax_block_cfg* c, FaxArena& ar, bool with_x, BlockSaved* s);
void fax_block_carve_scratch(const fax_block_cfg* c, FaxArena& ar, BlockScratch* s);
fax_status fax_block_forward_impl(fax_ctx* ctx, const fax_block_cfg* c, const fax_block_params* p,
                                  const void* x, void* y, const BlockSaved& s, bool copy_x,
                                  const BlockScratch* w = nullptr);
fax_status fax_block_backward_impl(fax_ctx* ctx, const fax_block_cfg* c, const fax_block_params* p,
                                   const void* dy, const BlockSaved& s, const void* x, void* dx,
                                   const fax_block_grads* gr, bool acc, const BlockScratch& w,
                                   const FaxAdamHook* hook = nullptr);
void fax_layer_views(const fax_layer_state* L, int prec, fax_block_params* p, fax_block_grads* g);
int fax_layer_adamw_tensors(const fax_layer_state* L, int prec, fax_adamw_tensor* out);
fax_status fax_layer_check(const fax_layer_state* L, const fax_block_cfg* c);
