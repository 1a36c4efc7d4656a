/*
 * fax_dp.h -- data parallelism over the batch (Sec. 3.3: different subsets of a
 * batch of data are processed on different devices in parallel; Sec. 2.2: a
 * named mesh with a data axis).  One process per GPU.  Every rank holds the
 * whole model, runs forward + loss + backward on its own sequences, and the
 * ranks then exchange once per step:
 *
 *   reduce-scatter of the float32 gradients  ->  AdamW on this rank's shard of
 *   w, m, v  ->  all-gather of the bf16 compute copies.
 *
 * The collectives themselves are the caller's (NCCL through torch.distributed in
 * the Python binding); this header has the two pieces that belong to the
 * library: how the parameters are cut into shards, and the AdamW launch over a
 * shard.  The parameters of a data-parallel model live back to back in flat
 * buffers (one each for w, m, v, g and the compute copy, same element offsets
 * in all of them), every tensor starting on a multiple of `align` elements;
 * rank r owns the flat elements [r * S, (r + 1) * S), S = the padded total
 * divided by the world size, rounded up to `align`.  A shard therefore cuts
 * through tensors: it is a list of pieces (tensor, first element, one past the
 * last), each of which AdamW treats like a tensor of its own.  All functions
 * here but fax_dp_adamw_shard are host-only arithmetic and need no GPU.
 */
#ifndef FAX_DP_H_
#define FAX_DP_H_

#include "fax.h"

#ifdef __cplusplus
extern "C" {
#endif

/* A piece of a shard: elements [begin, end) of tensor `tensor` (tensor-local
 * indices); flat_begin is the flat offset of element `begin`. */
typedef struct {
  int32_t tensor;
  uint64_t begin, end;
  uint64_t flat_begin;
} fax_dp_piece;

/* Flat layout of n tensors of sizes[i] elements: offsets[i] (host, n entries)
 * receives tensor i's first flat element (a multiple of align), *padded_total
 * the flat length (a multiple of align * world, so that all shards are equal).
 * align must be a power of two, world >= 1.  FAX_ERR_INVALID_ARG otherwise. */
fax_status fax_dp_layout(const uint64_t* sizes, int32_t n, int32_t align, int32_t world,
                         uint64_t* offsets, uint64_t* padded_total);

/* The shard of `rank`: *shard_begin, *shard_len (flat elements; equal for all
 * ranks) and its pieces in tensor order (pieces has room for max_pieces; n + 1
 * always suffices).  Every element of every tensor lies in exactly one rank's
 * pieces; padding between tensors belongs to no piece.
 * FAX_ERR_WORKSPACE_TOO_SMALL when max_pieces is too small. */
fax_status fax_dp_shard_map(const uint64_t* sizes, int32_t n, int32_t align, int32_t world, int32_t rank,
                            uint64_t* shard_begin, uint64_t* shard_len,
                            fax_dp_piece* pieces, int32_t max_pieces, int32_t* n_pieces);

/* AdamW (Table 1 caption: Adam; parameters stored as float32, Sec. 3) on this
 * rank's shard.  w, m, v and w_compute (bf16 or NULL) are the FLAT device
 * buffers (element 0 = flat element 0); g_shard is this rank's reduced
 * gradient shard (float32, element 0 = flat element shard_begin, i.e. what a
 * reduce-scatter of the flat gradient buffer leaves on this rank);
 * weight_decay[i] belongs to tensor i (host array).  Only the shard's elements
 * of w, m, v, w_compute are read or written.  Asynchronous on the context's
 * stream. */
fax_status fax_dp_adamw_shard(fax_ctx* ctx, float* w, float* m, float* v, const float* g_shard, void* w_compute,
                              const uint64_t* sizes, const float* weight_decay, int32_t n, int32_t align,
                              int32_t world, int32_t rank, const fax_adamw_hparams* hp);

#ifdef __cplusplus
}
#endif
#endif  /* FAX_DP_H_ */
