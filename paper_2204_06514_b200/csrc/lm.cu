// Host orchestration of the N-layer language-model training step: embedding,
// blocks, final LayerNorm, tied output projection with softmax cross-entropy
// (computed over row chunks so full logits never exist), backward through all
// of it, and AdamW over every tensor.
#include "block.cuh"
#include "graph.cuh"

#include <vector>

namespace {

// Logits rows per chunk of the head: as many as fit a 4 GiB logits buffer (at least 8192).  Large
// chunks matter for the dxf GEMM, whose output is only d wide: with 8192 rows and d = 768 it has 96
// tiles for 74 SM pairs (two waves, the second a third full); all 16384 rows at once need three
// waves instead of four.
constexpr int HEAD_ROWS_MIN = 8192;
constexpr size_t HEAD_LOGITS_BYTES = (size_t)4 << 30;
int head_rows_for(const fax_lm_cfg* c, size_t N, size_t V, size_t es) {
  size_t rows = HEAD_LOGITS_BYTES / (V * es) / 256 * 256;
  if (rows < (size_t)HEAD_ROWS_MIN) rows = HEAD_ROWS_MIN;
  if (c->head_rows > 0) rows = (size_t)c->head_rows;
  return (int)(N < rows ? N : rows);
}

struct LmSaved {
  std::vector<void*> act;           // act[l]: input of block l; act[L]: output of the last block
  std::vector<BlockSaved> blk;
  void* xf; float* muf; float* rstdf;
};
struct LmScratch {
  int32_t* ids; int32_t* targets;   // staging for the host entry point
  BlockScratch blk;
  void* dxa; void* dxb;             // gradient ping-pong between layers
  void* logits; int head_rows;
  float* row_loss;
};

fax_status lm_validate(const fax_lm_cfg* c) {
  if (!c) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_block_validate(&c->block));
  if (c->n_layers <= 0 || c->vocab <= 0 || c->max_seq < c->block.seq) return FAX_ERR_INVALID_ARG;
  if (c->head_rows < 0 || c->head_rows % 128) return FAX_ERR_INVALID_ARG;
  if (c->block.prec == FAX_PREC_BF16 && c->vocab % 128) return FAX_ERR_UNSUPPORTED_SHAPE;
  return FAX_OK;
}

void carve_saved(const fax_lm_cfg* c, FaxArena& ar, LmSaved* s) {
  const size_t es = fax_elem_size(c->block.prec);
  const size_t N = (size_t)c->block.batch * c->block.seq, d = c->block.d_model;
  s->act.resize(c->n_layers + 1);
  s->blk.resize(c->n_layers);
  for (int l = 0; l <= c->n_layers; ++l) s->act[l] = ar.take(N * d * es);
  for (int l = 0; l < c->n_layers; ++l) fax_block_carve_saved(&c->block, ar, false, &s->blk[l]);
  s->xf = ar.take(N * d * es);
  s->muf = (float*)ar.take(N * 4);
  s->rstdf = (float*)ar.take(N * 4);
}

void carve_scratch(const fax_lm_cfg* c, FaxArena& ar, LmScratch* s) {
  const size_t es = fax_elem_size(c->block.prec);
  const size_t N = (size_t)c->block.batch * c->block.seq, d = c->block.d_model;
  s->ids = (int32_t*)ar.take(N * 4);
  s->targets = (int32_t*)ar.take(N * 4);
  fax_block_carve_scratch(&c->block, ar, &s->blk);
  s->dxa = ar.take(N * d * es);
  s->dxb = ar.take(N * d * es);
  s->head_rows = head_rows_for(c, N, (size_t)c->vocab, es);
  s->logits = ar.take((size_t)s->head_rows * c->vocab * es);
  s->row_loss = (float*)ar.take(N * 4);
}

fax_status check_param(const fax_param& p, uint64_t n, int prec) {
  if (!p.w || !p.m || !p.v || !p.g || p.n != n) return FAX_ERR_INVALID_ARG;
  if (prec == FAX_PREC_BF16 && !p.w_compute) return FAX_ERR_INVALID_ARG;
  return FAX_OK;
}
const void* compute_ptr(const fax_param& p, int prec) {
  return (prec == FAX_PREC_BF16 || p.w_compute) ? (const void*)p.w_compute : (const void*)p.w;
}

fax_status lm_check_state(const fax_lm_cfg* c, const fax_lm_state* st) {
  if (!st || !st->layers || !st->saved || !st->scratch) return FAX_ERR_INVALID_ARG;
  const uint64_t d = c->block.d_model;
  const int prec = c->block.prec;
  FAX_TRY(check_param(st->wte, (uint64_t)c->vocab * d, prec));
  FAX_TRY(check_param(st->wpe, (uint64_t)c->max_seq * d, prec));
  FAX_TRY(check_param(st->lnf_g, d, prec));
  FAX_TRY(check_param(st->lnf_b, d, prec));
  for (int l = 0; l < c->n_layers; ++l) FAX_TRY(fax_layer_check(&st->layers[l], &c->block));
  if (!fax_aligned(st->saved, 256) || !fax_aligned(st->scratch, 256)) return FAX_ERR_INVALID_ARG;
  return FAX_OK;
}

fax_status lm_fwd_bwd(fax_ctx* ctx, const fax_lm_cfg* c, const fax_lm_state* st, const int32_t* ids,
                      const int32_t* targets, float* loss_device, const LmSaved& sv, const LmScratch& w,
                      const fax_adamw_hparams* hp, bool acc = false, float grad_scale = 1.f) {
  const fax_block_cfg* bc = &c->block;
  const int prec = bc->prec, L = c->n_layers;
  const int N = bc->batch * bc->seq, d = bc->d_model, V = c->vocab;
  const size_t es = fax_elem_size(prec);
  const void* wte = compute_ptr(st->wte, prec);
  const void* wpe = compute_ptr(st->wpe, prec);
  const void* lnf_g = compute_ptr(st->lnf_g, prec);
  const void* lnf_b = compute_ptr(st->lnf_b, prec);

  // forward
  FAX_TRY(fax_embed_fwd(ctx, prec, bc->batch, bc->seq, d, V, ids, wte, wpe, sv.act[0]));
  for (int l = 0; l < L; ++l) {
    fax_block_params p; fax_block_grads g;
    fax_layer_views(&st->layers[l], prec, &p, &g);
    FAX_TRY(fax_block_forward_impl(ctx, bc, &p, sv.act[l], sv.act[l + 1], sv.blk[l], false, &w.blk));
  }
  FAX_TRY(fax_layernorm_fwd(ctx, prec, N, d, sv.act[L], lnf_g, lnf_b, bc->ln_eps, sv.xf, sv.muf, sv.rstdf, nullptr));

  // head: logits chunk -> loss rows and dlogits in place -> dxf chunk, dwte accumulation
  void* dxf = w.dxa;
  for (int r0 = 0; r0 < N; r0 += w.head_rows) {
    const int R = (N - r0) < w.head_rows ? (N - r0) : w.head_rows;
    const char* xf_rows = (const char*)sv.xf + (size_t)r0 * d * es;
    FaxGemm g;
    g.adam = nullptr;
    g.alpha = 1.f; g.epi = EPI_NONE; g.bias = nullptr; g.resid = nullptr; g.ldr = 0; g.aux = nullptr; g.ldaux = 0;
    // logits = xf wte^T
    g.M = R; g.N = V; g.K = d;
    g.A = xf_rows; g.lda = d; g.a_mn_major = false;
    g.B = wte; g.ldb = d; g.b_mn_major = false;
    g.C = w.logits; g.ldc = V; g.c_f32 = false; g.accumulate = false;
    FAX_TRY(fax_gemm(ctx, prec, g));
    FAX_TRY(fax_xent(ctx, prec, R, V, w.logits, V, targets + r0, grad_scale / (float)N, w.row_loss + r0));
    // dxf = dlogits wte
    g.M = R; g.N = d; g.K = V;
    g.A = w.logits; g.lda = V; g.a_mn_major = false;
    g.B = wte; g.ldb = d; g.b_mn_major = true;
    g.C = (char*)dxf + (size_t)r0 * d * es; g.ldc = d; g.c_f32 = false; g.accumulate = false;
    FAX_TRY(fax_gemm(ctx, prec, g));
    // dwte (+)= dlogits^T xf
    g.M = V; g.N = d; g.K = R;
    g.A = w.logits; g.lda = V; g.a_mn_major = true;
    g.B = xf_rows; g.ldb = d; g.b_mn_major = true;
    g.C = st->wte.g; g.ldc = d; g.c_f32 = true; g.accumulate = acc || (r0 != 0);
    FAX_TRY(fax_gemm(ctx, prec, g));
  }
  FAX_TRY(fax_loss_mean(ctx, N, w.row_loss, loss_device));

  // backward through the final LayerNorm and the blocks
  void* dcur = w.dxb;
  FAX_TRY(fax_layernorm_bwd(ctx, prec, N, d, dxf, sv.act[L], sv.muf, sv.rstdf, lnf_g, nullptr, dcur,
                            st->lnf_g.g, st->lnf_b.g, acc, w.blk.partial, w.blk.partial_floats));
  void* dnext = w.dxa;
  for (int l = L - 1; l >= 0; --l) {
    fax_block_params p; fax_block_grads g;
    fax_layer_views(&st->layers[l], prec, &p, &g);
    fax_adamw_tensor t12[12];
    FaxAdamHook hook = {t12, hp};
    if (hp) fax_layer_adamw_tensors(&st->layers[l], prec, t12);
    FAX_TRY(fax_block_backward_impl(ctx, bc, &p, dcur, sv.blk[l], sv.act[l], dnext, &g, acc, w.blk,
                                    hp ? &hook : nullptr));
    void* t = dcur; dcur = dnext; dnext = t;
  }
  // embedding gradients: scatter into the tied dwte, batch-sum into dwpe
  return fax_embed_bwd(ctx, prec, bc->batch, bc->seq, c->max_seq, d, V, ids, dcur, st->wte.g, st->wpe.g, acc);
}

// AdamW of the tensors that are not inside a block (the blocks' tensors are updated under backward).
fax_status lm_adamw(fax_ctx* ctx, const fax_lm_cfg* c, const fax_lm_state* st, const fax_adamw_hparams* hp) {
  const int prec = c->block.prec;
  std::vector<fax_adamw_tensor> t;
  t.reserve(4);
  auto push = [&](const fax_param& p) {
    fax_adamw_tensor a;
    a.w = p.w; a.m = p.m; a.v = p.v; a.g = p.g;
    a.w_compute = (prec == FAX_PREC_BF16) ? p.w_compute : nullptr;
    a.n = p.n; a.weight_decay = p.weight_decay;
    t.push_back(a);
  };
  push(st->wte); push(st->wpe);
  push(st->lnf_g); push(st->lnf_b);
  FAX_TRY(fax_adamw_launch(ctx, t.data(), (int)t.size(), hp));
  return fax_adamw_join(ctx);
}

fax_status lm_run(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st, const int32_t* ids,
                  const int32_t* targets, const fax_adamw_hparams* hp, float* loss_device,
                  const int32_t* ids_host, const int32_t* targets_host) {
  FAX_TRY(lm_validate(cfg));
  FAX_TRY(lm_check_state(cfg, st));
  if (!loss_device) return FAX_ERR_INVALID_ARG;
  FaxArena ar(st->saved, st->saved_bytes), aw(st->scratch, st->scratch_bytes);
  LmSaved sv; LmScratch w;
  carve_saved(cfg, ar, &sv);
  carve_scratch(cfg, aw, &w);
  if (ar.used() > st->saved_bytes || aw.used() > st->scratch_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  if (ids_host) {
    const size_t nb = (size_t)cfg->block.batch * cfg->block.seq * sizeof(int32_t);
    FAX_CUDA_TRY(ctx, cudaMemcpyAsync(w.ids, ids_host, nb, cudaMemcpyHostToDevice, ctx->stream));
    FAX_CUDA_TRY(ctx, cudaMemcpyAsync(w.targets, targets_host, nb, cudaMemcpyHostToDevice, ctx->stream));
    ids = w.ids; targets = w.targets;
  }
  fax_adamw_hparams h;
  if (hp) {
    h = *hp;
    h.grad_is_bf16 = 0;
    if (h.step < 1) return FAX_ERR_INVALID_ARG;
  }
  FAX_TRY(lm_fwd_bwd(ctx, cfg, st, ids, targets, loss_device, sv, w, hp ? &h : nullptr));
  if (hp) FAX_TRY(lm_adamw(ctx, cfg, st, &h));
  return FAX_OK;
}

}  // namespace

extern "C" fax_status fax_lm_sizes(const fax_lm_cfg* cfg, size_t* saved_bytes, size_t* scratch_bytes) {
  FAX_TRY(lm_validate(cfg));
  FaxArena a(nullptr, 0), b(nullptr, 0);
  LmSaved s; LmScratch w;
  carve_saved(cfg, a, &s);
  carve_scratch(cfg, b, &w);
  if (saved_bytes) *saved_bytes = a.used();
  if (scratch_bytes) *scratch_bytes = b.used();
  return FAX_OK;
}

extern "C" fax_status fax_lm_arena_layout(const fax_lm_cfg* cfg, size_t* act_off, size_t* layer_saved_off,
                                          size_t* xf_off, size_t* row_loss_off, size_t* block_scratch_off) {
  FAX_TRY(lm_validate(cfg));
  if (!act_off || !layer_saved_off || !xf_off || !row_loss_off || !block_scratch_off) return FAX_ERR_INVALID_ARG;
  char* base = (char*)4096;
  FaxArena a(base, (size_t)-1), b(base, (size_t)-1);
  LmSaved s; LmScratch w;
  carve_saved(cfg, a, &s);
  carve_scratch(cfg, b, &w);
  for (int l = 0; l <= cfg->n_layers; ++l) act_off[l] = (size_t)((char*)s.act[l] - base);
  for (int l = 0; l < cfg->n_layers; ++l) layer_saved_off[l] = (size_t)((char*)s.blk[l].a - base);
  *xf_off = (size_t)((char*)s.xf - base);
  *row_loss_off = (size_t)((char*)w.row_loss - base);
  *block_scratch_off = (size_t)((char*)w.blk.bufF - base);
  return FAX_OK;
}

extern "C" fax_status fax_lm_forward_backward(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                              const int32_t* ids, const int32_t* targets, float* loss_device) {
  if (!ctx || !ids || !targets) return FAX_ERR_INVALID_ARG;
  return lm_run(ctx, cfg, st, ids, targets, nullptr, loss_device, nullptr, nullptr);
}

extern "C" fax_status fax_lm_accumulate(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                        const int32_t* ids, const int32_t* targets, float* loss_device,
                                        int32_t accumulate, float grad_scale) {
  if (!ctx || !ids || !targets || !loss_device) return FAX_ERR_INVALID_ARG;
  FAX_TRY(lm_validate(cfg));
  FAX_TRY(lm_check_state(cfg, st));
  FaxArena ar(st->saved, st->saved_bytes), aw(st->scratch, st->scratch_bytes);
  LmSaved sv; LmScratch w;
  carve_saved(cfg, ar, &sv);
  carve_scratch(cfg, aw, &w);
  if (ar.used() > st->saved_bytes || aw.used() > st->scratch_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  return lm_fwd_bwd(ctx, cfg, st, ids, targets, loss_device, sv, w, nullptr, accumulate != 0, grad_scale);
}

extern "C" fax_status fax_lm_apply_adamw(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                         const fax_adamw_hparams* hp) {
  if (!ctx || !hp) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  FAX_TRY(lm_validate(cfg));
  FAX_TRY(lm_check_state(cfg, st));
  fax_adamw_hparams h = *hp;
  h.grad_is_bf16 = 0;
  const int prec = cfg->block.prec;
  for (int l = 0; l < cfg->n_layers; ++l) {
    fax_adamw_tensor t12[12];
    fax_layer_adamw_tensors(&st->layers[l], prec, t12);
    FAX_TRY(fax_adamw_launch(ctx, t12, 12, &h));
  }
  return lm_adamw(ctx, cfg, st, &h);
}

extern "C" fax_status fax_lm_step(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                  const int32_t* ids, const int32_t* targets, const fax_adamw_hparams* hp,
                                  float* loss_device, float* loss_host) {
  if (!ctx || !ids || !targets || !hp || !cfg || !st) return FAX_ERR_INVALID_ARG;
  if (hp->step < 1 || cfg->n_layers <= 0 || !st->layers) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  FaxStepKey key;
  key.add('L');
  key.add(*cfg);
  key.add_param(st->wte); key.add_param(st->wpe);
  key.add_param(st->lnf_g); key.add_param(st->lnf_b);
  for (int l = 0; l < cfg->n_layers; ++l) key.add_layer(&st->layers[l]);
  key.add(st->saved); key.add(st->saved_bytes);
  key.add(st->scratch); key.add(st->scratch_bytes);
  key.add(ids); key.add(targets); key.add(loss_device);
  FAX_TRY(fax_run_step(ctx, key, hp, [&]() { return lm_run(ctx, cfg, st, ids, targets, hp, loss_device, nullptr, nullptr); }));
  if (loss_host) {
    FAX_CUDA_TRY(ctx, cudaMemcpyAsync(loss_host, loss_device, sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  }
  return FAX_OK;
}

extern "C" fax_status fax_lm_step_host(fax_ctx* ctx, const fax_lm_cfg* cfg, const fax_lm_state* st,
                                       const int32_t* ids_host, const int32_t* targets_host,
                                       const fax_adamw_hparams* hp, float* loss_device, float* loss_host) {
  if (!ctx || !ids_host || !targets_host || !hp || !loss_host) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  FAX_TRY(lm_run(ctx, cfg, st, nullptr, nullptr, hp, loss_device, ids_host, targets_host));
  FAX_CUDA_TRY(ctx, cudaMemcpyAsync(loss_host, loss_device, sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  return FAX_OK;
}
