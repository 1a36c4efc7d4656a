// Host orchestration of one pre-LayerNorm decoder block: forward (steps F1-F7),
// backward (B1-B7) and the whole block training step with AdamW.  Only enqueues
// kernels on the context's stream; every buffer is carved from caller arenas.
#include "block.cuh"
#include "graph.cuh"

fax_status fax_block_validate(const fax_block_cfg* c) {
  if (!c) return FAX_ERR_INVALID_ARG;
  if (c->batch <= 0 || c->seq <= 0 || c->d_model <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->d_ff <= 0)
    return FAX_ERR_INVALID_ARG;
  if ((int64_t)c->n_heads * c->head_dim != c->d_model) return FAX_ERR_INVALID_ARG;
  if (c->prec != FAX_PREC_BF16 && c->prec != FAX_PREC_FP32_VALIDATE) return FAX_ERR_INVALID_ARG;
  if (!(c->ln_eps > 0.f)) return FAX_ERR_INVALID_ARG;
  if (c->recompute != 0 && c->recompute != 1) return FAX_ERR_INVALID_ARG;
  if ((int64_t)c->batch * c->seq > (1 << 30)) return FAX_ERR_UNSUPPORTED_SHAPE;
  if (c->head_dim > 128) return FAX_ERR_UNSUPPORTED_SHAPE;
  if (c->prec == FAX_PREC_BF16) {
    if (c->head_dim != 64 && c->head_dim != 128) return FAX_ERR_UNSUPPORTED_SHAPE;
    if (c->d_model % 128 || c->d_ff % 128 || ((int64_t)c->batch * c->seq) % 128) return FAX_ERR_UNSUPPORTED_SHAPE;
  } else {
    if (c->d_model % 4 || c->d_ff % 4) return FAX_ERR_UNSUPPORTED_SHAPE;
  }
  return FAX_OK;
}

void fax_block_carve_saved(const fax_block_cfg* c, FaxArena& ar, bool with_x, BlockSaved* s) {
  const size_t es = fax_elem_size(c->prec);
  const size_t N = (size_t)c->batch * c->seq, d = c->d_model, f = c->d_ff;
  s->x = with_x ? ar.take(N * d * es) : nullptr;
  const bool keep = !c->recompute;       // LayerNorm outputs and GELU(h) are saved unless backward recomputes them
  s->a = keep ? ar.take(N * d * es) : nullptr;
  s->qkv = ar.take(N * 3 * d * es);
  s->o = ar.take(N * d * es);
  s->x1 = ar.take(N * d * es);
  s->m = keep ? ar.take(N * d * es) : nullptr;
  s->h = ar.take(N * f * es);
  s->g = keep ? ar.take(N * f * es) : nullptr;
  s->mu1 = (float*)ar.take(N * 4);
  s->rstd1 = (float*)ar.take(N * 4);
  s->mu2 = (float*)ar.take(N * 4);
  s->rstd2 = (float*)ar.take(N * 4);
  s->lse = (float*)ar.take((size_t)c->batch * c->n_heads * c->seq * 4);
}

void fax_block_carve_scratch(const fax_block_cfg* c, FaxArena& ar, BlockScratch* s) {
  const size_t es = fax_elem_size(c->prec);
  const size_t N = (size_t)c->batch * c->seq, d = c->d_model, f = c->d_ff;
  s->bufF = ar.take(N * f * es);
  s->bufQ = ar.take(N * 3 * d * es);
  s->bufA = ar.take(N * d * es);
  s->bufB = ar.take(N * d * es);
  size_t widest = f > 3 * d ? f : 3 * d;
  size_t pf = fax_colsum_partial_floats((int)N, (int)widest);
  size_t lp = fax_layernorm_bwd_partial_floats((int)N, (int)d);
  s->partial_floats = pf > lp ? pf : lp;
  s->partial = (float*)ar.take(s->partial_floats * 4);
  s->attn_bytes = fax_attention_bwd_scratch_bytes(c->prec, c->batch, c->seq, c->n_heads, c->head_dim);
  s->attn = ar.take(s->attn_bytes);
}

extern "C" fax_status fax_block_sizes(const fax_block_cfg* cfg, size_t* saved_bytes, size_t* scratch_bytes) {
  FAX_TRY(fax_block_validate(cfg));
  FaxArena a(nullptr, 0), b(nullptr, 0);
  BlockSaved s; BlockScratch w;
  fax_block_carve_saved(cfg, a, true, &s);
  fax_block_carve_scratch(cfg, b, &w);
  if (saved_bytes) *saved_bytes = a.used();
  if (scratch_bytes) *scratch_bytes = b.used();
  return FAX_OK;
}

static void saved_offsets(const BlockSaved& s, const char* base, size_t* off) {
  const void* p[13] = {s.x, s.a, s.qkv, s.o, s.x1, s.m, s.h, s.g, s.mu1, s.rstd1, s.mu2, s.rstd2, s.lse};
  for (int i = 0; i < 13; ++i) off[i] = p[i] ? (size_t)((const char*)p[i] - base) : (size_t)-1;
}

extern "C" fax_status fax_block_arena_layout(const fax_block_cfg* cfg, size_t* saved_off, size_t* scratch_off) {
  FAX_TRY(fax_block_validate(cfg));
  if (!saved_off || !scratch_off) return FAX_ERR_INVALID_ARG;
  char* base = (char*)4096;              // any non-null base: only differences are used
  FaxArena a(base, (size_t)-1), b(base, (size_t)-1);
  BlockSaved s; BlockScratch w;
  fax_block_carve_saved(cfg, a, true, &s);
  fax_block_carve_scratch(cfg, b, &w);
  saved_offsets(s, base, saved_off);
  scratch_off[0] = (size_t)((char*)w.bufF - base);
  scratch_off[1] = (size_t)((char*)w.bufQ - base);
  scratch_off[2] = (size_t)((char*)w.bufA - base);
  scratch_off[3] = (size_t)((char*)w.bufB - base);
  return FAX_OK;
}

static FaxGemm gemm_desc(int M, int N, int K) {
  FaxGemm g;
  g.M = M; g.N = N; g.K = K;
  g.A = nullptr; g.lda = 0; g.a_mn_major = false;
  g.B = nullptr; g.ldb = 0; g.b_mn_major = false;
  g.C = nullptr; g.ldc = N; g.c_f32 = false; g.accumulate = false;
  g.epi = EPI_NONE; g.bias = nullptr; g.resid = nullptr; g.ldr = 0; g.aux = nullptr; g.ldaux = 0;
  g.alpha = 1.f;
  g.adam = nullptr;
  return g;
}

// y = x W (+ epilogue): x [N,K] row-major, W [K,Nout] row-major
static fax_status linear_fwd(fax_ctx* ctx, int prec, int N, int K, int Nout, const void* x, const void* W,
                             const void* bias, int epi, const void* resid, void* aux, void* y) {
  FaxGemm g = gemm_desc(N, Nout, K);
  g.A = x; g.lda = K; g.a_mn_major = false;
  g.B = W; g.ldb = Nout; g.b_mn_major = true;
  g.C = y; g.ldc = Nout;
  g.epi = epi; g.bias = bias; g.resid = resid; g.ldr = Nout; g.aux = aux; g.ldaux = Nout;
  return fax_gemm(ctx, prec, g);
}
// dx = dy W^T (+ epilogue): dy [N,Nout], W [K,Nout] row-major -> dx [N,K]
static fax_status linear_bwd_data(fax_ctx* ctx, int prec, int N, int K, int Nout, const void* dy,
                                  const void* W, int epi, void* aux, void* dx) {
  FaxGemm g = gemm_desc(N, K, Nout);
  g.A = dy; g.lda = Nout; g.a_mn_major = false;
  g.B = W; g.ldb = Nout; g.b_mn_major = false;
  g.C = dx; g.ldc = K;
  g.epi = epi; g.aux = aux; g.ldaux = K;
  return fax_gemm(ctx, prec, g);
}
// dW (+)= x^T dy: x [N,K], dy [N,Nout] -> dW [K,Nout] float
// With `fuse` (the AdamW descriptor and hyper-parameters of this weight) the update happens in the
// GEMM's epilogue where that is possible; *fused tells the caller whether it did.
static fax_status linear_bwd_weight(fax_ctx* ctx, int prec, int N, int K, int Nout, const void* x,
                                    const void* dy, float* dW, bool accumulate,
                                    const fax_adamw_tensor* fuse = nullptr, const fax_adamw_hparams* hp = nullptr,
                                    bool* fused = nullptr) {
  FaxGemm g = gemm_desc(K, Nout, N);
  g.A = x; g.lda = K; g.a_mn_major = true;
  g.B = dy; g.ldb = Nout; g.b_mn_major = true;
  g.C = dW; g.ldc = Nout; g.c_f32 = true; g.accumulate = accumulate;
  if (fused) *fused = false;
  FaxFusedAdam ad;
  if (fuse && hp && fuse->w_compute && fuse->n == (uint64_t)K * Nout && fax_gemm_can_fuse_adam(ctx, g)) {
    ad.w = fuse->w; ad.m = fuse->m; ad.v = fuse->v; ad.w_compute = fuse->w_compute;
    ad.weight_decay = fuse->weight_decay;
    for (int i = 0; i < 8; ++i) ad.sc[i] = 0.f;
    fax_adamw_scalars(hp, ad.sc);
    ad.keep_grad = ctx->keep_fused_grads;
    g.adam = &ad;
    if (fused) *fused = true;
  }
  return fax_gemm(ctx, prec, g);
}

fax_status fax_block_forward_impl(fax_ctx* ctx, const fax_block_cfg* c, const fax_block_params* p,
                                  const void* x, void* y, const BlockSaved& s, bool copy_x, const BlockScratch* w) {
  const int N = c->batch * c->seq, d = c->d_model, f = c->d_ff, prec = c->prec;
  if (c->recompute && !w) return FAX_ERR_INVALID_ARG;
  // with recomputation the LayerNorm outputs and GELU(h) only live until their consumer has run
  void* a = c->recompute ? w->bufA : s.a;
  void* m = c->recompute ? w->bufB : s.m;
  void* g = c->recompute ? w->bufF : s.g;
  FAX_TRY(fax_layernorm_fwd(ctx, prec, N, d, x, p->ln1_g, p->ln1_b, c->ln_eps, a, s.mu1, s.rstd1,
                            copy_x ? s.x : nullptr));
  FAX_TRY(linear_fwd(ctx, prec, N, d, 3 * d, a, p->w_qkv, p->b_qkv, EPI_BIAS, nullptr, nullptr, s.qkv));
  FAX_TRY(fax_attention_fwd(ctx, prec, c->batch, c->seq, c->n_heads, c->head_dim, s.qkv, s.o, s.lse));
  FAX_TRY(linear_fwd(ctx, prec, N, d, d, s.o, p->w_o, p->b_o, EPI_BIAS_RESID, x, nullptr, s.x1));
  FAX_TRY(fax_layernorm_fwd(ctx, prec, N, d, s.x1, p->ln2_g, p->ln2_b, c->ln_eps, m, s.mu2, s.rstd2, nullptr));
  FAX_TRY(linear_fwd(ctx, prec, N, d, f, m, p->w_fc1, p->b_fc1, EPI_BIAS_GELU, nullptr, g, s.h));
  FAX_TRY(linear_fwd(ctx, prec, N, f, d, g, p->w_fc2, p->b_fc2, EPI_BIAS_RESID, s.x1, nullptr, y));
  return FAX_OK;
}

fax_status fax_block_backward_impl(fax_ctx* ctx, const fax_block_cfg* c, const fax_block_params* p,
                                   const void* dy, const BlockSaved& s, const void* x, void* dx,
                                   const fax_block_grads* gr, bool acc, const BlockScratch& w,
                                   const FaxAdamHook* hook) {
  const int N = c->batch * c->seq, d = c->d_model, f = c->d_ff, prec = c->prec;
  // once both gradients of a linear layer (or LayerNorm) exist and the data-gradient GEMM has
  // consumed the old weight, its AdamW update runs on the optimizer stream under the rest of backward
  const bool rc = c->recompute != 0;
  // (the fused update rewrites a weight inside its dW GEMM, so the dX GEMM must come first: not with
  // recomputation, where FC2's dW runs before its dX to free the GELU buffer)
  const bool try_fuse = hook && ctx->fused_update && prec == FAX_PREC_BF16 && !acc && !rc;
  // recomputed LayerNorm outputs need throw-away statistics: the head of the column-sum scratch
  if (rc && w.partial_floats < (size_t)2 * N) return FAX_ERR_WORKSPACE_TOO_SMALL;
  float* tmp_mu = w.partial; float* tmp_rstd = w.partial + N;
  auto update = [&](int first, bool matrix_done = false) -> fax_status {
    if (!hook) return FAX_OK;
    return matrix_done ? fax_adamw_async(ctx, hook->t + first + 1, 1, hook->hp)      // only the bias is left
                       : fax_adamw_async(ctx, hook->t + first, 2, hook->hp);
  };
  // The gradients of the two biases beside LayerNorm 2 - db_fc2 = column sums of dY (the residual
  // gradient that B3 adds) and db_o = column sums of dx1 (what B3 writes) - are taken inside the
  // LayerNorm backward kernel of B3, so b_fc2 is updated there, together with the LayerNorm's own tensors.
  bool fz = false;
  // B1: through FC2 and GELU
  if (rc) {
    // g = GELU(h) again, into the buffer that receives dh afterwards: dW2 first, then dh over it
    FAX_TRY(fax_gelu_fwd(ctx, prec, (size_t)N * f, s.h, w.bufF));
    FAX_TRY(linear_bwd_weight(ctx, prec, N, f, d, w.bufF, dy, gr->w_fc2, acc, nullptr, nullptr, &fz));
    FAX_TRY(linear_bwd_data(ctx, prec, N, f, d, dy, p->w_fc2, EPI_DGELU, s.h, w.bufF));        // dh
  } else {
    FAX_TRY(linear_bwd_data(ctx, prec, N, f, d, dy, p->w_fc2, EPI_DGELU, s.h, w.bufF));        // dh
    FAX_TRY(linear_bwd_weight(ctx, prec, N, f, d, s.g, dy, gr->w_fc2, acc, try_fuse ? hook->t + 10 : nullptr,
                              try_fuse ? hook->hp : nullptr, &fz));
  }
  if (hook && !fz) FAX_TRY(fax_adamw_async(ctx, hook->t + 10, 1, hook->hp));                    // w_fc2; b_fc2 after B3
  // B2: through FC1
  FAX_TRY(linear_bwd_data(ctx, prec, N, d, f, w.bufF, p->w_fc1, EPI_NONE, nullptr, w.bufA));    // dm
  const void* m_in = s.m;
  if (rc) {   // m = LN2(x1) again, into the buffer that receives dx1 in B3
    FAX_TRY(fax_layernorm_fwd(ctx, prec, N, d, s.x1, p->ln2_g, p->ln2_b, c->ln_eps, w.bufB, tmp_mu, tmp_rstd, nullptr));
    m_in = w.bufB;
  }
  FAX_TRY(linear_bwd_weight(ctx, prec, N, d, f, m_in, w.bufF, gr->w_fc1, acc, try_fuse ? hook->t + 8 : nullptr,
                            try_fuse ? hook->hp : nullptr, &fz));
  FAX_TRY(fax_colsum(ctx, prec, N, f, w.bufF, f, gr->b_fc1, acc, w.partial, w.partial_floats));
  FAX_TRY(update(8, fz));
  // B3: LN2 backward plus the residual branch
  FAX_TRY(fax_layernorm_bwd(ctx, prec, N, d, w.bufA, s.x1, s.mu2, s.rstd2, p->ln2_g, dy, w.bufB,
                            gr->ln2_g, gr->ln2_b, acc, w.partial, w.partial_floats, gr->b_fc2, gr->b_o));   // dx1
  if (hook) {
    const fax_adamw_tensor t3[3] = {hook->t[6], hook->t[7], hook->t[11]};                       // ln2_g, ln2_b, b_fc2
    FAX_TRY(fax_adamw_async(ctx, t3, 3, hook->hp));
  }
  // B4: through the attention output projection
  FAX_TRY(linear_bwd_data(ctx, prec, N, d, d, w.bufB, p->w_o, EPI_NONE, nullptr, w.bufA));      // do
  FAX_TRY(linear_bwd_weight(ctx, prec, N, d, d, s.o, w.bufB, gr->w_o, acc, try_fuse ? hook->t + 4 : nullptr,
                            try_fuse ? hook->hp : nullptr, &fz));
  FAX_TRY(update(4, fz));
  // B5: attention backward
  FAX_TRY(fax_attention_bwd(ctx, prec, c->batch, c->seq, c->n_heads, c->head_dim, s.qkv, s.o, s.lse,
                            w.bufA, w.bufQ, w.attn, w.attn_bytes));                             // dqkv
  // B6: through the QKV projection
  FAX_TRY(linear_bwd_data(ctx, prec, N, d, 3 * d, w.bufQ, p->w_qkv, EPI_NONE, nullptr, w.bufA)); // da
  const void* a_in = s.a;
  if (rc) {   // a = LN1(x) again, into the (by now free) dh buffer
    FAX_TRY(fax_layernorm_fwd(ctx, prec, N, d, x, p->ln1_g, p->ln1_b, c->ln_eps, w.bufF, tmp_mu, tmp_rstd, nullptr));
    a_in = w.bufF;
  }
  FAX_TRY(linear_bwd_weight(ctx, prec, N, d, 3 * d, a_in, w.bufQ, gr->w_qkv, acc, try_fuse ? hook->t + 2 : nullptr,
                            try_fuse ? hook->hp : nullptr, &fz));
  FAX_TRY(fax_colsum(ctx, prec, N, 3 * d, w.bufQ, 3 * d, gr->b_qkv, acc, w.partial, w.partial_floats));
  FAX_TRY(update(2, fz));
  // B7: LN1 backward plus the residual branch
  FAX_TRY(fax_layernorm_bwd(ctx, prec, N, d, w.bufA, x, s.mu1, s.rstd1, p->ln1_g, w.bufB, dx,
                            gr->ln1_g, gr->ln1_b, acc, w.partial, w.partial_floats));
  return update(0);
}

static fax_status check_params(const fax_block_params* p) {
  if (!p) return FAX_ERR_INVALID_ARG;
  const void* const* a = (const void* const*)p;
  for (int i = 0; i < 12; ++i)
    if (!a[i] || !fax_aligned(a[i], 16)) return FAX_ERR_INVALID_ARG;
  return FAX_OK;
}

extern "C" fax_status fax_block_forward(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_params* params,
                                        const void* x, void* y, void* saved, size_t saved_bytes,
                                        void* scratch, size_t scratch_bytes) {
  if (!ctx || !x || !y || !saved || x == y) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_block_validate(cfg));
  FAX_TRY(check_params(params));
  if (!fax_aligned(x, 16) || !fax_aligned(y, 16) || !fax_aligned(saved, 256)) return FAX_ERR_INVALID_ARG;
  FaxArena ar(saved, saved_bytes);
  BlockSaved s;
  fax_block_carve_saved(cfg, ar, true, &s);
  if (ar.used() > saved_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  if (!cfg->recompute) return fax_block_forward_impl(ctx, cfg, params, x, y, s, true);
  if (!scratch || !fax_aligned(scratch, 256)) return FAX_ERR_INVALID_ARG;
  FaxArena aw(scratch, scratch_bytes);
  BlockScratch w;
  fax_block_carve_scratch(cfg, aw, &w);
  if (aw.used() > scratch_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  return fax_block_forward_impl(ctx, cfg, params, x, y, s, true, &w);
}

extern "C" fax_status fax_block_backward(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_params* params,
                                         const void* dy, const void* saved, size_t saved_bytes, void* dx,
                                         const fax_block_grads* grads, int32_t accumulate, void* scratch,
                                         size_t scratch_bytes) {
  if (!ctx || !dy || !dx || !saved || !scratch || !grads) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_block_validate(cfg));
  FAX_TRY(check_params(params));
  const float* const* gp = (const float* const*)grads;
  for (int i = 0; i < 12; ++i)
    if (!gp[i] || !fax_aligned(gp[i], 16)) return FAX_ERR_INVALID_ARG;
  if (!fax_aligned(dy, 16) || !fax_aligned(dx, 16) || !fax_aligned(saved, 256) || !fax_aligned(scratch, 256))
    return FAX_ERR_INVALID_ARG;
  FaxArena ar((void*)saved, saved_bytes), aw(scratch, scratch_bytes);
  BlockSaved s; BlockScratch w;
  fax_block_carve_saved(cfg, ar, true, &s);
  fax_block_carve_scratch(cfg, aw, &w);
  if (ar.used() > saved_bytes || aw.used() > scratch_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  return fax_block_backward_impl(ctx, cfg, params, dy, s, s.x, dx, grads, accumulate != 0, w);
}

void fax_layer_views(const fax_layer_state* L, int prec, fax_block_params* p, fax_block_grads* g) {
  const fax_param* a = (const fax_param*)L;
  const void** pp = (const void**)p;
  float** gg = (float**)g;
  for (int i = 0; i < 12; ++i) {
    pp[i] = (prec == FAX_PREC_BF16 || a[i].w_compute) ? a[i].w_compute : (const void*)a[i].w;
    gg[i] = a[i].g;
  }
}

int fax_layer_adamw_tensors(const fax_layer_state* L, int prec, fax_adamw_tensor* out) {
  const fax_param* a = (const fax_param*)L;
  for (int i = 0; i < 12; ++i) {
    out[i].w = a[i].w; out[i].m = a[i].m; out[i].v = a[i].v; out[i].g = a[i].g;
    out[i].w_compute = (prec == FAX_PREC_BF16) ? a[i].w_compute : nullptr;
    out[i].n = a[i].n; out[i].weight_decay = a[i].weight_decay;
  }
  return 12;
}

fax_status fax_layer_check(const fax_layer_state* L, const fax_block_cfg* c) {
  const fax_param* a = (const fax_param*)L;
  const uint64_t d = c->d_model, f = c->d_ff;
  const uint64_t want[12] = {d, d, d * 3 * d, 3 * d, d * d, d, d, d, d * f, f, f * d, d};
  for (int i = 0; i < 12; ++i) {
    if (!a[i].w || !a[i].m || !a[i].v || !a[i].g) return FAX_ERR_INVALID_ARG;
    if (c->prec == FAX_PREC_BF16 && !a[i].w_compute) return FAX_ERR_INVALID_ARG;
    if (a[i].n != want[i]) return FAX_ERR_INVALID_ARG;
  }
  return FAX_OK;
}

// hooks of the host-buffer variant: dY arrives and y leaves on the copy stream while the
// forward / backward kernels run on the main stream
struct HostIo { const void* dy_host; void* dy_dev; void* y_host; size_t bytes; };

static fax_status block_step_impl(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_state* st,
                                  const void* x, const void* dy, void* y, void* dx,
                                  const fax_adamw_hparams* hp, size_t scratch_skip, const HostIo* io = nullptr) {
  FaxArena ar(st->saved, st->saved_bytes), aw((char*)st->scratch + scratch_skip, st->scratch_bytes - scratch_skip);
  BlockSaved s; BlockScratch w;
  fax_block_carve_saved(cfg, ar, true, &s);
  fax_block_carve_scratch(cfg, aw, &w);
  if (ar.used() > st->saved_bytes || aw.used() + scratch_skip > st->scratch_bytes) return FAX_ERR_WORKSPACE_TOO_SMALL;
  fax_block_params p; fax_block_grads g;
  fax_layer_views(&st->layer, cfg->prec, &p, &g);
  fax_adamw_tensor t[12];
  fax_layer_adamw_tensors(&st->layer, cfg->prec, t);
  fax_adamw_hparams h = *hp;
  h.grad_is_bf16 = 0;
  if (h.step < 1) return FAX_ERR_INVALID_ARG;
  FaxAdamHook hook = {t, &h};
  if (io) {
    // the copy stream may start once the main stream has reached this call (the staging buffers are free)
    FAX_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_copy_a, ctx->stream));
    FAX_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy, ctx->ev_copy_a, 0));
    FAX_CUDA_TRY(ctx, cudaMemcpyAsync(io->dy_dev, io->dy_host, io->bytes, cudaMemcpyHostToDevice, ctx->copy));
    FAX_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_copy_b, ctx->copy));
  }
  // the caller's x stays valid through the step, so backward reads it in place and the saved arena gets
  // no copy of it (unless dx is to overwrite x)
  const bool copy_x = (x == dx);
  FAX_TRY(fax_block_forward_impl(ctx, cfg, &p, x, y, s, copy_x, &w));
  if (io) {
    FAX_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_copy_a, ctx->stream));              // y is complete
    FAX_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy, ctx->ev_copy_a, 0));
    FAX_CUDA_TRY(ctx, cudaMemcpyAsync(io->y_host, y, io->bytes, cudaMemcpyDeviceToHost, ctx->copy));
    FAX_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_copy_b, 0));       // dY has arrived
  }
  FAX_TRY(fax_block_backward_impl(ctx, cfg, &p, dy, s, copy_x ? s.x : x, dx, &g, false, w, &hook));
  return fax_adamw_join(ctx);
}

extern "C" fax_status fax_block_step(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_state* st,
                                     const void* x, const void* dy, void* y, void* dx,
                                     const fax_adamw_hparams* hp) {
  if (!ctx || !st || !x || !dy || !y || !dx || !hp || !st->saved || !st->scratch || x == y) return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_block_validate(cfg));
  FAX_TRY(fax_layer_check(&st->layer, cfg));
  FAX_TRY(fax_adamw_check_hparams(hp));
  FaxStepKey key;
  key.add('B');
  key.add(*cfg);
  key.add_layer(&st->layer);
  key.add(st->saved); key.add(st->saved_bytes);
  key.add(st->scratch); key.add(st->scratch_bytes);
  key.add(x); key.add(dy); key.add(y); key.add(dx);
  return fax_run_step(ctx, key, hp, [&]() { return block_step_impl(ctx, cfg, st, x, dy, y, dx, hp, 0); });
}

extern "C" fax_status fax_block_host_scratch_bytes(const fax_block_cfg* cfg, size_t* scratch_bytes) {
  size_t sv = 0, sc = 0;
  FAX_TRY(fax_block_sizes(cfg, &sv, &sc));
  size_t nd = fax_round_up((size_t)cfg->batch * cfg->seq * cfg->d_model * fax_elem_size(cfg->prec), 256);
  if (scratch_bytes) *scratch_bytes = sc + 4 * nd;
  return FAX_OK;
}

extern "C" fax_status fax_block_step_host(fax_ctx* ctx, const fax_block_cfg* cfg, const fax_block_state* st,
                                          const void* x_host, const void* dy_host, void* y_host,
                                          void* dx_host, const fax_adamw_hparams* hp) {
  if (!ctx || !st || !x_host || !dy_host || !y_host || !dx_host || !hp || !st->saved || !st->scratch)
    return FAX_ERR_INVALID_ARG;
  FAX_TRY(fax_adamw_check_hparams(hp));
  FAX_TRY(fax_block_validate(cfg));
  FAX_TRY(fax_layer_check(&st->layer, cfg));
  const size_t bytes = (size_t)cfg->batch * cfg->seq * cfg->d_model * fax_elem_size(cfg->prec);
  const size_t nd = fax_round_up(bytes, 256);
  if (st->scratch_bytes < 4 * nd) return FAX_ERR_WORKSPACE_TOO_SMALL;
  char* base = (char*)st->scratch;
  void *x = base, *dy = base + nd, *y = base + 2 * nd, *dx = base + 3 * nd;
  HostIo io = {dy_host, dy, y_host, bytes};
  FAX_CUDA_TRY(ctx, cudaMemcpyAsync(x, x_host, bytes, cudaMemcpyHostToDevice, ctx->stream));
  FAX_TRY(block_step_impl(ctx, cfg, st, x, dy, y, dx, hp, 4 * nd, &io));
  FAX_CUDA_TRY(ctx, cudaMemcpyAsync(dx_host, dx, bytes, cudaMemcpyDeviceToHost, ctx->stream));
  FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->copy));
  return FAX_OK;
}
