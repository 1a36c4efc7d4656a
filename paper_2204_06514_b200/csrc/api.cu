// Context lifetime, status strings and the device status word.
#include "graph.cuh"

extern "C" const char* fax_status_string(fax_status s) {
  switch (s) {
    case FAX_OK: return "FAX_OK";
    case FAX_ERR_INVALID_ARG: return "FAX_ERR_INVALID_ARG";
    case FAX_ERR_UNSUPPORTED_SHAPE: return "FAX_ERR_UNSUPPORTED_SHAPE";
    case FAX_ERR_WORKSPACE_TOO_SMALL: return "FAX_ERR_WORKSPACE_TOO_SMALL";
    case FAX_ERR_CUDA: return "FAX_ERR_CUDA";
    case FAX_ERR_ARCH: return "FAX_ERR_ARCH";
    case FAX_ERR_TIMEOUT: return "FAX_ERR_TIMEOUT";
    default: return "FAX_ERR_UNKNOWN";
  }
}

extern "C" fax_status fax_create(fax_ctx** out, int32_t device_ordinal, void* cuda_stream) {
  if (!out) return FAX_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device_ordinal < 0 || device_ordinal >= count) {
    (void)cudaGetLastError();
    return FAX_ERR_CUDA;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device_ordinal) != cudaSuccess) return FAX_ERR_CUDA;
  if (prop.major != 10) return FAX_ERR_ARCH;
  if (cudaSetDevice(device_ordinal) != cudaSuccess) return FAX_ERR_CUDA;
  fax_ctx* c = new fax_ctx();
  c->device = device_ordinal;
  c->stream = (cudaStream_t)cuda_stream;
  c->last_cuda_error = 0;
  c->launches = 0;
  c->sm_count = prop.multiProcessorCount;
  c->dev_status = nullptr;
  c->encode_tiled = nullptr;
  c->prof_on = false;
  c->side = nullptr; c->ev_fork = nullptr; c->ev_join = nullptr; c->side_busy = false;
  c->copy = nullptr; c->ev_copy_a = nullptr; c->ev_copy_b = nullptr;
  c->overlap_adamw = true;
  c->use_2cta = true;
  c->use_pdl = true;
  c->attn_bwd_mode = 2;
  c->gemm_l2_budget = 48e6;
  c->use_graphs = true;
  c->fused_update = false;
  c->keep_fused_grads = false;
  c->graph_clock = 0;
  if (cudaMalloc((void**)&c->dev_status, 64) != cudaSuccess ||
      cudaMemset(c->dev_status, 0, 64) != cudaSuccess) {
    delete c;
    return FAX_ERR_CUDA;
  }
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    (void)cudaGetLastError();
    cudaFree(c->dev_status);
    delete c;
    return FAX_ERR_CUDA;
  }
  c->encode_tiled = fn;
  if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->copy, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_copy_a, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_copy_b, cudaEventDisableTiming) != cudaSuccess) {
    cudaFree(c->dev_status);
    delete c;
    return FAX_ERR_CUDA;
  }
  *out = c;
  return FAX_OK;
}

extern "C" fax_status fax_destroy(fax_ctx* ctx) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  if (ctx->side) { cudaStreamSynchronize(ctx->side); cudaStreamDestroy(ctx->side); }
  if (ctx->copy) { cudaStreamSynchronize(ctx->copy); cudaStreamDestroy(ctx->copy); }
  if (ctx->ev_copy_a) cudaEventDestroy(ctx->ev_copy_a);
  if (ctx->ev_copy_b) cudaEventDestroy(ctx->ev_copy_b);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->dev_status) cudaFree(ctx->dev_status);
  for (FaxProfRec& r : ctx->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  delete ctx;
  return FAX_OK;
}

extern "C" int32_t fax_last_cuda_error(const fax_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
extern "C" uint64_t fax_launch_count(const fax_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" fax_status fax_check_device_status(fax_ctx* ctx, int32_t* detail_host) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  int32_t h[2] = {0, 0};
  FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  FAX_CUDA_TRY(ctx, cudaMemcpy(h, ctx->dev_status, sizeof(h), cudaMemcpyDeviceToHost));
  if (detail_host) *detail_host = h[1];
  if (h[0] != 0) {
    FAX_CUDA_TRY(ctx, cudaMemset(ctx->dev_status, 0, 8));
    return FAX_ERR_TIMEOUT;
  }
  return FAX_OK;
}

extern "C" fax_status fax_set_adamw_overlap(fax_ctx* ctx, int32_t enable) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  ctx->overlap_adamw = enable != 0;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_set_fused_update(fax_ctx* ctx, int32_t enable, int32_t keep_gradients) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  ctx->fused_update = enable != 0;
  ctx->keep_fused_grads = keep_gradients != 0;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_set_graph_replay(fax_ctx* ctx, int32_t enable) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  ctx->use_graphs = enable != 0;
  if (!ctx->use_graphs) { cudaStreamSynchronize(ctx->stream); fax_graph_clear(ctx); }
  return FAX_OK;
}

extern "C" fax_status fax_set_gemm_two_cta(fax_ctx* ctx, int32_t enable) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  ctx->use_2cta = enable != 0;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_set_dependent_launch(fax_ctx* ctx, int32_t enable) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  ctx->use_pdl = enable != 0;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_set_gemm_l2_budget(fax_ctx* ctx, int64_t bytes) {
  if (!ctx || bytes < 0) return FAX_ERR_INVALID_ARG;
  ctx->gemm_l2_budget = (double)bytes;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_set_attention_backward_two_chains(fax_ctx* ctx, int32_t enable) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  if (enable < 0 || enable > 2) return FAX_ERR_INVALID_ARG;
  ctx->attn_bwd_mode = enable;
  cudaStreamSynchronize(ctx->stream);
  fax_graph_clear(ctx);
  return FAX_OK;
}

extern "C" fax_status fax_profile_begin(fax_ctx* ctx) {
  if (!ctx) return FAX_ERR_INVALID_ARG;
  for (FaxProfRec& r : ctx->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  ctx->prof.clear();
  ctx->prof_on = true;
  return FAX_OK;
}

extern "C" fax_status fax_profile_end(fax_ctx* ctx, fax_profile_entry* out, int32_t n_out) {
  if (!ctx || !out || n_out < FAX_KERNEL_CLASSES) return FAX_ERR_INVALID_ARG;
  ctx->prof_on = false;
  FAX_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
  for (int i = 0; i < FAX_KERNEL_CLASSES; ++i) { out[i].launches = 0; out[i].ms = 0; out[i].flops = 0; out[i].bytes = 0; }
  for (FaxProfRec& r : ctx->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess && r.cls >= 0 && r.cls < FAX_KERNEL_CLASSES) {
      out[r.cls].launches += 1; out[r.cls].ms += ms; out[r.cls].flops += r.flops; out[r.cls].bytes += r.bytes;
    }
    cudaEventDestroy(r.e0); cudaEventDestroy(r.e1);
  }
  ctx->prof.clear();
  return FAX_OK;
}

extern "C" const char* fax_kernel_class_name(int32_t cls) {
  static const char* names[FAX_KERNEL_CLASSES] = {"gemm_tcgen05", "gemm_simt", "attention_fwd", "attention_bwd",
                                                  "layernorm_fwd", "layernorm_bwd", "adamw", "colsum", "embed", "xent"};
  return (cls >= 0 && cls < FAX_KERNEL_CLASSES) ? names[cls] : "unknown";
}
