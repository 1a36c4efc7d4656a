// CUDA-graph replay of the whole-step calls.  A step is a fixed sequence of a few dozen to a
// few hundred launches whose arguments do not change from one step to the next, except the
// AdamW scalars (learning rate, bias corrections).  The second time a step is requested with
// the same configuration and the same buffers it is captured into a graph; later steps patch
// the AdamW nodes' scalars and launch the graph, which removes the per-launch gaps.
#include "graph.cuh"

#include <cstring>

uint64_t fax_hash_bytes(uint64_t h, const void* data, size_t n) {
  const unsigned char* p = (const unsigned char*)data;
  for (size_t i = 0; i < n; ++i) { h ^= p[i]; h *= 1099511628211ull; }
  return h;
}

void fax_graph_clear(fax_ctx* ctx) {
  for (FaxGraphEntry& e : ctx->graphs) {
    if (e.exec) cudaGraphExecDestroy(e.exec);
    if (e.graph) cudaGraphDestroy(e.graph);
  }
  ctx->graphs.clear();
}

static fax_status patch_and_launch(fax_ctx* ctx, FaxGraphEntry& e, const fax_adamw_hparams* hp) {
  unsigned char sc[32];
  fax_adamw_scalars(hp, sc);
  for (size_t i = 0; i < e.adam_nodes.size(); ++i) {
    cudaKernelNodeParams np = e.adam_params[i];
    void* args[2] = {np.kernelParams[0], sc};
    np.kernelParams = args;
    FAX_CUDA_TRY(ctx, cudaGraphExecKernelNodeSetParams(e.exec, e.adam_nodes[i], &np));
  }
  // weight-gradient GEMMs with AdamW in their epilogue carry the scalars inside their parameter struct
  for (FaxGemmPatch& g : e.gemm_nodes) {
    memcpy(g.blob.data() + g.sc_offset, sc, 6 * sizeof(float));
    cudaKernelNodeParams np = g.params;
    void* args[3] = {np.kernelParams[0], np.kernelParams[1], g.blob.data()};
    np.kernelParams = args;
    FAX_CUDA_TRY(ctx, cudaGraphExecKernelNodeSetParams(e.exec, g.node, &np));
  }
  FAX_CUDA_TRY(ctx, cudaGraphLaunch(e.exec, ctx->stream));
  ctx->launches += e.launches;
  e.last_use = ++ctx->graph_clock;
  return FAX_OK;
}

fax_status fax_run_step(fax_ctx* ctx, const FaxStepKey& key, const fax_adamw_hparams* hp,
                        const std::function<fax_status()>& enqueue) {
  if (!ctx->use_graphs || ctx->prof_on || !hp) return enqueue();
  for (FaxGraphEntry& e : ctx->graphs)
    if (e.key == key.hash && e.material == key.material) {
      if (e.exec) return patch_and_launch(ctx, e, hp);
      if (e.failed) return enqueue();
      // second request with this key: capture
      cudaGraph_t graph = nullptr;
      const uint64_t launches_before = ctx->launches;
      if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        (void)cudaGetLastError();
        e.failed = true;
        return enqueue();
      }
      fax_status s = enqueue();
      cudaError_t ce = cudaStreamEndCapture(ctx->stream, &graph);
      const uint64_t n_launch = ctx->launches - launches_before;
      ctx->launches = launches_before;
      if (s != FAX_OK || ce != cudaSuccess || !graph) {
        (void)cudaGetLastError();
        if (graph) cudaGraphDestroy(graph);
        e.failed = true;
        return s != FAX_OK ? s : enqueue();
      }
      cudaGraphExec_t exec = nullptr;
      if (cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaGraphDestroy(graph);
        e.failed = true;
        return enqueue();
      }
      // find the AdamW kernel nodes: their second argument (the scalars) changes every step
      size_t n_nodes = 0;
      cudaGraphGetNodes(graph, nullptr, &n_nodes);
      std::vector<cudaGraphNode_t> nodes(n_nodes);
      if (n_nodes) cudaGraphGetNodes(graph, nodes.data(), &n_nodes);
      for (cudaGraphNode_t nd : nodes) {
        cudaGraphNodeType t;
        if (cudaGraphNodeGetType(nd, &t) != cudaSuccess || t != cudaGraphNodeTypeKernel) continue;
        cudaKernelNodeParams np;
        if (cudaGraphKernelNodeGetParams(nd, &np) != cudaSuccess) continue;
        if (fax_adamw_is_kernel(np.func)) { e.adam_nodes.push_back(nd); e.adam_params.push_back(np); continue; }
        size_t psize = 0, sc_off = 0;
        if (np.kernelParams && (fax_gemm_patch_info_2cta(np.func, np.kernelParams[2], &psize, &sc_off) ||
                                fax_gemm_patch_info_1cta(np.func, np.kernelParams[2], &psize, &sc_off))) {
          FaxGemmPatch gp;
          gp.node = nd; gp.params = np; gp.sc_offset = sc_off;
          gp.blob.assign((const unsigned char*)np.kernelParams[2], (const unsigned char*)np.kernelParams[2] + psize);
          e.gemm_nodes.push_back(gp);
        }
      }
      e.graph = graph; e.exec = exec; e.launches = n_launch;
      return patch_and_launch(ctx, e, hp);
    }
  // first request with this key: run as is and remember it
  if (ctx->graphs.size() >= 8) {
    size_t victim = 0;
    for (size_t i = 1; i < ctx->graphs.size(); ++i)
      if (ctx->graphs[i].last_use < ctx->graphs[victim].last_use) victim = i;
    if (ctx->graphs[victim].exec) cudaGraphExecDestroy(ctx->graphs[victim].exec);
    if (ctx->graphs[victim].graph) cudaGraphDestroy(ctx->graphs[victim].graph);
    ctx->graphs.erase(ctx->graphs.begin() + victim);
  }
  FaxGraphEntry e;
  e.key = key.hash; e.material = key.material; e.graph = nullptr; e.exec = nullptr; e.failed = false; e.launches = 0; e.last_use = ++ctx->graph_clock;
  ctx->graphs.push_back(e);
  return enqueue();
}
