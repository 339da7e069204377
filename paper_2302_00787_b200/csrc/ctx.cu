// Context, workspace and status handling of the FAVOR# library.
#include <new>

#include "common.cuh"

extern "C" {

int fsharp_create(fsharp_ctx** out, int device, void* stream) {
  if (!out) return FSHARP_E_BADARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    (void)cudaGetLastError();
    return FSHARP_E_CUDA;
  }
  FS_CUDA_OK(cudaSetDevice(device));
  fsharp_ctx* c = new (std::nothrow) fsharp_ctx();
  if (!c) return FSHARP_E_NOMEM;
  c->device = device;
  c->stream = reinterpret_cast<cudaStream_t>(stream);
  c->impl = FSHARP_IMPL_AUTO;
  c->ws = nullptr;
  c->ws_bytes = 0;
  c->launches = 0;
  c->d_status = nullptr;
  c->sm_count = 148;
  c->timing = 0;
  c->t_used = 0;
  c->t_ev = nullptr;
  c->t_tag = nullptr;
  c->copy_stream = nullptr;
  c->down_stream = nullptr;
  c->ev_inputs = nullptr;
  c->ev_v = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) c->sm_count = prop.multiProcessorCount;
  if (cudaMalloc(&c->d_status, sizeof(int)) != cudaSuccess) {
    (void)cudaGetLastError();
    delete c;
    return FSHARP_E_NOMEM;
  }
  if (cudaMemset(c->d_status, 0, sizeof(int)) != cudaSuccess) {
    (void)cudaGetLastError();
    cudaFree(c->d_status);
    delete c;
    return FSHARP_E_CUDA;
  }
  *out = c;
  return FSHARP_OK;
}

int fsharp_destroy(fsharp_ctx* ctx) {
  if (!ctx) return FSHARP_E_BADARG;
  cudaSetDevice(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  if (ctx->ws) cudaFree(ctx->ws);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->copy_stream) {
    cudaStreamSynchronize(ctx->copy_stream);
    cudaStreamDestroy(ctx->copy_stream);
    cudaStreamSynchronize(ctx->down_stream);
    cudaStreamDestroy(ctx->down_stream);
    cudaEventDestroy(ctx->ev_inputs);
    cudaEventDestroy(ctx->ev_v);
  }
  if (ctx->t_ev) {
    for (int i = 0; i < 2 * FS_TIMING_SLOTS; i++) cudaEventDestroy(ctx->t_ev[i]);
    delete[] ctx->t_ev;
    delete[] ctx->t_tag;
  }
  delete ctx;
  return FSHARP_OK;
}

int fsharp_set_stream(fsharp_ctx* ctx, void* stream) {
  if (!ctx) return FSHARP_E_BADARG;
  ctx->stream = reinterpret_cast<cudaStream_t>(stream);
  return FSHARP_OK;
}

int fsharp_set_impl(fsharp_ctx* ctx, int impl) {
  if (!ctx || impl < FSHARP_IMPL_AUTO || impl > FSHARP_IMPL_TENSOR) return FSHARP_E_BADARG;
  ctx->impl = impl;
  return FSHARP_OK;
}

int fsharp_status(fsharp_ctx* ctx, int* code) {
  if (!ctx || !code) return FSHARP_E_BADARG;
  FS_CUDA_OK(cudaStreamSynchronize(ctx->stream));
  int h = 0;
  FS_CUDA_OK(cudaMemcpy(&h, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (h != 0) FS_CUDA_OK(cudaMemset(ctx->d_status, 0, sizeof(int)));
  *code = h;
  return FSHARP_OK;
}

int64_t fsharp_launch_count(const fsharp_ctx* ctx) { return ctx ? ctx->launches : 0; }

size_t fsharp_workspace_bytes(const fsharp_ctx* ctx) { return ctx ? ctx->ws_bytes : 0; }

const char* fsharp_strerror(int code) {
  switch (code) {
    case FSHARP_OK: return "ok";
    case FSHARP_E_BADARG: return "bad argument";
    case FSHARP_E_SHAPE: return "unsupported or inconsistent shape";
    case FSHARP_E_ALIGN: return "pointer or stride not 16-byte aligned";
    case FSHARP_E_DTYPE: return "unsupported dtype";
    case FSHARP_E_NOMEM: return "out of memory";
    case FSHARP_E_CONSTRAINT: return "parameter constraint violated (singular M or 8A not below I)";
    case FSHARP_E_NONFINITE: return "non-finite value met on the device";
    case FSHARP_E_TIMEOUT: return "bounded device-side wait expired";
    case FSHARP_E_CUDA: return "CUDA call failed";
    case FSHARP_E_LIMIT: return "problem exceeds the fixed scratch of the no-allocation entry point";
    case FSHARP_E_INTERNAL: return "index check of the debug build failed on the device";
    default: return "unknown error";
  }
}

int fsharp_set_timing(fsharp_ctx* ctx, int on) {
  if (!ctx) return FSHARP_E_BADARG;
  if (on && !ctx->t_ev) {
    FS_CUDA_OK(cudaSetDevice(ctx->device));
    ctx->t_ev = new (std::nothrow) cudaEvent_t[2 * FS_TIMING_SLOTS];
    ctx->t_tag = new (std::nothrow) int[FS_TIMING_SLOTS];
    if (!ctx->t_ev || !ctx->t_tag) return FSHARP_E_NOMEM;
    for (int i = 0; i < 2 * FS_TIMING_SLOTS; i++) FS_CUDA_OK(cudaEventCreate(&ctx->t_ev[i]));
  }
  ctx->timing = on ? 1 : 0;
  ctx->t_used = 0;
  return FSHARP_OK;
}

int fsharp_read_timing(fsharp_ctx* ctx, int cap, float* total_ms, int* launches) {
  if (!ctx || !total_ms || !launches || cap <= 0) return FSHARP_E_BADARG;
  for (int i = 0; i < cap; i++) { total_ms[i] = 0.f; launches[i] = 0; }
  if (!ctx->t_ev) return FSHARP_OK;
  FS_CUDA_OK(cudaStreamSynchronize(ctx->stream));
  for (int i = 0; i < ctx->t_used; i++) {
    float ms = 0.f;
    FS_CUDA_OK(cudaEventElapsedTime(&ms, ctx->t_ev[2 * i], ctx->t_ev[2 * i + 1]));
    int tag = ctx->t_tag[i];
    if (tag >= 0 && tag < cap) { total_ms[tag] += ms; launches[tag]++; }
  }
  ctx->t_used = 0;
  return FSHARP_OK;
}

const char* fsharp_kernel_name(int id) {
  switch (id) {
    case FS_K_STATS: return "stats_kernel";
    case FS_K_FIT: return "fit_kernel";
    case FS_K_PREP: return "prep_kernel";
    case FS_K_ROWTERM: return "rowterm_kernel";
    case FS_K_LOGITS: return "logits_kernel";
    case FS_K_GROUPMAX: return "groupmax_kernel";
    case FS_K_EXPSHIFT: return "expshift_kernel";
    case FS_K_KV: return "kv_kernel";
    case FS_K_PREFIX: return "prefix_kernel";
    case FS_K_SCORES: return "scores_kernel";
    case FS_K_OUT: return "out_kernel";
    case FS_K_PAIRS: return "pairs_kernel";
    case FS_K_PAIRVAR_PREP: return "pairvar_prep_kernel";
    case FS_K_PAIRVAR: return "pairvar_kernel";
    case FS_K_PAIRPOOL: return "pairpool_kernel";
    case FS_K_TC_KV: return "tc_kv_kernel";
    case FS_K_TC_OUT: return "tc_out_kernel";
    case FS_K_TC_CAUSAL: return "tc_causal_kernel";
    case FS_K_TC_STATS: return "tc_stats_kernel";
    case FS_K_TC_ROWTERM: return "tc_rowterm_kernel";
    case FS_K_TC_FEAT: return "tc_feat_kernel";
    case FS_K_TC_LOGITS128: return "tc_logits128_kernel";
    case FS_K_TC_SCORES128: return "tc_scores128_kernel";
    case FS_K_TC_KV128: return "tc_kv128_kernel";
    case FS_K_TC_OUT128: return "tc_out128_kernel";
    default: return "";
  }
}

size_t fsharp_stats_doubles(int d) { return StatsLayout{d}.total(); }
size_t fsharp_params_doubles(int d) { return ParamsLayout{d}.total(); }

}  // extern "C"

void fs_time_begin(fsharp_ctx* ctx, int tag) {
  if (ctx->t_used >= FS_TIMING_SLOTS) return;
  ctx->t_tag[ctx->t_used] = tag;
  cudaEventRecord(ctx->t_ev[2 * ctx->t_used], ctx->stream);
}

void fs_time_end(fsharp_ctx* ctx) {
  if (ctx->t_used >= FS_TIMING_SLOTS) return;
  cudaEventRecord(ctx->t_ev[2 * ctx->t_used + 1], ctx->stream);
  ctx->t_used++;
}

int fs_ws_reserve(fsharp_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->ws_bytes) return FSHARP_OK;
  // Growing: wait for work that may still use the old block, then replace it.
  FS_CUDA_OK(cudaStreamSynchronize(ctx->stream));
  if (ctx->ws) {
    cudaFree(ctx->ws);
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
  }
  size_t want = bytes + (bytes >> 3);
  void* p = nullptr;
  if (cudaMalloc(&p, want) != cudaSuccess) {
    (void)cudaGetLastError();
    want = bytes;
    if (cudaMalloc(&p, want) != cudaSuccess) {
      (void)cudaGetLastError();
      return FSHARP_E_NOMEM;
    }
  }
  ctx->ws = static_cast<char*>(p);
  ctx->ws_bytes = want;
  return FSHARP_OK;
}
