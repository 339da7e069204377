// fsharp_featurize_static: the feature map for callers that may not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need features: code
// that runs inside a memory-pool owner which forbids foreign allocations, a real-time loop
// that must not take the allocator's locks or trigger an implicit device synchronisation,
// or a process that has already handed every free byte of HBM to its own arena.  For them
// the scratch that fsharp_featurize takes from its context's growing workspace (the per-group
// W / a / C block, the per-token quadratic term and the per-(batch, head) maximum) is carved
// from one file-scope array that is part of the loaded module.  Every GPU that loads the
// library therefore holds FS_STATIC_SCRATCH_BYTES of device memory until the process exits.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t FS_STATIC_SCRATCH_BYTES = (size_t)8 << 20;   // 8 MiB
constexpr int FS_MAX_DEVICES = 64;

// In host code this name is only a handle for the runtime; the device address is obtained
// once per device with cudaGetSymbolAddress (device code could name the array directly).
static __device__ __align__(256) unsigned char fs_static_scratch[FS_STATIC_SCRATCH_BYTES];
static __device__ int fs_static_status;

std::mutex g_lock;
unsigned char* g_scratch_ptr[FS_MAX_DEVICES];
int* g_status_ptr[FS_MAX_DEVICES];
int g_sm_count[FS_MAX_DEVICES];

// Per-device set-up: resolves the device addresses of the two symbols.  No allocation.
int setup_device(int dev) {
  std::lock_guard<std::mutex> guard(g_lock);
  if (g_scratch_ptr[dev]) return FSHARP_OK;
  void* p = nullptr;
  void* s = nullptr;
  FS_CUDA_OK(cudaGetSymbolAddress(&p, fs_static_scratch));
  FS_CUDA_OK(cudaGetSymbolAddress(&s, fs_static_status));
  int sms = 148;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    (void)cudaGetLastError();
    sms = 148;
  }
  g_sm_count[dev] = sms;
  g_status_ptr[dev] = static_cast<int*>(s);
  g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  return FSHARP_OK;
}

}  // namespace

extern "C" size_t fsharp_static_scratch_bytes(void) { return FS_STATIC_SCRATCH_BYTES; }

extern "C" int fsharp_featurize_static(void* stream, const void* X, const float* Omega, const double* params,
                                       int side, const fsharp_dims* dims, int dtype, float qk_scale, int stab,
                                       float* phi, float* logscale, int* device_status) {
  if (!X || !Omega || !params || !phi || !dims) return FSHARP_E_BADARG;
  const int d = dims->d, M = dims->M;
  if (!(d == 16 || d == 32 || d == 64 || d == 128)) return FSHARP_E_SHAPE;
  if (M <= 0 || M % 16 != 0 || M > 1024) return FSHARP_E_SHAPE;
  if (dims->B < 0 || dims->H < 0 || dims->Lq < 0 || dims->Lk < 0) return FSHARP_E_SHAPE;
  if ((int64_t)dims->B * dims->H > 65535) return FSHARP_E_SHAPE;
  if (dims->pool != FSHARP_POOL_PER_BH && dims->pool != FSHARP_POOL_PER_HEAD) return FSHARP_E_BADARG;
  if (dtype != FSHARP_F32 && dtype != FSHARP_BF16) return FSHARP_E_DTYPE;
  if (side != 1 && side != 2) return FSHARP_E_BADARG;
  if (stab < FSHARP_STAB_NONE || stab > FSHARP_STAB_GROUP) return FSHARP_E_BADARG;
  if (stab != FSHARP_STAB_NONE && !logscale) return FSHARP_E_BADARG;
  const int L = side == 1 ? dims->Lq : dims->Lk;
  const int64_t* st = side == 1 ? dims->q_stride : dims->k_stride;
  const size_t es = dtype == FSHARP_F32 ? 4 : 2;
  if (reinterpret_cast<uintptr_t>(X) % 16 != 0) return FSHARP_E_ALIGN;
  for (int i = 0; i < 3; i++)
    if (st[i] < 0 || (st[i] * es) % 16 != 0) return FSHARP_E_ALIGN;
  const size_t BH = (size_t)dims->B * dims->H;
  if (BH == 0 || L == 0) return FSHARP_OK;

  // the fixed scratch must hold: prep block, per-token term, per-(batch, head) maximum
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{d, M}.total();
  const size_t need = ws_round(prep_f * 4) + ws_round(BH * L * 4) + ws_round(BH * 4);
  if (need > FS_STATIC_SCRATCH_BYTES) return FSHARP_E_LIMIT;

  int dev = 0;
  FS_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= FS_MAX_DEVICES) return FSHARP_E_BADARG;
  FS_TRY(setup_device(dev));

  // a context that lives on this stack frame: no workspace of its own, no event pool
  fsharp_ctx ctx;
  ctx.device = dev;
  ctx.stream = reinterpret_cast<cudaStream_t>(stream);
  ctx.impl = FSHARP_IMPL_SIMT;
  ctx.ws = reinterpret_cast<char*>(g_scratch_ptr[dev]);
  ctx.ws_bytes = FS_STATIC_SCRATCH_BYTES;
  ctx.d_status = device_status ? device_status : g_status_ptr[dev];
  ctx.launches = 0;
  ctx.sm_count = g_sm_count[dev];
  ctx.timing = 0;
  ctx.t_used = 0;
  ctx.t_ev = nullptr;
  ctx.t_tag = nullptr;
  ctx.copy_stream = nullptr;
  ctx.down_stream = nullptr;
  ctx.ev_inputs = nullptr;
  ctx.ev_v = nullptr;

  WsAlloc ws{ctx.ws, 0};
  float* prep = ws.take<float>(prep_f);
  float* rowc = ws.take<float>(BH * L);
  unsigned* gmax = ws.take<unsigned>(BH);
  // everything in the scratch is written before it is read in this call (the maximum words are
  // cleared by the feature kernels' own memset), so what an earlier call left behind is harmless
  FS_TRY(fs_run_prep(&ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{d}.total(), G, dims->H,
                     dims->pool, d, M, prep));
  return fs_simt_featurize(&ctx, X, dtype, fs_addr(st, dims->H, L, d), dims->B, dims->H, L, d, M, dims->pool, prep,
                           side, qk_scale, stab, rowc, gmax, phi, logscale);
}
