// Shared declarations of the FAVOR# library: context, blob layouts, launch helpers.
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/fsharp.h"

#define FS_LOG2E 1.4426950408889634f

// Layout of the per-group parameter blob (doubles); see fsharp_params_doubles().
struct ParamsLayout {
  int d;
  __host__ __device__ size_t dd() const { return (size_t)d * d; }
  __host__ __device__ size_t A() const { return 0; }
  __host__ __device__ size_t B(int k) const { return dd() * (size_t)k; }        // k = 1, 2
  __host__ __device__ size_t C(int k) const { return dd() * (size_t)(2 + k); }  // k = 1, 2
  __host__ __device__ size_t tail() const { return 5 * dd(); }
  __host__ __device__ size_t total() const { return 5 * dd() + 8; }
};
enum { PT_LOGD = 0, PT_OBJ = 1, PT_PHI = 2 };   // tail[3..7] reserved (zero)

struct StatsLayout {
  int d;
  __host__ __device__ size_t M(int k) const { return (size_t)d * d * (size_t)(k - 1); }               // k = 1, 2
  __host__ __device__ size_t mu(int k) const { return 2 * (size_t)d * d + (size_t)d * (k - 4); }      // k = 4, 5
  __host__ __device__ size_t total() const { return 2 * (size_t)d * d + 2 * (size_t)d; }
};

// What prep produces per (group, side): everything the feature kernels need (fp32).
//   W      [M, d]  row m = (B^T w_m)^T
//   a      [M]     w_m^T A w_m
//   scal   [8]     see PS_* below
//   Cmat   [d, d]  copy of C (row-major)
struct PrepLayout {
  int d, M;
  __host__ __device__ size_t W() const { return 0; }
  __host__ __device__ size_t a() const { return (size_t)M * d; }
  __host__ __device__ size_t scal() const { return (size_t)M * d + M; }
  __host__ __device__ size_t Cmat() const { return (size_t)M * d + M + 8; }
  __host__ __device__ size_t total() const { return (size_t)M * d + M + 8 + (size_t)d * d; }
};
// PS_BIAS logD - 1/2 log M; PS_CSCALAR 1 if C = gamma I; PS_CGAMMA gamma.
enum { PS_BIAS = 0, PS_CSCALAR = 3, PS_CGAMMA = 4 };

// Kernel ids for the optional per-kernel timing (fsharp_set_timing / fsharp_read_timing).
enum {
  FS_K_STATS = 1, FS_K_FIT, FS_K_PREP, FS_K_ROWTERM, FS_K_LOGITS, FS_K_GROUPMAX, FS_K_EXPSHIFT, FS_K_KV,
  FS_K_PREFIX, FS_K_SCORES, FS_K_OUT, FS_K_PAIRS, FS_K_PAIRVAR_PREP, FS_K_PAIRVAR, FS_K_PAIRPOOL,
  FS_K_TC_KV, FS_K_TC_OUT, FS_K_TC_CAUSAL, FS_K_TC_STATS, FS_K_TC_ROWTERM, FS_K_TC_FEAT, FS_K_TC_LOGITS128, FS_K_TC_SCORES128, FS_K_TC_KV128, FS_K_TC_OUT128,
  FS_K_COUNT
};
constexpr int FS_TIMING_SLOTS = 4096;

struct fsharp_ctx {
  int device;
  cudaStream_t stream;
  int impl;
  char* ws;
  size_t ws_bytes;
  int* d_status;      // device status word
  int64_t launches;
  int sm_count;
  // timing: pairs of events around each launch while enabled
  int timing;
  int t_used;
  cudaEvent_t* t_ev;  // 2 * FS_TIMING_SLOTS, created on first use
  int* t_tag;
  // the two copy streams and events of fsharp_forward_host (uploads, downloads and the path overlap batch element by
  // batch element); created on first use
  cudaStream_t copy_stream, down_stream;
  cudaEvent_t ev_inputs, ev_v;
};

// NVTX range of a host-side stage (a no-op unless a tool that listens to NVTX is attached)
struct FsRange {
  explicit FsRange(const char* name) { nvtxRangePushA(name); }
  ~FsRange() { nvtxRangePop(); }
  FsRange(const FsRange&) = delete;
  FsRange& operator=(const FsRange&) = delete;
};
#define FS_RANGE(name) FsRange fs_range_guard_(name)

// Programmatic dependent launch: a kernel launched with fs_launch_chained may be scheduled while the kernel before it
// in the stream is still draining; it must not touch global memory before fs_grid_dependency_wait() (which returns
// when that kernel has completed and its writes are visible), and it lets ITS successor be scheduled only after that
// wait, so everything older than its predecessor is complete as well.  Launched the ordinary way both calls do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void fs_grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t fs_launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

void fs_time_begin(fsharp_ctx* ctx, int tag);
void fs_time_end(fsharp_ctx* ctx);
#define FS_TIME_BEGIN(ctx, tag) do { if ((ctx)->timing) fs_time_begin((ctx), (tag)); } while (0)
#define FS_TIME_END(ctx) do { if ((ctx)->timing) fs_time_end((ctx)); } while (0)

// Bump allocator over the context workspace.
struct WsAlloc {
  char* base;
  size_t off;
  template <typename T>
  T* take(size_t n) {
    size_t bytes = (n * sizeof(T) + 255) & ~(size_t)255;
    T* p = reinterpret_cast<T*>(base + off);
    off += bytes;
    return p;
  }
};
static inline size_t ws_round(size_t bytes) { return (bytes + 255) & ~(size_t)255; }

int fs_ws_reserve(fsharp_ctx* ctx, size_t bytes);   // grows the workspace; FSHARP_OK or error

#define FS_CUDA_OK(expr)                         \
  do {                                           \
    cudaError_t _e = (expr);                     \
    if (_e != cudaSuccess) {                     \
      (void)cudaGetLastError();                  \
      return FSHARP_E_CUDA;                      \
    }                                            \
  } while (0)

#define FS_LAUNCH_CHECK(ctx)                                   \
  do {                                                         \
    (ctx)->launches++;                                         \
    if (cudaPeekAtLastError() != cudaSuccess) {                \
      (void)cudaGetLastError();                                \
      return FSHARP_E_CUDA;                                    \
    }                                                          \
  } while (0)

#define FS_TRY(expr)                 \
  do {                               \
    int _rc = (expr);                \
    if (_rc != FSHARP_OK) return _rc; \
  } while (0)

// Resolved addressing of one [B,H,L,inner] tensor.
struct TensorAddr {
  int64_t sb, sh, sl;
};
static inline TensorAddr fs_addr(const int64_t s[3], int H, int L, int inner) {
  TensorAddr t;
  if (s[0] == 0 && s[1] == 0 && s[2] == 0) {
    t.sl = inner;
    t.sh = (int64_t)L * inner;
    t.sb = (int64_t)H * L * inner;
  } else {
    t.sb = s[0];
    t.sh = s[1];
    t.sl = s[2];
  }
  return t;
}

__device__ __forceinline__ float fs_load(const float* p) { return *p; }
__device__ __forceinline__ float fs_load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void fs_store(float* p, float v) { *p = v; }
__device__ __forceinline__ void fs_store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

static inline int fs_groups(const fsharp_dims* dm) {
  return dm->pool == FSHARP_POOL_PER_BH ? dm->B * dm->H : dm->H;
}

// ---- stage entry points (host side, defined in the .cu files) -------------
int fs_run_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dm, int dtype,
                 float qk_scale, double* stats);
// Tensor-core statistics (bf16, d = 64, 16-byte aligned rows); `stats` must already be zero.
int fs_tc_stats_supported(const void* Q, const void* K, const fsharp_dims* dm, int dtype);
int fs_tc_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dm, float qk_scale, double* stats);
int fs_run_fit(fsharp_ctx* ctx, const double* stats, int G, int d, int variant, double ridge,
               double* params, double* scratch);
size_t fs_fit_scratch_doubles(int G, int d);
// params_stride: doubles between the blobs of two groups (0 = every group reads the same blob)
int fs_run_prep(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                int64_t params_stride, int G, int H, int pool, int d, int M, float* prep /* [G][2][PrepLayout] */);
// The same, and (images != nullptr; d = 64, M = 256) the tensor-core path's operand images and flag words too.
int fs_run_prep_images(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                       int64_t params_stride, int G, int H, int pool, int d, int M, float* prep, float qk_scale,
                       uint8_t* images, int* flags);
// rowc: scratch [B*H*L] floats.  gmax: scratch [B*H] words.  phi: [B,H,L,M] floats.
int fs_simt_featurize(fsharp_ctx* ctx, const void* X, int dtype, TensorAddr ax, int B, int H, int L, int d,
                      int M, int pool, const float* prep, int side, float qk_scale, int stab,
                      float* rowc, unsigned* gmax, float* phi, float* logscale);
// Exponents of bf16 tokens with d = 128 on the tensor cores (tc_logits128.cu); phi [B*H][L][M] fp32, rowc [B*H][L].
int fs_tc_logits128_supported(const void* X, int dtype, TensorAddr ax, int L, int d, int M);
int fs_tc_logits128(fsharp_ctx* ctx, const void* X, TensorAddr ax, int B, int H, int L, int M, int pool, const float* prep,
                    int side, float qk_scale, const float* rowc, float* phi);
// Masked in-chunk scores from bf16 feature matrices [BH][L][M] on the tensor cores (tc_scores128.cu); sc [BH * L / C][C][C] fp32.
int fs_tc_scores128_supported(int M, int C);
int fs_tc_scores128(fsharp_ctx* ctx, const void* phiQ16, const void* phiK16, int BH, int L, int M, int C, float* sc, void* sc16);
// Per-chunk key-side sums from the bf16 copy of phi(K) on the tensor cores (tc_kv128.cu); st [BH * L / C][129][M] fp32.
int fs_tc_kv128_supported(const void* V, TensorAddr av, int dv, int M, int C);
int fs_tc_kv128(fsharp_ctx* ctx, const void* phiK16, const void* V, TensorAddr av, int B, int H, int L, int M, int C, float* st);
// Query side of the causal chunked form from bf16 copies of phi(Q), the running sums and the scores (tc_out128.cu).
int fs_tc_out128_supported(const void* Y, TensorAddr ay);
int fs_tc_out128(fsharp_ctx* ctx, const void* phiQ16, const void* st16, const void* sc16, const void* V, TensorAddr av, void* Y,
                 TensorAddr ay, int B, int H, int L, int M, int C);
int fs_simt_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm,
                   int dtype, int causal, int chunk, float qk_scale, const float* prep, void* Y,
                   WsAlloc* ws);
size_t fs_simt_attend_scratch_bytes(const fsharp_dims* dm, int causal, int chunk);
int fs_simt_kernel_apply(fsharp_ctx* ctx, const void* X, const void* Yset, const void* Cmat, const fsharp_dims* dm,
                         int dtype, float qk_scale, const float* prep, void* out, WsAlloc* ws);
size_t fs_backward_scratch_bytes(const fsharp_dims* dm, int causal, int chunk);
int fs_backward(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const void* dY, const fsharp_dims* dm,
                int dtype, int causal, int chunk, float qk_scale, const float* prep, void* dQ, void* dK, void* dV,
                WsAlloc* ws);
int fs_shift_c(fsharp_ctx* ctx, const double* params, double* out, int G, int d, double alpha);
int fs_run_pairs(fsharp_ctx* ctx, const float* X, const float* Y, const float* Omega, const double* params,
                 int64_t npairs, int d, int M, int R, float* est, double* var_cf, double* pooled, WsAlloc* ws);
size_t fs_pairs_scratch_bytes(int d, int M, int R);
