// Set statistics of Theorems 4.2 and 4.3: M1 = L^-1 sum x x^T, M2 = L^-1 sum y y^T,
// mu4 = mean x, mu5 = mean y.
//
// One thread block accumulates the Gram matrix of a slice of tokens of one
// (batch, head, side): products in fp32 over 128 tokens, then folded into fp64
// registers; slices are combined with fp64 atomics.
#include "common.cuh"

namespace {

constexpr int ST_THREADS = 256;
constexpr int ST_TT = 32;        // tokens per shared-memory tile
constexpr int ST_FLUSH = 4;      // tiles between fp32 -> fp64 folds

template <typename T, int D>
__global__ void __launch_bounds__(ST_THREADS)
stats_kernel(const T* __restrict__ Q, const T* __restrict__ K, TensorAddr aq, TensorAddr ak, int H, int Lq, int Lk,
             int pool, int Bpool, float qk_scale, int tokens_per_split, double* __restrict__ stats,
             int* __restrict__ status) {
  constexpr int RB = D / 16;
  __shared__ float xs[ST_TT][D + 1];
  const int side = blockIdx.z;           // 0: queries, 1: keys
  const int bh = blockIdx.y;
  const int b = bh / H, h = bh % H;
  const int L = side ? Lk : Lq;
  const TensorAddr ad = side ? ak : aq;
  const T* X = (side ? K : Q) + b * ad.sb + h * ad.sh;
  const int t0 = blockIdx.x * tokens_per_split;
  const int t1 = min(L, t0 + tokens_per_split);
  if (t0 >= t1) return;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  float acc[RB][RB];
  double accd[RB][RB];
#pragma unroll
  for (int i = 0; i < RB; i++)
#pragma unroll
    for (int j = 0; j < RB; j++) { acc[i][j] = 0.f; accd[i][j] = 0.0; }
  float colacc = 0.f;
  double colaccd = 0.0;
  bool bad = false;
  int since = 0;

  for (int tb = t0; tb < t1; tb += ST_TT) {
    for (int e = tid; e < ST_TT * D; e += ST_THREADS) {
      int t = e / D, c = e % D;
      float v = 0.f;
      if (tb + t < t1) v = qk_scale * fs_load(X + (int64_t)(tb + t) * ad.sl + c);
      if (!isfinite(v)) bad = true;
      xs[t][c] = v;
    }
    __syncthreads();
#pragma unroll 4
    for (int t = 0; t < ST_TT; t++) {
      float a[RB], bb[RB];
#pragma unroll
      for (int i = 0; i < RB; i++) { a[i] = xs[t][ty + 16 * i]; bb[i] = xs[t][tx + 16 * i]; }
#pragma unroll
      for (int i = 0; i < RB; i++)
#pragma unroll
        for (int j = 0; j < RB; j++) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    if (tid < D) {
      float s = 0.f;
      for (int t = 0; t < ST_TT; t++) s += xs[t][tid];
      colacc += s;
    }
    __syncthreads();
    if (++since == ST_FLUSH) {
      since = 0;
#pragma unroll
      for (int i = 0; i < RB; i++)
#pragma unroll
        for (int j = 0; j < RB; j++) { accd[i][j] += (double)acc[i][j]; acc[i][j] = 0.f; }
      colaccd += (double)colacc;
      colacc = 0.f;
    }
  }
  const double inv = 1.0 / ((double)L * (double)Bpool);
  StatsLayout sl{D};
  double* out = stats + (size_t)g * sl.total();
  double* Mo = out + sl.M(side + 1);
#pragma unroll
  for (int i = 0; i < RB; i++)
#pragma unroll
    for (int j = 0; j < RB; j++)
      atomicAdd(&Mo[(size_t)(ty + 16 * i) * D + (tx + 16 * j)], (accd[i][j] + (double)acc[i][j]) * inv);
  if (tid < D) atomicAdd(&out[sl.mu(side + 4) + tid], (colaccd + (double)colacc) * inv);
  if (bad) atomicExch(status, FSHARP_E_NONFINITE);
}

template <typename T>
int launch_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dm, float qk_scale,
                 double* stats) {
  const int BH = dm->B * dm->H;
  const int Lmax = dm->Lq > dm->Lk ? dm->Lq : dm->Lk;
  int nsplit = (4 * ctx->sm_count + 2 * BH - 1) / (2 * BH);
  int maxsplit = (Lmax + 127) / 128;
  if (nsplit > maxsplit) nsplit = maxsplit;
  if (nsplit < 1) nsplit = 1;
  int tps = (Lmax + nsplit - 1) / nsplit;
  tps = (tps + ST_TT - 1) / ST_TT * ST_TT;
  nsplit = (Lmax + tps - 1) / tps;
  dim3 grid(nsplit, BH, 2);
  TensorAddr aq = fs_addr(dm->q_stride, dm->H, dm->Lq, dm->d);
  TensorAddr ak = fs_addr(dm->k_stride, dm->H, dm->Lk, dm->d);
  const int Bpool = dm->pool == FSHARP_POOL_PER_BH ? 1 : dm->B;
#define FS_ST(DD)                                                                                           \
  stats_kernel<T, DD><<<grid, ST_THREADS, 0, ctx->stream>>>((const T*)Q, (const T*)K, aq, ak, dm->H, dm->Lq, \
                                                            dm->Lk, dm->pool, Bpool, qk_scale, tps, stats,   \
                                                            ctx->d_status)
  FS_TIME_BEGIN(ctx, FS_K_STATS);
  switch (dm->d) {
    case 16: FS_ST(16); break;
    case 32: FS_ST(32); break;
    case 64: FS_ST(64); break;
    case 128: FS_ST(128); break;
    default: return FSHARP_E_SHAPE;
  }
#undef FS_ST
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}

}  // namespace

int fs_run_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dm, int dtype,
                 float qk_scale, double* stats) {
  const int G = fs_groups(dm);
  FS_CUDA_OK(cudaMemsetAsync(stats, 0, (size_t)G * StatsLayout{dm->d}.total() * sizeof(double), ctx->stream));
  if (dm->Lq == 0 && dm->Lk == 0) return FSHARP_OK;
  if (ctx->impl != FSHARP_IMPL_SIMT && fs_tc_stats_supported(Q, K, dm, dtype)) return fs_tc_stats(ctx, Q, K, dm, qk_scale, stats);
  if (dtype == FSHARP_F32) return launch_stats<float>(ctx, Q, K, dm, qk_scale, stats);
  return launch_stats<__nv_bfloat16>(ctx, Q, K, dm, qk_scale, stats);
}
