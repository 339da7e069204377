// Per-group precomputation for the feature kernels (Section 4, cost paragraph):
// W^(k) = Omega B^(k) (row m = (B^(k)T w_m)^T), a_m = w_m^T A w_m, the constant
// log D - 1/2 log M.
#include "common.cuh"

namespace {

constexpr int PREP_THREADS = 256;

__global__ void __launch_bounds__(PREP_THREADS)
prep_kernel(const float* __restrict__ Omega, int64_t omega_head_stride, const double* __restrict__ params,
            int64_t params_stride, int H, int pool, int d, int M, float* __restrict__ prep) {
  __shared__ float red[PREP_THREADS];
  __shared__ int redi[PREP_THREADS];
  const int g = blockIdx.x, side = blockIdx.y + 1, tid = threadIdx.x;
  const int h = pool == FSHARP_POOL_PER_BH ? g % H : g;
  const float* Om = Omega + (int64_t)h * omega_head_stride;
  ParamsLayout pl{d};
  PrepLayout pr{d, M};
  const double* P = params + (size_t)g * params_stride;
  const double* A = P + pl.A();
  const double* Bm = P + pl.B(side);
  const double* Cm = P + pl.C(side);
  const double* tail = P + pl.tail();
  float* out = prep + ((size_t)g * 2 + (side - 1)) * pr.total();
  float* W = out + pr.W();
  float* av = out + pr.a();
  float* scal = out + pr.scal();
  float* Cf = out + pr.Cmat();

  for (int e = tid; e < M * d; e += PREP_THREADS) {
    int m = e / d, j = e % d;
    double s = 0.0;
    for (int i = 0; i < d; i++) s = fma((double)Om[m * d + i], Bm[i * d + j], s);
    W[e] = (float)s;
  }
  float amax = -3.0e38f;
  for (int m = tid; m < M; m += PREP_THREADS) {
    double s = 0.0;
    for (int i = 0; i < d; i++) {
      double r = 0.0;
      for (int j = 0; j < d; j++) r = fma(A[i * d + j], (double)Om[m * d + j], r);
      s = fma((double)Om[m * d + i], r, s);
    }
    av[m] = (float)s;
    amax = fmaxf(amax, (float)s);
  }
  // C = gamma I exactly?
  int cscalar = 1;
  const double gamma = Cm[0];
  for (int e = tid; e < d * d; e += PREP_THREADS) {
    int i = e / d, j = e % d;
    Cf[e] = (float)Cm[e];
    if (i == j ? (Cm[e] != gamma) : (Cm[e] != 0.0)) cscalar = 0;
  }
  red[tid] = amax; redi[tid] = cscalar;
  __syncthreads();
  for (int s = PREP_THREADS / 2; s > 0; s >>= 1) {
    if (tid < s) {
      red[tid] = fmaxf(red[tid], red[tid + s]);
      redi[tid] = redi[tid] & redi[tid + s];
    }
    __syncthreads();
  }
  if (tid == 0) {
    for (int i = 0; i < 8; i++) scal[i] = 0.f;
    scal[PS_BIAS] = (float)(tail[PT_LOGD] - 0.5 * log((double)M));
    scal[PS_AMAX] = red[0];
    scal[PS_CSCALAR] = redi[0] ? 1.f : 0.f;
    scal[PS_CGAMMA] = (float)gamma;
  }
}

}  // namespace

int fs_run_prep(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                int64_t params_stride, int G, int H, int pool, int d, int M, float* prep) {
  if (G == 0) return FSHARP_OK;
  FS_TIME_BEGIN(ctx, FS_K_PREP);
  prep_kernel<<<dim3(G, 2), PREP_THREADS, 0, ctx->stream>>>(Omega, omega_head_stride, params, params_stride, H, pool, d, M,
                                                                 prep);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
