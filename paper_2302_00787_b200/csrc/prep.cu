// Per-group precomputation for the feature kernels (Section 4, cost paragraph):
// W^(k) = Omega B^(k) (row m = (B^(k)T w_m)^T), a_m = w_m^T A w_m, the constant
// log D - 1/2 log M, and the bound that fixes the per-group shift of the keys.
#include "common.cuh"

namespace {

constexpr int PREP_THREADS = 256;

__global__ void __launch_bounds__(PREP_THREADS)
prep_kernel(const float* __restrict__ Omega, int64_t omega_head_stride, const double* __restrict__ params,
            int64_t params_stride, int H, int pool, int d, int M, float* __restrict__ prep) {
  __shared__ float red[PREP_THREADS];
  __shared__ float red2[PREP_THREADS];
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
  __syncthreads();   // W complete
  float wmax = 0.f;
  for (int m = tid; m < M; m += PREP_THREADS) {
    float s = 0.f;
    for (int j = 0; j < d; j++) s = fmaf(W[m * d + j], W[m * d + j], s);
    wmax = fmaxf(wmax, sqrtf(s));
  }
  red[tid] = amax; red2[tid] = wmax; redi[tid] = cscalar;
  __syncthreads();
  for (int s = PREP_THREADS / 2; s > 0; s >>= 1) {
    if (tid < s) {
      red[tid] = fmaxf(red[tid], red[tid + s]);
      red2[tid] = fmaxf(red2[tid], red2[tid + s]);
      redi[tid] = redi[tid] & redi[tid + s];
    }
    __syncthreads();
  }
  if (tid == 0) {
    amax = red[0];
    wmax = red2[0] * 1.0001f;   // round the norm bound upwards
    const float bias = (float)(tail[PT_LOGD] - 0.5 * log((double)M));
    const float kappa = (float)fmax(tail[side == 1 ? PT_KAPPA1 : PT_KAPPA2], 0.0);
    const double rho2 = tail[side == 1 ? PT_RHO2X : PT_RHO2Y];
    // exponent <= bias + a_max + max_{0 <= rho <= rho_max} (w_max rho - kappa rho^2)   (Cauchy-Schwarz)
    float lin;
    const bool rho_ok = isfinite(rho2) && rho2 >= 0.0;
    const float rhomax = rho_ok ? (float)sqrt(rho2) * 1.0001f : 0.f;
    if (kappa > 0.f) {
      float rstar = wmax / (2.f * kappa);
      lin = (!rho_ok || rhomax >= rstar) ? wmax * wmax / (4.f * kappa) : wmax * rhomax - kappa * rhomax * rhomax;
    } else {
      lin = wmax * rhomax;
    }
    scal[PS_BIAS] = bias;
    scal[PS_AMAX] = amax;
    scal[PS_WMAX] = wmax;
    scal[PS_CSCALAR] = redi[0] ? 1.f : 0.f;
    scal[PS_CGAMMA] = (float)gamma;
    scal[PS_GSHIFT] = bias + amax + lin - FS_MARGIN;
    scal[PS_KAPPA] = kappa;
    scal[PS_RHO2] = (float)rho2;
  }
}

}  // namespace

int fs_run_prep(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                int64_t params_stride, int G, int H, int pool, int d, int M, float* prep) {
  if (G == 0) return FSHARP_OK;
  prep_kernel<<<dim3(G, 2), PREP_THREADS, 0, ctx->stream>>>(Omega, omega_head_stride, params, params_stride, H, pool, d, M,
                                                                 prep);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
