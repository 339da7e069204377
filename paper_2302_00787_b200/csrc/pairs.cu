// Kernel estimation for (x, y) pairs (Section 2.1: Khat = sum_m P_m S_m) with R feature
// draws, and the closed-form variance of Theorem 4.1 divided by M (Section 2.1).
#include "common.cuh"
#include "simt_tile.cuh"

namespace {

// c = x^T C x for the 64 pairs of a tile; 4 threads per pair.
__device__ __forceinline__ void tile_quadratic(const float* __restrict__ X, int64_t p0, int64_t np, int d,
                                               const float* __restrict__ scal, const float* __restrict__ Cm,
                                               float* out /* shared [64] */) {
  const int tid = threadIdx.x, r = tid >> 2, part = tid & 3;
  float s = 0.f;
  if (p0 + r < np) {
    const float* x = X + (p0 + r) * d;
    if (scal[PS_CSCALAR] != 0.f) {
      for (int j = part; j < d; j += 4) s = fmaf(x[j], x[j], s);
      s *= scal[PS_CGAMMA];
    } else {
      for (int j = part; j < d; j += 4) {
        float t = 0.f;
        for (int k = 0; k < d; k++) t = fmaf(x[k], Cm[k * d + j], t);
        s = fmaf(t, x[j], s);
      }
    }
  }
  s += __shfl_xor_sync(0xffffffffu, s, 1);
  s += __shfl_xor_sync(0xffffffffu, s, 2);
  if (part == 0) out[r] = s;
}

__global__ void __launch_bounds__(NTH)
pairs_kernel(const float* __restrict__ X, const float* __restrict__ Y, int64_t np, int d, int M,
             const float* __restrict__ prep, float* __restrict__ est) {
  __shared__ Tiles sm;
  __shared__ float cx[TM], cy[TM];
  const int draw = blockIdx.y;
  const int64_t p0 = (int64_t)blockIdx.x * TM;
  PrepLayout pr{d, M};
  const float* p1 = prep + ((size_t)draw * 2 + 0) * pr.total();
  const float* p2 = prep + ((size_t)draw * 2 + 1) * pr.total();
  tile_quadratic(X, p0, np, d, p1 + pr.scal(), p1 + pr.Cmat(), cx);
  tile_quadratic(Y, p0, np, d, p2 + pr.scal(), p2 + pr.Cmat(), cy);
  __syncthreads();
  const float bias2 = 2.f * p1[pr.scal() + PS_BIAS];
  const float* W1 = p1 + pr.W();
  const float* W2 = p2 + pr.W();
  const float* av = p1 + pr.a();
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float rowsum[4] = {0.f, 0.f, 0.f, 0.f};
  for (int m0 = 0; m0 < M; m0 += TN) {
    float ax[4][4] = {}, ay[4][4] = {};
    tile_gemm<true, true>(
        ax, d, [&](int r, int k) { return (p0 + r < np) ? X[(p0 + r) * d + k] : 0.f; },
        [&](int k, int c) { return (m0 + c < M) ? W1[(size_t)(m0 + c) * d + k] : 0.f; }, sm);
    tile_gemm<true, true>(
        ay, d, [&](int r, int k) { return (p0 + r < np) ? Y[(p0 + r) * d + k] : 0.f; },
        [&](int k, int c) { return (m0 + c < M) ? W2[(size_t)(m0 + c) * d + k] : 0.f; }, sm);
#pragma unroll
    for (int i = 0; i < 4; i++) {
      float base = bias2 + cx[ty + 16 * i] + cy[ty + 16 * i];
#pragma unroll
      for (int j = 0; j < 4; j++) {
        int m = m0 + tx + 16 * j;
        if (m < M) rowsum[i] += expf(base + 2.f * av[m] + ax[i][j] + ay[i][j]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++) {
    float s = rowsum[i];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    int64_t p = p0 + ty + 16 * i;
    if (tx == 0 && p < np) est[(int64_t)draw * np + p] = s;
  }
}

// E1 = 2 (C1 + B1^T R B1), E2 = 2 (C2 + B2^T R B2), E12 = 4 B1^T R B2 with R = (I - 8A)^-1
// (A diagonal), and k0 = 4 log D - 1/2 log det(I - 8A).   ev: [3 d^2 + 1] doubles.
__global__ void __launch_bounds__(NTH)
pairvar_prep_kernel(const double* __restrict__ params, int d, double* __restrict__ ev, int* __restrict__ status) {
  ParamsLayout pl{d};
  const double* A = params + pl.A();
  const double* B1 = params + pl.B(1);
  const double* B2 = params + pl.B(2);
  const double* C1 = params + pl.C(1);
  const double* C2 = params + pl.C(2);
  const int tid = threadIdx.x;
  for (int e = tid; e < d * d; e += NTH) {
    int i = e / d, j = e % d;
    if (i != j && A[e] != 0.0) atomicExch(status, FSHARP_E_CONSTRAINT);
    double s1 = 0.0, s2 = 0.0, s12 = 0.0;
    for (int l = 0; l < d; l++) {
      double r = 1.0 / (1.0 - 8.0 * A[l * d + l]);
      s1 = fma(B1[l * d + i] * r, B1[l * d + j], s1);
      s2 = fma(B2[l * d + i] * r, B2[l * d + j], s2);
      s12 = fma(B1[l * d + i] * r, B2[l * d + j], s12);
    }
    ev[e] = 2.0 * (C1[e] + s1);
    ev[d * d + e] = 2.0 * (C2[e] + s2);
    ev[2 * d * d + e] = 4.0 * s12;
  }
  if (tid == 0) {
    double ld = 0.0;
    for (int l = 0; l < d; l++) {
      double v = 1.0 - 8.0 * A[l * d + l];
      if (!(v > 0.0)) atomicExch(status, FSHARP_E_CONSTRAINT);
      ld += log(v);
    }
    ev[3 * d * d] = 4.0 * params[pl.tail() + PT_LOGD] - 0.5 * ld;
  }
}

// One warp per pair: Var = (exp(k0 + x^T E1 x + y^T E2 y + x^T E12 y) - exp(2 x^T y)) / M.
__global__ void __launch_bounds__(NTH)
pairvar_kernel(const float* __restrict__ X, const float* __restrict__ Y, int64_t np, int d, int M,
               const double* __restrict__ ev, double* __restrict__ var) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * (NTH / 32) + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * (NTH / 32);
  const double* E1 = ev;
  const double* E2 = ev + d * d;
  const double* E12 = ev + 2 * d * d;
  const double k0 = ev[3 * d * d];
  for (int64_t p = warp; p < np; p += nwarps) {
    const float* x = X + p * d;
    const float* y = Y + p * d;
    double q = 0.0, xy = 0.0;
    for (int j = lane; j < d; j += 32) {
      double t1 = 0.0, t2 = 0.0, t12 = 0.0;
      for (int k = 0; k < d; k++) {
        t1 = fma((double)x[k], E1[k * d + j], t1);
        t2 = fma((double)y[k], E2[k * d + j], t2);
        t12 = fma((double)x[k], E12[k * d + j], t12);
      }
      q += t1 * x[j] + (t2 + t12) * y[j];
      xy += (double)x[j] * (double)y[j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      q += __shfl_xor_sync(0xffffffffu, q, o);
      xy += __shfl_xor_sync(0xffffffffu, xy, o);
    }
    if (lane == 0) var[p] = (exp(k0 + q) - exp(2.0 * xy)) / (double)M;
  }
}

// Pooled relative variances (Section 5.1), one warp per pair: the unbiased sample variance of the R estimates and
// the closed-form variance, both over K^2 = exp(2 x^T y), averaged over the pairs.  pooled[0] += empirical / np,
// pooled[1] += closed form / np (fp64 atomics; pooled is zero on entry).
__global__ void __launch_bounds__(NTH)
pairpool_kernel(const float* __restrict__ X, const float* __restrict__ Y, int64_t np, int d, int R,
                const float* __restrict__ est, const double* __restrict__ var, double* __restrict__ pooled) {
  __shared__ double red[2][NTH / 32];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int64_t warp = (int64_t)blockIdx.x * (NTH / 32) + wib;
  const int64_t nwarps = (int64_t)gridDim.x * (NTH / 32);
  double acc_e = 0.0, acc_c = 0.0;                    // lane 0's running sums over this warp's pairs
  for (int64_t p = warp; p < np; p += nwarps) {
    const float* x = X + p * d;
    const float* y = Y + p * d;
    double xy = 0.0, s1 = 0.0;
    for (int j = lane; j < d; j += 32) xy += (double)x[j] * (double)y[j];
    for (int r = lane; r < R; r += 32) s1 += (double)est[(int64_t)r * np + p];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      xy += __shfl_xor_sync(0xffffffffu, xy, o);
      s1 += __shfl_xor_sync(0xffffffffu, s1, o);
    }
    const double mean = s1 / (double)R;
    double s2 = 0.0;
    for (int r = lane; r < R; r += 32) {
      const double dv = (double)est[(int64_t)r * np + p] - mean;
      s2 = fma(dv, dv, s2);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    if (lane == 0) {
      const double ik2 = exp(-2.0 * xy);
      acc_e += (R > 1 ? s2 / (double)(R - 1) : 0.0) * ik2;
      acc_c += var[p] * ik2;
    }
  }
  if (lane == 0) { red[0][wib] = acc_e; red[1][wib] = acc_c; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double e = 0.0, c = 0.0;
    for (int i = 0; i < NTH / 32; i++) { e += red[0][i]; c += red[1][i]; }
    atomicAdd(&pooled[0], e / (double)np);
    atomicAdd(&pooled[1], c / (double)np);
  }
}

}  // namespace

size_t fs_pairs_scratch_bytes(int d, int M, int R) {
  return ws_round((size_t)R * 2 * PrepLayout{d, M}.total() * sizeof(float)) +
         ws_round((3 * (size_t)d * d + 1) * sizeof(double));
}

int fs_run_pairs(fsharp_ctx* ctx, const float* X, const float* Y, const float* Omega, const double* params,
                 int64_t npairs, int d, int M, int R, float* est, double* var_cf, double* pooled, WsAlloc* ws) {
  float* prep = ws->take<float>((size_t)R * 2 * PrepLayout{d, M}.total());
  double* ev = ws->take<double>(3 * (size_t)d * d + 1);
  // one "group" per draw, all reading the same parameter blob
  FS_TRY(fs_run_prep(ctx, Omega, (int64_t)M * d, params, 0, R, R, FSHARP_POOL_PER_HEAD, d, M, prep));
  if (npairs == 0) return FSHARP_OK;
  int64_t tiles = (npairs + TM - 1) / TM;
  if (tiles > 2147483647LL) return FSHARP_E_SHAPE;
  FS_TIME_BEGIN(ctx, FS_K_PAIRS);
  pairs_kernel<<<dim3((unsigned)tiles, R), NTH, 0, ctx->stream>>>(X, Y, npairs, d, M, prep, est);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  if (var_cf) {
    FS_TIME_BEGIN(ctx, FS_K_PAIRVAR_PREP);
    pairvar_prep_kernel<<<1, NTH, 0, ctx->stream>>>(params, d, ev, ctx->d_status);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
    int64_t blocks = (npairs + 7) / 8;
    if (blocks > 8 * ctx->sm_count) blocks = 8 * ctx->sm_count;
    FS_TIME_BEGIN(ctx, FS_K_PAIRVAR);
    pairvar_kernel<<<(unsigned)blocks, NTH, 0, ctx->stream>>>(X, Y, npairs, d, M, ev, var_cf);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
    if (pooled) {
      FS_CUDA_OK(cudaMemsetAsync(pooled, 0, 2 * sizeof(double), ctx->stream));
      FS_TIME_BEGIN(ctx, FS_K_PAIRPOOL);
      pairpool_kernel<<<(unsigned)blocks, NTH, 0, ctx->stream>>>(X, Y, npairs, d, R, est, var_cf, pooled);
      FS_TIME_END(ctx);
      FS_LAUNCH_CHECK(ctx);
    }
  }
  return FSHARP_OK;
}
