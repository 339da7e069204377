// Per-group precomputation for the feature kernels (Section 4, cost paragraph):
// W^(k) = Omega B^(k) (row m = (B^(k)T w_m)^T), a_m = w_m^T A w_m, the constant
// log D - 1/2 log M.
#include "common.cuh"

namespace {

constexpr int PREP_THREADS = 256;

__global__ void __launch_bounds__(PREP_THREADS)
prep_kernel(const float* __restrict__ Omega, int64_t omega_head_stride, const double* __restrict__ params,
            int64_t params_stride, int H, int pool, int d, int M, float* __restrict__ prep) {
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

  // W = Omega B and a = diag(Omega A Omega^T) in fp32 (both end up in fp32 / bf16 operands);
  // B and A are staged through shared memory 32 rows at a time.
  extern __shared__ float stage[];            // [32][d] slice of B or A, then Omega rows per warp
  float* slice = stage;                       // 32 * d
  const int lane = tid & 31, warp = tid >> 5;
  for (int pass = 0; pass < 2; pass++) {      // pass 0: W (matrix B), pass 1: a (matrix A)
    const double* Mat = pass == 0 ? Bm : A;
    {
      const int m0 = blockIdx.z * 64;          // one block per chunk of 64 features
      // each thread owns outputs (m, j): m = m0 + warp + 8 * u, j = lane + 32 * v
      float acc[8][4];
#pragma unroll
      for (int u = 0; u < 8; u++)
#pragma unroll
        for (int v = 0; v < 4; v++) acc[u][v] = 0.f;
      for (int i0 = 0; i0 < d; i0 += 32) {
        __syncthreads();
        for (int e = tid; e < 32 * d; e += PREP_THREADS)
          slice[e] = (i0 + e / d < d) ? (float)Mat[(size_t)(i0 + e / d) * d + (e % d)] : 0.f;
        __syncthreads();
#pragma unroll
        for (int u = 0; u < 8; u++) {
          const int m = m0 + warp + 8 * u;
          const float om = (m < M && i0 + lane < d) ? Om[(size_t)m * d + i0 + lane] : 0.f;   // Omega[m][i0 + lane]
#pragma unroll 8
          for (int ii = 0; ii < 32; ii++) {
            const float o = __shfl_sync(0xffffffffu, om, ii);
#pragma unroll
            for (int v = 0; v < 4; v++)
              if (lane + 32 * v < d) acc[u][v] = fmaf(o, slice[ii * d + lane + 32 * v], acc[u][v]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int m = m0 + warp + 8 * u;
        if (m < M) {
          if (pass == 0) {
#pragma unroll
            for (int v = 0; v < 4; v++)
              if (lane + 32 * v < d) W[(size_t)m * d + lane + 32 * v] = acc[u][v];
          } else {
            // a_m = sum_j (Omega A)_mj Omega_mj
            float sacc = 0.f;
#pragma unroll
            for (int v = 0; v < 4; v++)
              if (lane + 32 * v < d) sacc = fmaf(acc[u][v], Om[(size_t)m * d + lane + 32 * v], sacc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, o);
            if (lane == 0) av[m] = sacc;
          }
        }
      }
    }
  }
  if (blockIdx.z != 0) return;
  // C = gamma I exactly?
  int cscalar = 1;
  const double gamma = Cm[0];
  for (int e = tid; e < d * d; e += PREP_THREADS) {
    int i = e / d, j = e % d;
    Cf[e] = (float)Cm[e];
    if (i == j ? (Cm[e] != gamma) : (Cm[e] != 0.0)) cscalar = 0;
  }
  redi[tid] = cscalar;
  __syncthreads();
  for (int s = PREP_THREADS / 2; s > 0; s >>= 1) {
    if (tid < s) redi[tid] = redi[tid] & redi[tid + s];
    __syncthreads();
  }
  if (tid == 0) {
    for (int i = 0; i < 8; i++) scal[i] = 0.f;
    scal[PS_BIAS] = (float)(tail[PT_LOGD] - 0.5 * log((double)M));
    scal[PS_CSCALAR] = redi[0] ? 1.f : 0.f;
    scal[PS_CGAMMA] = (float)gamma;
  }
}

}  // namespace

int fs_run_prep(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                int64_t params_stride, int G, int H, int pool, int d, int M, float* prep) {
  if (G == 0) return FSHARP_OK;
  FS_TIME_BEGIN(ctx, FS_K_PREP);
  prep_kernel<<<dim3(G, 2, (M + 63) / 64), PREP_THREADS, 32 * (size_t)d * sizeof(float), ctx->stream>>>(Omega, omega_head_stride, params, params_stride, H, pool, d, M,
                                                                 prep);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
