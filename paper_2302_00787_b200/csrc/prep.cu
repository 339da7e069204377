// Per-group precomputation for the feature kernels (Section 4, cost paragraph):
// W^(k) = Omega B^(k) (row m = (B^(k)T w_m)^T), a_m = w_m^T A w_m, the constant
// log D - 1/2 log M.
#include "common.cuh"

namespace {

constexpr int PREP_THREADS = 256;
constexpr int PREP_MB = 64;                   // features per block
constexpr int PREP_LDO = PREP_MB + 4;         // row stride of the transposed Omega chunk (keeps 16-byte alignment)

// One block = one (group, side, chunk of 64 features).  Omega's chunk (transposed) and the d x d
// matrix (B, then A) sit in shared memory in fp32; every thread owns a 4 x d/16 tile of the
// 64 x d product and walks the inner index with vector loads.
template <int D>
__global__ void __launch_bounds__(PREP_THREADS)
prep_kernel(const float* __restrict__ Omega, int64_t omega_head_stride, const double* __restrict__ params,
            int64_t params_stride, int H, int pool, int M, float* __restrict__ prep) {
  constexpr int d = D, NC = D / 16;
  __shared__ int redi[PREP_THREADS];
  extern __shared__ __align__(16) float stage[];
  float* Ot = stage;                          // [d][PREP_LDO]: Ot[i][m] = Omega[m0 + m][i]
  float* Ms = stage + d * PREP_LDO;           // [d][d]
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

  const int m0 = blockIdx.z * PREP_MB;
  const int ty = tid >> 4, tx = tid & 15;     // rows m0 + 4 ty + u, columns NC tx + v
  for (int e = tid; e < PREP_MB * d; e += PREP_THREADS) {
    const int m = e % PREP_MB, i = e / PREP_MB;
    Ot[i * PREP_LDO + m] = (m0 + m < M) ? Om[(size_t)(m0 + m) * d + i] : 0.f;
  }
  for (int pass = 0; pass < 2; pass++) {      // pass 0: W = Omega B, pass 1: a = diag(Omega A Omega^T)
    const double* Mat = pass == 0 ? Bm : A;
    __syncthreads();
    for (int e = tid; e < d * d; e += PREP_THREADS) Ms[e] = (float)Mat[e];
    __syncthreads();
    float acc[4][NC];
#pragma unroll
    for (int u = 0; u < 4; u++)
#pragma unroll
      for (int v = 0; v < NC; v++) acc[u][v] = 0.f;
#pragma unroll 4
    for (int i = 0; i < d; i++) {
      const float4 a4 = *reinterpret_cast<const float4*>(Ot + i * PREP_LDO + 4 * ty);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w};
      float b[NC];
      if (NC >= 4) {
#pragma unroll
        for (int v4 = 0; v4 < NC / 4; v4++) {
          const float4 b4 = *reinterpret_cast<const float4*>(Ms + i * d + NC * tx + 4 * v4);
          b[4 * v4] = b4.x; b[4 * v4 + 1] = b4.y; b[4 * v4 + 2] = b4.z; b[4 * v4 + 3] = b4.w;
        }
      } else {
#pragma unroll
        for (int v = 0; v < NC; v++) b[v] = Ms[i * d + NC * tx + v];
      }
#pragma unroll
      for (int u = 0; u < 4; u++)
#pragma unroll
        for (int v = 0; v < NC; v++) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
    }
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const int m = m0 + 4 * ty + u;
      if (pass == 0) {
        if (m < M) {
#pragma unroll
          for (int v = 0; v < NC; v++) W[(size_t)m * d + NC * tx + v] = acc[u][v];
        }
      } else {
        // a_m = sum_j (Omega A)_mj Omega_mj, summed over the 16 threads that share row m
        float sacc = 0.f;
#pragma unroll
        for (int v = 0; v < NC; v++) sacc = fmaf(acc[u][v], Ot[(NC * tx + v) * PREP_LDO + 4 * ty + u], sacc);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, o);
        if (tx == 0 && m < M) av[m] = sacc;
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
  const dim3 grid(G, 2, (M + PREP_MB - 1) / PREP_MB);
  const size_t smem = ((size_t)d * PREP_LDO + (size_t)d * d) * sizeof(float);
#define FS_PREP(DD)                                                                                                  \
  do {                                                                                                               \
    FS_CUDA_OK(cudaFuncSetAttribute(prep_kernel<DD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));        \
    FS_TIME_BEGIN(ctx, FS_K_PREP);                                                                                    \
    prep_kernel<DD><<<grid, PREP_THREADS, smem, ctx->stream>>>(Omega, omega_head_stride, params, params_stride, H,   \
                                                               pool, M, prep);                                       \
  } while (0)
  switch (d) {
    case 16: FS_PREP(16); break;
    case 32: FS_PREP(32); break;
    case 64: FS_PREP(64); break;
    case 128: FS_PREP(128); break;
    default: return FSHARP_E_SHAPE;
  }
#undef FS_PREP
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
