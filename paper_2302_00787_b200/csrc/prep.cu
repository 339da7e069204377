// Per-group precomputation for the feature kernels (Section 4, cost paragraph):
// W^(k) = Omega B^(k) (row m = (B^(k)T w_m)^T), a_m = w_m^T A w_m, the constant
// log D - 1/2 log M.
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

namespace {

constexpr int PREP_THREADS = 256;
constexpr int PREP_MB = 64;                   // features per block
constexpr int PREP_LDO = PREP_MB + 1;         // row stride of the transposed Omega chunk: odd, so that the transposing stores
                                              // (32 consecutive rows, one column) fall into 32 different banks

// One block = one (group, role, chunk of 64 features) with role 0, 1: W of side 1, 2; role 2: a (the same for both
// sides, written for both); role 3: C, the scalars and the flags of side blockIdx.z + 1.  Omega's chunk
// (transposed) and the d x d matrix (B or A) sit in shared memory in fp32; every thread owns a 4 x d/16 tile of
// the 64 x d product and walks the inner index with vector loads.  The roles are separate blocks because a
// block's time is the latency of its dependent global loads: short blocks side by side finish sooner.
template <int D>
__global__ void __launch_bounds__(PREP_THREADS)
prep_kernel(const float* __restrict__ Omega, int64_t omega_head_stride, const double* __restrict__ params,
            int64_t params_stride, int H, int pool, int M, float* __restrict__ prep, float qk_scale,
            uint8_t* __restrict__ images, int* __restrict__ img_flags) {
  fs_grid_dependency_wait();
  // images != nullptr (d = 64, M = 256 only): the tensor-core path's operand images of this (group, side)
  // are written as well, in the layouts of tc_layout.cuh
  constexpr int d = D, NC = D / 16;
  __shared__ int redi[PREP_THREADS];
  extern __shared__ __align__(16) float stage[];
  float* Ot = stage;                          // [d][PREP_LDO]: Ot[i][m] = Omega[m0 + m][i]
  float* Ms = stage + d * PREP_LDO;           // [d][d]
  const int g = blockIdx.x, role = blockIdx.y, tid = threadIdx.x;
  const int side = role == 3 ? (int)blockIdx.z + 1 : (role == 1 ? 2 : 1);
  if (role == 3 ? blockIdx.z >= 2 : (int)blockIdx.z * PREP_MB >= M) return;
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
  if (role < 3) {
    // pass 0 (roles 0, 1): W = Omega B; pass 1 (role 2): a = diag(Omega A Omega^T)
    const int pass = role == 2 ? 1 : 0;
    const double* Mat = pass == 0 ? Bm : A;
    // global loads in batches of eight ahead of the shared-memory stores (a store between two loads would keep
    // the second load from being issued early)
    for (int e0 = tid; e0 < PREP_MB * d; e0 += 8 * PREP_THREADS) {    // coalesced read, transposed store
      float v[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * PREP_THREADS, m = e / d, i = e % d;
        v[q] = (e < PREP_MB * d && m0 + m < M) ? Om[(size_t)(m0 + m) * d + i] : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * PREP_THREADS, m = e / d, i = e % d;
        if (e < PREP_MB * d) Ot[i * PREP_LDO + m] = v[q];
      }
    }
    for (int e0 = tid; e0 < d * d; e0 += 8 * PREP_THREADS) {
      double v[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * PREP_THREADS;
        v[q] = e < d * d ? Mat[e] : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * PREP_THREADS;
        if (e < d * d) Ms[e] = (float)v[q];
      }
    }
    __syncthreads();
    float acc[4][NC];
#pragma unroll
    for (int u = 0; u < 4; u++)
#pragma unroll
      for (int v = 0; v < NC; v++) acc[u][v] = 0.f;
#pragma unroll 4
    for (int i = 0; i < d; i++) {
      const float* ap = Ot + i * PREP_LDO + 4 * ty;       // (two addresses per warp: broadcast reads)
      const float a[4] = {ap[0], ap[1], ap[2], ap[3]};
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
          // (the fp32 copy serves the fp32 kernels only; the tensor-core path reads the operand image)
          if (images == nullptr) {
#pragma unroll
            for (int v = 0; v < NC; v++) W[(size_t)m * d + NC * tx + v] = acc[u][v];
          } else {
            // log2e * qk_scale * W rounded to fp16, two neighbours per store
            uint8_t* img = images + ((size_t)g * 2 + (side - 1)) * tcl::IMG_BYTES;
            const float sw = FS_LOG2E * qk_scale;
#pragma unroll
            for (int v = 0; v + 1 < NC; v += 2)
              *reinterpret_cast<__half2*>(img + tcl::IMG_WH + tc::sw128_offset(m, NC * tx + v)) =
                  __floats2half2_rn(acc[u][v] * sw, acc[u][v + 1] * sw);
          }
        }
      } else {
        // a_m = sum_j (Omega A)_mj Omega_mj, summed over the 16 threads that share row m
        float sacc = 0.f;
#pragma unroll
        for (int v = 0; v < NC; v++) sacc = fmaf(acc[u][v], Ot[(NC * tx + v) * PREP_LDO + 4 * ty + u], sacc);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, o);
        if (tx == 0 && m < M) {
          av[m] = sacc;
          av[pr.total() + m] = sacc;          // side 2's copy
          if (images != nullptr) {
            reinterpret_cast<float*>(images + ((size_t)g * 2 + 0) * tcl::IMG_BYTES + tcl::IMG_A2)[m] = 2.f * FS_LOG2E * sacc;
            reinterpret_cast<float*>(images + ((size_t)g * 2 + 1) * tcl::IMG_BYTES + tcl::IMG_A2)[m] = 2.f * FS_LOG2E * sacc;
          }
        }
      }
    }
    return;
  }
  // C = gamma I exactly?  The operand images (row j, column i = C[i][j], 128-byte swizzle) are put together in shared
  // memory and leave in 16-byte pieces: element-wise stores of a transposed 2-byte layout would touch a sector each.
  int cscalar = 1, lo_nonzero = 0;
  const double gamma = Cm[0];
  uint8_t* simg = reinterpret_cast<uint8_t*>(stage);             // [hi image | lo image], IMG_C_BYTES each (d = 64 only)
  for (int e0 = tid; e0 < d * d; e0 += 8 * PREP_THREADS) {
    double cv[8];
#pragma unroll
    for (int q = 0; q < 8; q++) {
      const int e = e0 + q * PREP_THREADS;
      cv[q] = e < d * d ? Cm[e] : 0.0;
    }
#pragma unroll
    for (int q = 0; q < 8; q++) {
      const int e = e0 + q * PREP_THREADS;
      if (e >= d * d) continue;
      const int i = e / d, j = e % d;
      if (images == nullptr) Cf[e] = (float)cv[q];
      if (i == j ? (cv[q] != gamma) : (cv[q] != 0.0)) cscalar = 0;
      if (images != nullptr) {
        // log2e * qk_scale^2 * C[i][j] goes to row j, column i of the MMA operand
        const float v = (float)cv[q] * (FS_LOG2E * qk_scale * qk_scale);
        const __nv_bfloat16 hi = __float2bfloat16_rn(v), lo = __float2bfloat16_rn(v - __bfloat162float(hi));
        if (__bfloat162float(lo) != 0.f) lo_nonzero = 1;
        *reinterpret_cast<__nv_bfloat16*>(simg + tc::sw128_offset(j, i)) = hi;
        *reinterpret_cast<__nv_bfloat16*>(simg + tcl::IMG_C_BYTES + tc::sw128_offset(j, i)) = lo;
      }
    }
  }
  lo_nonzero = __syncthreads_or(lo_nonzero);
  if (images != nullptr) {
    // the two images are adjacent in the operand image block as well (IMG_CLO = IMG_CHI + IMG_C_BYTES)
    uint4* dst = reinterpret_cast<uint4*>(images + ((size_t)g * 2 + (side - 1)) * tcl::IMG_BYTES + tcl::IMG_CHI);
    const uint4* src = reinterpret_cast<const uint4*>(simg);
    for (int e = tid; e < (int)(2 * tcl::IMG_C_BYTES / 16); e += PREP_THREADS) dst[e] = src[e];
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
    if (images != nullptr) {
      int* fl = img_flags + ((size_t)g * 2 + (side - 1)) * tcl::FLAG_WORDS;
      fl[0] = (redi[0] ? 0 : tcl::FLAG_C_DENSE) | (lo_nonzero ? tcl::FLAG_C_LO : 0);
      fl[1] = __float_as_int((float)gamma * (FS_LOG2E * qk_scale * qk_scale));
    }
  }
}

}  // namespace

int fs_run_prep(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                int64_t params_stride, int G, int H, int pool, int d, int M, float* prep) {
  return fs_run_prep_images(ctx, Omega, omega_head_stride, params, params_stride, G, H, pool, d, M, prep, 1.f, nullptr, nullptr);
}

int fs_run_prep_images(fsharp_ctx* ctx, const float* Omega, int64_t omega_head_stride, const double* params,
                       int64_t params_stride, int G, int H, int pool, int d, int M, float* prep, float qk_scale,
                       uint8_t* images, int* flags) {
  FS_RANGE("operand images");
  if (G == 0) return FSHARP_OK;
  if (images != nullptr && (d != tcl::TC_D || M != tcl::TC_M)) return FSHARP_E_SHAPE;
  const int nchunks = (M + PREP_MB - 1) / PREP_MB;
  const dim3 grid(G, 4, nchunks > 2 ? nchunks : 2);
  const size_t smem = ((size_t)d * PREP_LDO + (size_t)d * d) * sizeof(float);
#define FS_PREP(DD)                                                                                                  \
  do {                                                                                                               \
    FS_CUDA_OK(cudaFuncSetAttribute(prep_kernel<DD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));        \
    FS_TIME_BEGIN(ctx, FS_K_PREP);                                                                                    \
    (void)fs_launch_chained(prep_kernel<DD>, grid, dim3(PREP_THREADS), smem, ctx->stream, Omega, omega_head_stride, params, params_stride, H,   \
                                                               pool, M, prep, qk_scale, images, flags);              \
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
