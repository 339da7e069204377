// Host side of the tensor-core path: operand images, TMA descriptors, dispatch.
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tcl;

size_t fs_tc_bidir_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal_supported(const fsharp_dims* dm, int chunk);
size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, float qk_scale,
                 const float* prep, void* Y, WsAlloc* ws);
int fs_tc_bidir(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, float qk_scale,
                const float* prep, void* Y, WsAlloc* ws);

namespace {

// Builds the per-(group, side) operand images from the fp32 prep block; block z converts a
// quarter of every array.  The flag words must be zero on entry (blocks OR their bits in).
constexpr int TCP_SPLIT = 4;
__global__ void __launch_bounds__(256)
tc_prep_kernel(const float* __restrict__ prep, float qk_scale, uint8_t* __restrict__ images, int* __restrict__ flags) {
  const int g = blockIdx.x, side = blockIdx.y, z = blockIdx.z, tid = threadIdx.x;
  PrepLayout pr{TC_D, TC_M};
  const float* pp = prep + ((size_t)g * 2 + side) * pr.total();
  const float* W = pp + pr.W();
  const float* av = pp + pr.a();
  const float* Cm = pp + pr.Cmat();
  const float* scal = pp + pr.scal();
  uint8_t* img = images + ((size_t)g * 2 + side) * IMG_BYTES;
  int* fl = flags + ((size_t)g * 2 + side) * FLAG_WORDS;
  const float sw = FS_LOG2E * qk_scale, sc = FS_LOG2E * qk_scale * qk_scale;
  constexpr int WQ = TC_M * TC_D / TCP_SPLIT, CQ = TC_D * TC_D / TCP_SPLIT, AQ = TC_M / TCP_SPLIT;
  // two neighbouring elements per thread: one 4-byte store into each image
  for (int e2 = tid; e2 < WQ / 2; e2 += 256) {
    const int e = z * WQ + 2 * e2, m = e / TC_D, k = e % TC_D;
    const float2 w2 = *reinterpret_cast<const float2*>(W + e);
    const float v0 = w2.x * sw, v1 = w2.y * sw;
    const __nv_bfloat16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
    *reinterpret_cast<__nv_bfloat162*>(img + IMG_W + tc::sw128_offset(m, k)) = __nv_bfloat162(h0, h1);
    *reinterpret_cast<__nv_bfloat162*>(img + IMG_WLO + tc::sw128_offset(m, k)) =
        __nv_bfloat162(__float2bfloat16_rn(v0 - __bfloat162float(h0)), __float2bfloat16_rn(v1 - __bfloat162float(h1)));
  }
  int lo_nonzero = 0;
  for (int e = z * CQ + tid; e < (z + 1) * CQ; e += 256) {
    int k = e / TC_D, n = e % TC_D;          // C[k][n] goes to row n, column k of the B operand
    float v = Cm[e] * sc;
    __nv_bfloat16 hi = __float2bfloat16_rn(v);
    __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    if (__bfloat162float(lo) != 0.f) lo_nonzero = 1;
    *reinterpret_cast<__nv_bfloat16*>(img + IMG_CHI + tc::sw128_offset(n, k)) = hi;
    *reinterpret_cast<__nv_bfloat16*>(img + IMG_CLO + tc::sw128_offset(n, k)) = lo;
  }
  if (tid < AQ) reinterpret_cast<float*>(img + IMG_A2)[z * AQ + tid] = 2.f * FS_LOG2E * av[z * AQ + tid];
  if (__syncthreads_or(lo_nonzero) && tid == 0) atomicOr(&fl[0], FLAG_C_LO);
  if (z == 0 && tid == 0) {
    if (scal[PS_CSCALAR] == 0.f) atomicOr(&fl[0], FLAG_C_DENSE);
    fl[1] = __float_as_int(scal[PS_CGAMMA] * sc);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

namespace tchost {

// [B, H, L, inner] bf16 tensor with element strides a -> 4-D map (inner, token, head, batch),
// box 64 x 128 x 1 x 1, 128-byte swizzle; rows beyond L read as zero.
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FSHARP_E_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)inner, (cuuint64_t)L, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)a.sl * 2, (cuuint64_t)a.sh * 2, (cuuint64_t)a.sb * 2};
  // a dimension of size one may carry any stride; give it a legal one
  if (H == 1 && strides[1] == 0) strides[1] = strides[0] * (cuuint64_t)L;
  if (B == 1 && strides[2] == 0) strides[2] = strides[1] * (cuuint64_t)H;
  cuuint32_t box[4] = {64, (cuuint32_t)TILE, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FSHARP_OK : FSHARP_E_CUDA;
}

// kvt [BH, 80, 256] fp16 or bf16 -> 3-D map (feature, row, bh), box 64 x 80 x 1, 128-byte swizzle.
int make_map_kvt(CUtensorMap* map, const void* base, int BH, int bf16) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FSHARP_E_CUDA;
  cuuint64_t dims[3] = {(cuuint64_t)TC_M, (cuuint64_t)TC_NV, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)TC_M * 2, (cuuint64_t)TC_M * TC_NV * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)TC_NV, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FSHARP_OK : FSHARP_E_CUDA;
}

// bf16 features [BH, Lpad, 256] -> 3-D map (feature, token, bh), box 64 x 128 x 1, 128-byte swizzle.
int make_map_feat(CUtensorMap* map, const void* base, int BH, int Lpad) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FSHARP_E_CUDA;
  cuuint64_t dims[3] = {(cuuint64_t)TC_M, (cuuint64_t)Lpad, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)TC_M * 2, (cuuint64_t)TC_M * 2 * (cuuint64_t)Lpad};
  cuuint32_t box[3] = {64, (cuuint32_t)TILE, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FSHARP_OK : FSHARP_E_CUDA;
}

}  // namespace tchost

int fs_tc_prep(fsharp_ctx* ctx, const float* prep, int G, float qk_scale, uint8_t* images, int* flags) {
  FS_CUDA_OK(cudaMemsetAsync(flags, 0, (size_t)G * 2 * FLAG_WORDS * sizeof(int), ctx->stream));
  FS_TIME_BEGIN(ctx, FS_K_TC_PREP);
  tc_prep_kernel<<<dim3(G, 2, TCP_SPLIT), 256, 0, ctx->stream>>>(prep, qk_scale, images, flags);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}

int fs_tc_supported(const fsharp_dims* dm, int dtype, int causal, int chunk, float qk_scale) {
  (void)chunk;
  (void)qk_scale;
  if (dtype != FSHARP_BF16) return 0;
  if (dm->d != TC_D || dm->dv != TC_DV || dm->M != TC_M) return 0;
  if (dm->Lq <= 0 || dm->Lk <= 0) return 0;
  if (causal) return fs_tc_causal_supported(dm, chunk);
  return 1;
}

size_t fs_tc_attend_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm, int causal, int chunk) {
  (void)chunk;
  return causal ? fs_tc_causal_scratch_bytes(ctx, dm) : fs_tc_bidir_scratch_bytes(ctx, dm);
}

int fs_tc_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, int causal,
                 int chunk, float qk_scale, const float* prep, void* Y, WsAlloc* ws) {
  (void)chunk;
  if (causal) return fs_tc_causal(ctx, Q, K, V, dm, qk_scale, prep, Y, ws);
  return fs_tc_bidir(ctx, Q, K, V, dm, qk_scale, prep, Y, ws);
}
