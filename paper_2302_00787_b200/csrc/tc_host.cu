// Host side of the tensor-core path: TMA descriptors and dispatch (the operand images are written by prep.cu).
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tcl;

size_t fs_tc_bidir_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal_supported(const fsharp_dims* dm, int chunk);
size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                 const int* flags, void* Y, WsAlloc* ws);
int fs_tc_bidir(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                const int* flags, void* Y, WsAlloc* ws);

namespace {

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
int make_map_rows(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner, int box_rows);
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner) {
  return make_map_rows(map, base, a, B, H, L, inner, TILE);
}

// The same with a box of 64 x box_rows (box_rows a multiple of 8, at most 256).
int make_map_rows(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FSHARP_E_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)inner, (cuuint64_t)L, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)a.sl * 2, (cuuint64_t)a.sh * 2, (cuuint64_t)a.sb * 2};
  // a dimension of size one may carry any stride; give it a legal one
  if (H == 1 && strides[1] == 0) strides[1] = strides[0] * (cuuint64_t)L;
  if (B == 1 && strides[2] == 0) strides[2] = strides[1] * (cuuint64_t)H;
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FSHARP_OK : FSHARP_E_CUDA;
}

// Output rows as TMA store tiles: 32 rows x 32 values (64 bytes), staged in shared memory with the 64-byte swizzle.
int make_map_out(CUtensorMap* map, void* base, TensorAddr a, int B, int H, int L, int inner) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FSHARP_E_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)inner, (cuuint64_t)L, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)a.sl * 2, (cuuint64_t)a.sh * 2, (cuuint64_t)a.sb * 2};
  if (H == 1 && strides[1] == 0) strides[1] = strides[0] * (cuuint64_t)L;
  if (B == 1 && strides[2] == 0) strides[2] = strides[1] * (cuuint64_t)H;
  cuuint32_t box[4] = {32, 32, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FSHARP_OK : FSHARP_E_CUDA;
}

}  // namespace tchost

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
                 int chunk, const uint8_t* images, const int* flags, void* Y, WsAlloc* ws) {
  (void)chunk;
  if (causal) return fs_tc_causal(ctx, Q, K, V, dm, images, flags, Y, ws);
  return fs_tc_bidir(ctx, Q, K, V, dm, images, flags, Y, ws);
}

// ------------------------------------------------------------------------------------------
// self-test of the bounded waits
// ------------------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(32)
bounded_wait_selftest_kernel(long long limit_cycles, int* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncwarp();
  // nothing ever arrives on `bar`: the wait runs into its limit, latches FSHARP_E_TIMEOUT and returns false
  const bool ok = tc::mbar_wait(&bar, 0, &abort_flag, status, false, limit_cycles);
  if (ok) atomicExch(status, FSHARP_E_INTERNAL);       // (a wait that returned true here would be a bug of mbar_wait)
}
}  // namespace

extern "C" int fsharp_selftest_bounded_wait(fsharp_ctx* ctx, int limit_us) {
  if (!ctx) return FSHARP_E_BADARG;
  if (limit_us < 1 || limit_us > 100000) return FSHARP_E_BADARG;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  int khz = 0;
  FS_CUDA_OK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, ctx->device));
  const long long cycles = (long long)limit_us * (long long)(khz > 0 ? khz : 1965000) / 1000;
  bounded_wait_selftest_kernel<<<1, 32, 0, ctx->stream>>>(cycles, ctx->d_status);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
