// Masked in-chunk scores of the causal form (Section 2.2's Khat = P S^T under the lower-triangular mask, chunk by
// chunk) on the tensor cores, for the shapes that have no fused kernel (d = 128): sc[bh, c][i][j] = (j <= i) phiQ_i . phiK_j
// for the tokens i, j of chunk c, from the bf16 copies of the two feature matrices [B*H][L][M].
//
// One block = one 128 x 128 tile of a chunk's C x C score block.  Tiles above the diagonal are all zero and are only
// written.  The feature index is the contraction: 64 features of both token tiles per TMA stage (two panels with the
// 128-byte swizzle), four MMAs of N = 128 per stage into one accumulator in tensor memory; the epilogue masks the
// diagonal tile and writes the rows (fp32, bf16, or both).
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int SC_STAGES = 3;
constexpr int SC_EPI_THREADS = 128, SC_WARP_TMA = 4, SC_WARP_MMA = 5, SC_THREADS = 192;
constexpr uint32_t SC_TMEM_COLS = 128;
constexpr uint32_t SC_STAGE_BYTES = 2 * TILE_BYTES;     // 64 features of the query tile, then of the key tile

struct ScSmem {
  static constexpr uint32_t A0 = 0, MISC = SC_STAGES * SC_STAGE_BYTES, TOTAL = MISC + 256;
};
struct ScMisc {
  uint64_t full[SC_STAGES], empty[SC_STAGES], acc_full;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(ScMisc) <= 256, "misc block");

__global__ void __launch_bounds__(SC_THREADS, 2)
tc_scores128_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, float* __restrict__ sc,
                    __nv_bfloat16* __restrict__ sc16, int M, int C, int nch, int* __restrict__ status) {
  // sc (fp32) and sc16 (bf16): either may be null
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  ScMisc* misc = reinterpret_cast<ScMisc*>(sm + ScSmem::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = C / TILE, ti = blockIdx.x / nt, tj = blockIdx.x % nt;
  const int c = blockIdx.y, bh = blockIdx.z;
  const size_t toff = ((size_t)bh * nch + c) * C * C + (size_t)ti * TILE * C + (size_t)tj * TILE;
  float* S = sc + toff;
  __nv_bfloat16* S16 = sc16 + toff;
  if (tj > ti) {                               // above the diagonal: zeros (uniform over the block)
    for (int e = threadIdx.x; e < TILE * (TILE / 4); e += SC_THREADS) {
      const size_t o = (size_t)(e / (TILE / 4)) * C + 4 * (e % (TILE / 4));
      if (sc) *reinterpret_cast<float4*>(S + o) = make_float4(0.f, 0.f, 0.f, 0.f);
      if (sc16) *reinterpret_cast<uint2*>(S16 + o) = make_uint2(0u, 0u);
    }
    return;
  }
  const int nk = M / 64;
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < SC_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    mbar_init(&misc->acc_full, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == SC_WARP_MMA) {
    tmem_alloc(&misc->tmem_base, SC_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == SC_WARP_TMA) {
    if (lane == 0) {
      prefetch_tmap(&tmQ);
      prefetch_tmap(&tmK);
      const int rq = c * C + ti * TILE, rk = c * C + tj * TILE;
      int issued = 0;
      for (int ks = 0; ks < nk; ks++) {
        const int st = ks % SC_STAGES;
        if (!mbar_wait(&misc->empty[st], ((ks / SC_STAGES) & 1) ^ 1, abortp, status)) break;
        mbar_expect_tx(&misc->full[st], SC_STAGE_BYTES);
        tma_load_4d(sm + ScSmem::A0 + st * SC_STAGE_BYTES, &tmQ, &misc->full[st], 64 * ks, rq, bh, 0);
        tma_load_4d(sm + ScSmem::A0 + st * SC_STAGE_BYTES + TILE_BYTES, &tmK, &misc->full[st], 64 * ks, rk, bh, 0);
        issued = ks + 1;
      }
      // no copy of this block may still be in flight when it exits
      for (int ks = max(0, issued - SC_STAGES); ks < issued; ks++)
        mbar_wait(&misc->full[ks % SC_STAGES], (ks / SC_STAGES) & 1, abortp, status, false);
    }
  } else if (warp == SC_WARP_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues
    // (two of these blocks share an SM).
    constexpr uint32_t ID = idesc_bf16(128, 128, 0, 0);
    const uint64_t dA0 = smem_desc(smem_u32(sm + ScSmem::A0), 16, 1024, SWZ_128B);
    uint32_t al0 = (uint32_t)dA0;
    const uint32_t ah = (uint32_t)(dA0 >> 32);
    bool ok = true;
    for (int ks = 0; ks < nk; ks++) {
      const int st = ks % SC_STAGES;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[st], (ks / SC_STAGES) & 1, abortp, status))) { ok = false; break; }
      tcgen05_fence_after();
      opaque(al0);
      const uint32_t al = al0 + st * (SC_STAGE_BYTES / 16), bl = al + TILE_BYTES / 16;
      if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 4; k++) mma_bf16_lh(tmem, al + 2 * k, ah, bl + 2 * k, ah, ID, (ks | k) ? 1u : 0u);
        mma_commit(&misc->empty[st]);
        if (ks == nk - 1) mma_commit(&misc->acc_full);
      }
      __syncwarp();
    }
    (void)ok;
  } else {
    // epilogue: one score row per thread
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    if (mbar_wait(&misc->acc_full, 0, abortp, status, false)) {
      __syncwarp();
      tcgen05_fence_after();
      float* out = S + (size_t)row * C;
      __nv_bfloat16* out16 = S16 + (size_t)row * C;
      const int last = ti == tj ? row : TILE;          // columns up to `last` (inclusive) are kept
#pragma unroll
      for (int cc = 0; cc < TILE / 16; cc++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + cc * 16, t);
        tmem_wait_ld();
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; j++) v[j] = cc * 16 + j <= last ? __uint_as_float(t[j]) : 0.f;
        if (sc) {
#pragma unroll
          for (int j = 0; j < 4; j++) *reinterpret_cast<float4*>(out + cc * 16 + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
        if (sc16) {
          uint32_t o[8];
#pragma unroll
          for (int j = 0; j < 8; j++) o[j] = pack_bf16(v[2 * j], v[2 * j + 1]);
          *reinterpret_cast<uint4*>(out16 + cc * 16) = make_uint4(o[0], o[1], o[2], o[3]);
          *reinterpret_cast<uint4*>(out16 + cc * 16 + 8) = make_uint4(o[4], o[5], o[6], o[7]);
        }
      }
      tcgen05_fence_before();
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == SC_WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, SC_TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}

// bf16 feature matrices, M a multiple of 64, chunks of 128 or 256 tokens
int fs_tc_scores128_supported(int M, int C) { return M % 64 == 0 && M >= 64 && (C == 128 || C == 256); }

// phiQ16, phiK16: [BH][L][M] bf16 (L a multiple of C); sc (fp32) and sc16 (bf16): [BH * L / C][C][C], either may be null
int fs_tc_scores128(fsharp_ctx* ctx, const void* phiQ16, const void* phiK16, int BH, int L, int M, int C, float* sc, void* sc16) {
  const int nch = L / C, nt = C / TILE;
  CUtensorMap tmQ, tmK;
  TensorAddr a{(int64_t)BH * L * M, (int64_t)L * M, (int64_t)M};
  FS_TRY(tchost::make_map_tokens(&tmQ, phiQ16, a, 1, BH, L, M));
  FS_TRY(tchost::make_map_tokens(&tmK, phiK16, a, 1, BH, L, M));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_scores128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScSmem::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_SCORES128);
  tc_scores128_kernel<<<dim3(nt * nt, nch, BH), SC_THREADS, ScSmem::TOTAL + 1024, ctx->stream>>>(tmQ, tmK, sc, (__nv_bfloat16*)sc16, M, C, nch, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
