// Query side of the causal chunked form (Section 2.2 with Khat = P S^T under the lower-triangular mask) on the tensor
// cores for the shapes that have no fused kernel (bf16, dv = 128, M a multiple of 128, chunks of 128 or 256):
//   [num | den]_i = phi(Q)_i KV_c + sum_{j <= i in chunk c} sc_ij [V_j | 1],   Y_i = num_i / den_i
// with KV_c the sum of the earlier chunks' key-side sums (bf16 copy, [129][M], feature index contiguous) and sc the
// masked in-chunk scores (bf16 copy, [C][C]).
//
// One block = one 128-token tile.  First the features are the contraction (128 per stage: phi(Q) and the rows of
// KV_c as K-major operands, N = 128 for the numerators and N = 16 for the normaliser's row), then the chunk's keys up
// to the tile's last token (128 per stage: the scores K-major, V as an MN-major operand, the ones column from a
// constant tile).  One accumulator of 144 columns in tensor memory; the epilogue divides and writes bf16 rows.
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int OU_ST = 3;
constexpr int OUE_THREADS = 128, OUW_TMA = 4, OUW_MMA = 5, OUT_T = 192;
constexpr uint32_t OU_TMEM_COLS = 256;                 // 128 numerators + 16 (normaliser in the first)
constexpr uint32_t OU_DEN_BYTES = 2048;                // 16 rows x 128 bytes
constexpr uint32_t OU_STAGE = 4 * TILE_BYTES + 2 * OU_DEN_BYTES;   // A panels 0, 1; B panels 0, 1; normaliser rows of panels 0, 1

struct OuSm {
  static constexpr uint32_t A0 = 0, ONES = OU_ST * OU_STAGE, MISC = ONES + TILE_BYTES, TOTAL = MISC + 256;
};
struct OuMs {
  uint64_t full[OU_ST], empty[OU_ST], acc_full;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(OuMs) <= 256, "misc block");
static_assert(OU_STAGE % 1024 == 0 && OuSm::TOTAL + 1024 <= 232448, "shared memory budget");

__global__ void __launch_bounds__(OUT_T, 1)
tc_out128_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmS,
                 const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmC,
                 const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ Y, TensorAddr ay, int H, int L, int M,
                 int C, int nch, int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  OuMs* misc = reinterpret_cast<OuMs*>(sm + OuSm::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
  const int tpc = C / TILE, c = tile / tpc, ti = tile % tpc;
  const int nf = M / 128;                      // stages over the features
  const int nkt = ti + 1;                      // stages over the chunk's keys
  const int nst = nf + nkt;
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < OU_ST; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    mbar_init(&misc->acc_full, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  for (int i = threadIdx.x; i < (int)(TILE_BYTES / 16); i += OUT_T) reinterpret_cast<uint4*>(sm + OuSm::ONES)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (threadIdx.x < TILE)
    *reinterpret_cast<__nv_bfloat16*>(sm + OuSm::ONES + sw128_offset(threadIdx.x, 0)) = __float2bfloat16(1.f);
  fence_proxy_async_smem();
  if (warp == OUW_MMA) {
    tmem_alloc(&misc->tmem_base, OU_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == OUW_TMA) {
    if (lane == 0) {
      prefetch_tmap(&tmQ); prefetch_tmap(&tmS); prefetch_tmap(&tmD); prefetch_tmap(&tmC); prefetch_tmap(&tmV);
      const int tok = tile * TILE, unit = bh * nch + c;
      int issued = 0;
      for (int it = 0; it < nst; it++) {
        const int s = it % OU_ST;
        if (!mbar_wait(&misc->empty[s], ((it / OU_ST) & 1) ^ 1, abortp, status)) break;
        uint8_t* base = sm + OuSm::A0 + s * OU_STAGE;
        if (it < nf) {
          const int x = it * 128;
          mbar_expect_tx(&misc->full[s], OU_STAGE);
          tma_load_4d(base, &tmQ, &misc->full[s], x, tok, bh, 0);
          tma_load_4d(base + TILE_BYTES, &tmQ, &misc->full[s], x + 64, tok, bh, 0);
          tma_load_4d(base + 2 * TILE_BYTES, &tmS, &misc->full[s], x, 0, unit, 0);
          tma_load_4d(base + 3 * TILE_BYTES, &tmS, &misc->full[s], x + 64, 0, unit, 0);
          tma_load_4d(base + 4 * TILE_BYTES, &tmD, &misc->full[s], x, 128, unit, 0);
          tma_load_4d(base + 4 * TILE_BYTES + OU_DEN_BYTES, &tmD, &misc->full[s], x + 64, 128, unit, 0);
        } else {
          const int kt = it - nf;
          mbar_expect_tx(&misc->full[s], 4 * TILE_BYTES);
          tma_load_4d(base, &tmC, &misc->full[s], kt * 128, ti * TILE, unit, 0);
          tma_load_4d(base + TILE_BYTES, &tmC, &misc->full[s], kt * 128 + 64, ti * TILE, unit, 0);
          tma_load_4d(base + 2 * TILE_BYTES, &tmV, &misc->full[s], 0, c * C + kt * TILE, h, b);
          tma_load_4d(base + 3 * TILE_BYTES, &tmV, &misc->full[s], 64, c * C + kt * TILE, h, b);
        }
        issued = it + 1;
      }
      // no copy of this block may still be in flight when it exits
      for (int it = max(0, issued - OU_ST); it < issued; it++)
        mbar_wait(&misc->full[it % OU_ST], (it / OU_ST) & 1, abortp, status, false);
    }
  } else if (warp == OUW_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues.
    constexpr uint32_t ID_KK = idesc_bf16(128, 128, 0, 0), ID_KK16 = idesc_bf16(128, 16, 0, 0);    // both K-major
    constexpr uint32_t ID_KM = idesc_bf16(128, 128, 0, 1), ID_KM16 = idesc_bf16(128, 16, 0, 1);    // B MN-major
    const uint32_t sA0 = smem_u32(sm + OuSm::A0), sOnes = smem_u32(sm + OuSm::ONES);
    for (int it = 0; it < nst; it++) {
      const int s = it % OU_ST;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[s], (it / OU_ST) & 1, abortp, status))) break;
      tcgen05_fence_after();
      const uint32_t sA = sA0 + s * OU_STAGE, sB = sA + 2 * TILE_BYTES, sD = sA + 4 * TILE_BYTES;
      const uint64_t dA = smem_desc(sA, 16, 1024, SWZ_128B);
      uint32_t al = (uint32_t)dA;
      const uint32_t ah = (uint32_t)(dA >> 32);
      if (it < nf) {
        const uint64_t dB = smem_desc(sB, 16, 1024, SWZ_128B), dD = smem_desc(sD, 16, 1024, SWZ_128B);
        uint32_t bl = (uint32_t)dB, dl = (uint32_t)dD;
        opaque(al); opaque(bl); opaque(dl);
        if (lane == 0) {
#pragma unroll
          for (int p = 0; p < 2; p++)
#pragma unroll
            for (int k = 0; k < 4; k++) {
              const uint32_t first = (it | p | k) ? 1u : 0u;
              mma_bf16_lh(tmem, al + p * (TILE_BYTES / 16) + 2 * k, ah, bl + p * (TILE_BYTES / 16) + 2 * k, ah, ID_KK, first);
              mma_bf16_lh(tmem + 128, al + p * (TILE_BYTES / 16) + 2 * k, ah, dl + p * (OU_DEN_BYTES / 16) + 2 * k, ah, ID_KK16, first);
            }
          mma_commit(&misc->empty[s]);
        }
      } else {
        // V: two 64-column panels (leading offset = their distance), 16 keys per step = 16 rows of 128 bytes
        const uint64_t dV = smem_desc(sB, TILE_BYTES, 1024, SWZ_128B), dE = smem_desc(sOnes, TILE_BYTES, 1024, SWZ_128B);
        uint32_t vl = (uint32_t)dV, el = (uint32_t)dE;
        const uint32_t vh = (uint32_t)(dV >> 32), eh = (uint32_t)(dE >> 32);
        opaque(al); opaque(vl); opaque(el);
        if (lane == 0) {
#pragma unroll
          for (int k = 0; k < 8; k++) {
            const uint32_t a = al + (k >> 2) * (TILE_BYTES / 16) + 2 * (k & 3);
            mma_bf16_lh(tmem, a, ah, vl + k * 128, vh, ID_KM, 1u);
            mma_bf16_lh(tmem + 128, a, ah, el + k * 128, eh, ID_KM16, 1u);
          }
          mma_commit(&misc->empty[s]);
          if (it == nst - 1) mma_commit(&misc->acc_full);
        }
      }
      __syncwarp();
    }
  } else {
    // epilogue: one token row per thread
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    if (mbar_wait(&misc->acc_full, 0, abortp, status, false)) {
      __syncwarp();
      tcgen05_fence_after();
      uint32_t dd[8];
      tmem_ld8(lane_addr + 128, dd);
      tmem_wait_ld();
      const float den = __uint_as_float(dd[0]);
      const int64_t tok = (int64_t)tile * TILE + row;
      if (tok < L && (!(den > 0.f) || !isfinite(den))) atomicExch(status, FSHARP_E_NONFINITE);
      const float inv = 1.f / den;
      __nv_bfloat16* out = Y + b * ay.sb + h * ay.sh + tok * ay.sl;
#pragma unroll
      for (int cc = 0; cc < 8; cc++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + cc * 16, t);
        tmem_wait_ld();
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; j++) o[j] = pack_bf16(inv * __uint_as_float(t[2 * j]), inv * __uint_as_float(t[2 * j + 1]));
        if (tok < L) {
          *reinterpret_cast<uint4*>(out + cc * 16) = make_uint4(o[0], o[1], o[2], o[3]);
          *reinterpret_cast<uint4*>(out + cc * 16 + 8) = make_uint4(o[4], o[5], o[6], o[7]);
        }
      }
      tcgen05_fence_before();
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == OUW_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, OU_TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
int make_map_rows(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner, int box_rows);
}

// Y: bf16 [B,H,L,128] with 16-byte aligned rows
int fs_tc_out128_supported(const void* Y, TensorAddr ay) {
  if (reinterpret_cast<uintptr_t>(Y) % 16 != 0) return 0;
  return (ay.sl * 2) % 16 == 0 && (ay.sh * 2) % 16 == 0 && (ay.sb * 2) % 16 == 0;
}

// phiQ16 [BH][L][M], st16 [BH * L / C][129][M] (sums of the earlier chunks), sc16 [BH * L / C][C][C] (masked scores),
// all bf16; V, Y [B,H,L,128] bf16
int fs_tc_out128(fsharp_ctx* ctx, const void* phiQ16, const void* st16, const void* sc16, const void* V, TensorAddr av, void* Y,
                 TensorAddr ay, int B, int H, int L, int M, int C) {
  const int BH = B * H, nch = L / C;
  CUtensorMap tmQ, tmS, tmD, tmC, tmV;
  TensorAddr aq{(int64_t)BH * L * M, (int64_t)L * M, (int64_t)M};
  TensorAddr as{(int64_t)BH * nch * 129 * M, (int64_t)129 * M, (int64_t)M};
  TensorAddr ac{(int64_t)BH * nch * C * C, (int64_t)C * C, (int64_t)C};
  FS_TRY(tchost::make_map_tokens(&tmQ, phiQ16, aq, 1, BH, L, M));
  FS_TRY(tchost::make_map_tokens(&tmS, st16, as, 1, BH * nch, 129, M));
  FS_TRY(tchost::make_map_rows(&tmD, st16, as, 1, BH * nch, 129, M, 16));
  FS_TRY(tchost::make_map_tokens(&tmC, sc16, ac, 1, BH * nch, C, C));
  FS_TRY(tchost::make_map_tokens(&tmV, V, av, B, H, L, 128));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_out128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)OuSm::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_OUT128);
  tc_out128_kernel<<<dim3(L / TILE, BH), OUT_T, OuSm::TOTAL + 1024, ctx->stream>>>(tmQ, tmS, tmD, tmC, tmV, (__nv_bfloat16*)Y, ay, H,
                                                                                  L, M, C, nch, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
