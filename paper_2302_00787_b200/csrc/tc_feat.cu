// Tensor-core path, the feature map alone (Section 4's DERF with Section 2.1's M^-1/2) for bf16, d = 64, M = 256:
//
//   phi[i, m] * exp(logscale[i]) = M^-1/2 D exp(w_m^T A w_m + w_m^T B x_i + x_i^T C x_i)
//
// with the same arithmetic as the attention kernels: the token tile is converted to fp16 in shared memory,
// the logits are one tcgen05 product with the fp16 image of W plus one more K step that adds log2e w^T A w
// (an A operand [1, 1, 0, ...] in tensor memory, the term as an fp16 value and its remainder in the B operand),
// the per-token term comes from tc_rowterm_kernel, and the exponentials are shared between the special-function
// unit and the multiply-add pipe.  Row shift (the row's largest exponent) or no shift; phi is float32 [B,H,L,M].
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int FT_STAGES = 3;
constexpr int FT_WARP_CVT = WARP_MMA + 1;
constexpr int FT_POLY_PAIRS = 1;
struct FtSmem {
  static constexpr uint32_t X0 = 0, WH = FT_STAGES * TILE_BYTES, ROWMAX = WH + IMG_W_BYTES, AOP = ROWMAX + 2 * 2 * TILE * 4,
                            MISC = AOP + TC_M * 32, TOTAL = MISC + 256;
};
struct FtMisc {
  uint64_t full[FT_STAGES], conv[FT_STAGES], empty[FT_STAGES], logits_full, logits_free, const_bar;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr uint32_t FT_COL_LOGITS = 0, FT_COL_ONE = 256;      // tensor memory columns: logits, then the A operand of the extra K step

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_feat_kernel(const __grid_constant__ CUtensorMap tmX, const uint8_t* __restrict__ images, const float* __restrict__ crow,
               const float* __restrict__ prep, int side, int H, int pool, int L, int Lpad, int tiles_per_split, int stab,
               float* __restrict__ phi, float* __restrict__ logscale, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  FtMisc* misc = reinterpret_cast<FtMisc*>(sm + FtSmem::MISC);
  float* rowmax = reinterpret_cast<float*>(sm + FtSmem::ROWMAX);   // [tile % 2][half][row]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = blockIdx.x * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  const uint8_t* img = images + ((size_t)g * 2 + (side - 1)) * IMG_BYTES;
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < FT_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->conv[i], 1); mbar_init(&misc->empty[i], 1); }
    mbar_init(&misc->logits_full, 1);
    mbar_init(&misc->logits_free, EPI_THREADS / 32);
    mbar_init(&misc->const_bar, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  // log2e w_m^T A w_m = a2_m / 2 as an fp16 value and its fp16 remainder: K elements 0 and 1 of row m
  if (threadIdx.x < TC_M) {
    const float a = 0.5f * reinterpret_cast<const float*>(img + IMG_A2)[threadIdx.x];
    const __half hi = __float2half_rn(a), lo = __float2half_rn(a - __half2float(hi));
    uint8_t* rowp = sm + FtSmem::AOP + (threadIdx.x >> 3) * 256 + (threadIdx.x & 7) * 16;
    *reinterpret_cast<uint4*>(rowp) = make_uint4((uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16), 0, 0, 0);
    *reinterpret_cast<uint4*>(rowp + 128) = make_uint4(0, 0, 0, 0);
  }
  fence_proxy_async_smem();
  if (warp == WARP_MMA) {
    tmem_alloc(&misc->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp >= WARP_TMA) {
    regs_release<REGS_PRODUCER>();
    if (warp == WARP_TMA) {
      if (lane == 0) {
        prefetch_tmap(&tmX);
        mbar_expect_tx(&misc->const_bar, IMG_W_BYTES);
        bulk_load(sm + FtSmem::WH, img + IMG_WH, IMG_W_BYTES, &misc->const_bar);
        int issued = 0;
        for (int it = 0; it < ntiles; it++) {
          const int st = it % FT_STAGES;
          if (!mbar_wait(&misc->empty[st], ((it / FT_STAGES) & 1) ^ 1, abortp, status)) break;
          mbar_expect_tx(&misc->full[st], TILE_BYTES);
          tma_load_4d(sm + FtSmem::X0 + st * TILE_BYTES, &tmX, &misc->full[st], 0, (tile0 + it) * TILE, h, b);
          issued = it + 1;
        }
        mbar_wait(&misc->const_bar, 0, abortp, status, false);
        for (int it = max(0, issued - FT_STAGES); it < issued; it++)
          mbar_wait(&misc->full[it % FT_STAGES], (it / FT_STAGES) & 1, abortp, status, false);
      }
    } else if (warp == FT_WARP_CVT) {
      for (int it = 0; it < ntiles; it++) {
        const int st = it % FT_STAGES;
        if (!mbar_wait(&misc->full[st], (it / FT_STAGES) & 1, abortp, status, false)) break;
        uint4* xt = reinterpret_cast<uint4*>(sm + FtSmem::X0 + st * TILE_BYTES);
#pragma unroll 4
        for (int i = 0; i < (int)(TILE_BYTES / 16) / 32; i++) {
          uint4 u = xt[lane + i * 32];
          u.x = pack_f16(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
          u.y = pack_f16(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
          u.z = pack_f16(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
          u.w = pack_f16(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
          xt[lane + i * 32] = u;
        }
        fence_proxy_async_smem();
        mbar_arrive_warp(&misc->conv[st], lane);
      }
    } else if (warp == WARP_MMA) {
      constexpr uint32_t ID_LOGITS = idesc_f16(128, TC_M, 0, 0);
      const uint64_t dX0 = smem_desc(smem_u32(sm + FtSmem::X0), 16, 1024, SWZ_128B);
      const uint64_t dW = smem_desc(smem_u32(sm + FtSmem::WH), 16, 1024, SWZ_128B);
      const uint64_t dA = smem_desc(smem_u32(sm + FtSmem::AOP), 128, 256, SWZ_NONE);
      uint32_t xl = (uint32_t)dX0, wl = (uint32_t)dW, al = (uint32_t)dA;
      const uint32_t xh = (uint32_t)(dX0 >> 32), wh = (uint32_t)(dW >> 32), ah = (uint32_t)(dA >> 32);
      for (int it = 0; it < ntiles; it++) {
        const int st = it % FT_STAGES;
        opaque(xl); opaque(wl); opaque(al);
        if (it == 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->const_bar, 0, abortp, status))) break;
        if (!__all_sync(0xffffffffu, mbar_wait(&misc->conv[st], (it / FT_STAGES) & 1, abortp, status))) break;
        // the epilogue arrives once before the first tile (after writing the A operand of the extra K step), then once
        // per tile when it has taken the logits out of tensor memory
        if (!__all_sync(0xffffffffu, mbar_wait(&misc->logits_free, it & 1, abortp, status))) break;
        tcgen05_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < TC_D / 16; k++)
            mma_bf16_lh(tmem + FT_COL_LOGITS, xl + st * (TILE_BYTES / 16) + 2 * k, xh, wl + 2 * k, wh, ID_LOGITS, k > 0);
          mma_bf16_ta_lh(tmem + FT_COL_LOGITS, tmem + FT_COL_ONE, al, ah, ID_LOGITS, 1u);
          mma_commit(&misc->logits_full);
          mma_commit(&misc->empty[st]);
        }
        __syncwarp();
      }
    }
  } else {
    regs_acquire<REGS_EPILOGUE>();
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    if (hf == 0) {
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %2, %2, %2, %2, %2, %2};" ::"r"(lane_addr + FT_COL_ONE),
                   "r"(0x3C003C00u), "r"(0u) : "memory");
      tmem_wait_st();
    }
    tcgen05_fence_before();
    mbar_arrive_warp(&misc->logits_free, lane);
    const PrepLayout prl{TC_D, TC_M};
    const float bias = prep[((size_t)g * 2 + (side - 1)) * prl.total() + prl.scal() + PS_BIAS];      // log D - 1/2 log M
    const float* cptr = crow + (size_t)bh * Lpad + (size_t)tile0 * TILE + row;
    float* phib = phi + (size_t)bh * L * TC_M;
    for (int it = 0; it < ntiles; it++) {
      FS_DBG(tile0 + it < total_tiles && (size_t)tile0 * TILE + (size_t)(it + 1) * TILE <= (size_t)Lpad && row < TILE, status);
      FS_DBG(FT_COL_LOGITS + TC_M <= FT_COL_ONE && FT_COL_ONE + 8 <= TMEM_COLS, status);
      const float ci = cptr[(size_t)it * TILE];
      if (!mbar_wait(&misc->logits_full, it & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      uint32_t v[128];
#pragma unroll
      for (int c = 0; c < 8; c++) tmem_ld16(lane_addr + FT_COL_LOGITS + hf * 128 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->logits_free, lane);
      float shift2;                                            // what is subtracted, in log2 units
      if (stab == FSHARP_STAB_ROW) {
        float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
          mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
          mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
          mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
        }
        float mx = fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3]));
        rowmax[(it & 1) * 2 * TILE + hf * TILE + row] = mx;
        named_bar_sync(2 + q, 64);
        mx = fmaxf(mx, rowmax[(it & 1) * 2 * TILE + (hf ^ 1) * TILE + row]);
        shift2 = mx;
      } else {
        shift2 = -(ci + bias * FS_LOG2E);                      // no shift: the whole exponent goes into phi
      }
      const int64_t r = (int64_t)(tile0 + it) * TILE + row;
      if (stab == FSHARP_STAB_ROW && hf == 0 && r < L) logscale[(size_t)bh * L + r] = (shift2 + ci) * 0.6931471805599453f + bias;
      float* out = phib + r * TC_M + hf * 128;
#pragma unroll
      for (int c = 0; c < 32; c++) {
        float o[4];
#pragma unroll
        for (int j = 0; j < 2; j++) {
          uint32_t& e0 = v[c * 4 + 2 * j];
          uint32_t& e1 = v[c * 4 + 2 * j + 1];
          add2(e0, e1, -shift2, -shift2);
          if (((c * 2 + j) & 3) < FT_POLY_PAIRS) {
            exp2_poly2(e0, e1);
            o[2 * j] = __uint_as_float(e0);
            o[2 * j + 1] = __uint_as_float(e1);
          } else {
            o[2 * j] = ex2(__uint_as_float(e0));
            o[2 * j + 1] = ex2(__uint_as_float(e1));
          }
        }
        if (r < L) *reinterpret_cast<float4*>(out + c * 4) = make_float4(o[0], o[1], o[2], o[3]);
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}
int fs_tc_rowterm_side(fsharp_ctx* ctx, const void* X, const fsharp_dims* dm, int side, const uint8_t* images, const int* flags,
                       int Lpad, float* crow);

int fs_tc_featurize_supported(const fsharp_dims* dm, int dtype, int stab) {
  return dtype == FSHARP_BF16 && dm->d == TC_D && dm->M == TC_M && (stab == FSHARP_STAB_ROW || stab == FSHARP_STAB_NONE);
}

size_t fs_tc_featurize_scratch_bytes(const fsharp_dims* dm, int side) {
  const size_t BH = (size_t)dm->B * dm->H, G = fs_groups(dm);
  const size_t L = side == 1 ? dm->Lq : dm->Lk, Lpad = (L + TILE - 1) / TILE * TILE;
  return ws_round(G * 2 * IMG_BYTES) + ws_round(G * 2 * FLAG_WORDS * 4 + 64) + ws_round(BH * Lpad * 4);
}

// prep: the fp32 prep block [G][2][PrepLayout] (its scalars hold the bias); images, flags: written by fs_run_prep_images.
int fs_tc_featurize(fsharp_ctx* ctx, const void* X, const fsharp_dims* dm, int side, int stab, const float* prep,
                    const uint8_t* images, const int* flags, float* phi, float* logscale, WsAlloc* ws) {
  const int B = dm->B, H = dm->H, BH = B * H, L = side == 1 ? dm->Lq : dm->Lk;
  const int tiles = (L + TILE - 1) / TILE, Lpad = tiles * TILE;
  float* crow = ws->take<float>((size_t)BH * Lpad);
  FS_TRY(fs_tc_rowterm_side(ctx, X, dm, side, images, flags, Lpad, crow));
  CUtensorMap tmX;
  FS_TRY(tchost::make_map_tokens(&tmX, X, fs_addr(side == 1 ? dm->q_stride : dm->k_stride, H, L, dm->d), B, H, L, dm->d));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_feat_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FtSmem::TOTAL + 1024));
  int ns = ctx->sm_count / BH;
  ns = ns < 1 ? 1 : (ns > tiles ? tiles : ns);
  const int tps = (tiles + ns - 1) / ns;
  ns = (tiles + tps - 1) / tps;
  FS_TIME_BEGIN(ctx, FS_K_TC_FEAT);
  tc_feat_kernel<<<dim3(ns, BH), TC_THREADS, FtSmem::TOTAL + 1024, ctx->stream>>>(
      tmX, images, crow, prep, side, H, dm->pool, L, Lpad, tps, stab, phi, logscale, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
