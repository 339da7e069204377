// Per-key term of the feature exponent (Theorem 4.1: the x^T C^(2) x part of phi) on the tensor
// cores, for bf16 keys with d = 64:  c_j = log2e * qk_scale^2 * x_j^T C x_j, one fp32 value per key.
//
// T = X C (tcgen05, C split into a bf16 value and its bf16 remainder) lands in TMEM; thread j of
// the epilogue dots row j of T with x_j, which it reads from the same shared-memory tile.
// Computing c_j ahead of the key-side kernel keeps that kernel's TMEM and shared memory for the
// feature tiles; the keys read here stay in L2 for it.
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int RT_STAGES = 4;
constexpr int RT_EPI_THREADS = 128, RT_WARP_TMA = 4, RT_WARP_MMA = 5, RT_THREADS = 192;
constexpr uint32_t RT_TMEM_COLS = 128;       // two T buffers of 64 columns

struct RtSmem {
  static constexpr uint32_t X0 = 0, CHI = RT_STAGES * TILE_BYTES, CLO = CHI + IMG_C_BYTES, MISC = CLO + IMG_C_BYTES,
                            TOTAL = MISC + 256;
};
struct RtMisc {
  uint64_t full[RT_STAGES], empty[RT_STAGES], t_full[2], t_free[2], const_bar;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(RtMisc) <= 256, "misc block");

__global__ void __launch_bounds__(RT_THREADS)
tc_rowterm_kernel(const __grid_constant__ CUtensorMap tmK, const uint8_t* __restrict__ images,
                  const int* __restrict__ img_flags, int side, int H, int pool, int L, int Lpad, int tiles_per_split,
                  float* __restrict__ crow, int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  RtMisc* misc = reinterpret_cast<RtMisc*>(sm + RtSmem::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = blockIdx.x * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  const uint8_t* img = images + ((size_t)g * 2 + (side - 1)) * IMG_BYTES;        // side 1: queries (C1), side 2: keys (C2)
  const bool clo = (img_flags[((size_t)g * 2 + (side - 1)) * FLAG_WORDS] & FLAG_C_LO) != 0;
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < RT_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], RT_EPI_THREADS / 32); }
    for (int i = 0; i < 2; i++) { mbar_init(&misc->t_full[i], 1); mbar_init(&misc->t_free[i], RT_EPI_THREADS / 32); }
    mbar_init(&misc->const_bar, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == RT_WARP_MMA) {
    tmem_alloc(&misc->tmem_base, RT_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == RT_WARP_TMA) {
    if (lane == 0) {
      prefetch_tmap(&tmK);
      mbar_expect_tx(&misc->const_bar, 2 * IMG_C_BYTES);
      bulk_load(sm + RtSmem::CHI, img + IMG_CHI, IMG_C_BYTES, &misc->const_bar);
      bulk_load(sm + RtSmem::CLO, img + IMG_CLO, IMG_C_BYTES, &misc->const_bar);
      int issued = 0;
      for (int it = 0; it < ntiles; it++) {
        const int st = it % RT_STAGES;
        if (!mbar_wait(&misc->empty[st], ((it / RT_STAGES) & 1) ^ 1, abortp, status)) break;
        mbar_expect_tx(&misc->full[st], TILE_BYTES);
        tma_load_4d(sm + RtSmem::X0 + st * TILE_BYTES, &tmK, &misc->full[st], 0, (tile0 + it) * TILE, h, b);
        issued = it + 1;
      }
      // no copy of this block may still be in flight when it exits
      mbar_wait(&misc->const_bar, 0, abortp, status, false);
      for (int it = max(0, issued - RT_STAGES); it < issued; it++)
        mbar_wait(&misc->full[it % RT_STAGES], (it / RT_STAGES) & 1, abortp, status, false);
    }
  } else if (warp == RT_WARP_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues.
    constexpr uint32_t ID_T = idesc_bf16(128, TC_D, 0, 0);
    const uint64_t dX0 = smem_desc(smem_u32(sm + RtSmem::X0), 16, 1024, SWZ_128B);
    const uint64_t dChi = smem_desc(smem_u32(sm + RtSmem::CHI), 16, 1024, SWZ_128B);
    const uint64_t dClo = smem_desc(smem_u32(sm + RtSmem::CLO), 16, 1024, SWZ_128B);
    uint32_t xl0 = (uint32_t)dX0, chl = (uint32_t)dChi, cll = (uint32_t)dClo;
    const uint32_t xh = (uint32_t)(dX0 >> 32), ch = (uint32_t)(dChi >> 32);
    bool ok = __all_sync(0xffffffffu, mbar_wait(&misc->const_bar, 0, abortp, status));
    for (int it = 0; ok && it < ntiles; it++) {
      const int st = it % RT_STAGES, buf = it & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[st], (it / RT_STAGES) & 1, abortp, status))) break;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->t_free[buf], ((it >> 1) & 1) ^ 1, abortp, status))) break;
      tcgen05_fence_after();
      opaque(xl0); opaque(chl); opaque(cll);
      const uint32_t xl = xl0 + st * (TILE_BYTES / 16);
      // (a fixed lane, not an elected one: with two of these blocks on an SM the elected form gave wrong products now and then)
      if (lane == 0) {
#pragma unroll
        for (int k = 0; k < TC_D / 16; k++) mma_bf16_lh(tmem + buf * TC_D, xl + 2 * k, xh, chl + 2 * k, ch, ID_T, k > 0 ? 1u : 0u);
        if (clo) {
#pragma unroll
          for (int k = 0; k < TC_D / 16; k++) mma_bf16_lh(tmem + buf * TC_D, xl + 2 * k, xh, cll + 2 * k, ch, ID_T, 1u);
        }
        mma_commit(&misc->t_full[buf]);
      }
      __syncwarp();
    }
  } else {
    // epilogue: one key row per thread
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    float* out = crow + (size_t)bh * Lpad + (size_t)tile0 * TILE + row;
    for (int it = 0; it < ntiles; it++) {
      const int st = it % RT_STAGES, buf = it & 1;
      if (!mbar_wait(&misc->full[st], (it / RT_STAGES) & 1, abortp, status, false)) break;
      if (!mbar_wait(&misc->t_full[buf], (it >> 1) & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      const uint8_t* xrow = sm + RtSmem::X0 + st * TILE_BYTES + row * 128;
      float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < TC_D / 16; c++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + buf * TC_D + c * 16, t);
        const uint4 u0 = *reinterpret_cast<const uint4*>(xrow + (((2 * c) ^ (row & 7)) << 4));
        const uint4 u1 = *reinterpret_cast<const uint4*>(xrow + (((2 * c + 1) ^ (row & 7)) << 4));
        const uint32_t w8[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 8; j++) {
          part[j & 3] = fmaf(__uint_as_float(t[2 * j]), __uint_as_float(w8[j] << 16), part[j & 3]);
          part[j & 3] = fmaf(__uint_as_float(t[2 * j + 1]), __uint_as_float(w8[j] & 0xffff0000u), part[j & 3]);
        }
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&misc->t_free[buf]);
        mbar_arrive(&misc->empty[st]);
      }
      out[(size_t)it * TILE] = (part[0] + part[1]) + (part[2] + part[3]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == RT_WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, RT_TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}

// crow: [B*H][Lpad] floats with Lpad = ceil(L / 128) * 128; rows at and beyond L come out as zero.  side 1: X is the
// query tensor (q_stride, Lq) and C1 is used; side 2: the key tensor (k_stride, Lk) and C2.
int fs_tc_rowterm_side(fsharp_ctx* ctx, const void* X, const fsharp_dims* dm, int side, const uint8_t* images, const int* flags,
                       int Lpad, float* crow) {
  const int B = dm->B, H = dm->H, L = side == 1 ? dm->Lq : dm->Lk;
  CUtensorMap tmX;
  FS_TRY(tchost::make_map_tokens(&tmX, X, fs_addr(side == 1 ? dm->q_stride : dm->k_stride, H, L, dm->d), B, H, L, dm->d));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_rowterm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RtSmem::TOTAL + 1024));
  // The output is indexed by token, so this kernel has a split of its own: two of its blocks fit an SM, and a block
  // is bound by its single MMA-issuing thread, so it takes about two blocks per SM.
  const int total = (L + TILE - 1) / TILE;
  int ns = (2 * ctx->sm_count) / (B * H);
  ns = ns < 1 ? 1 : (ns > total ? total : ns);
  const int tps = (total + ns - 1) / ns;
  ns = (total + tps - 1) / tps;
  FS_TIME_BEGIN(ctx, FS_K_TC_ROWTERM);
  (void)fs_launch_chained(tc_rowterm_kernel, dim3(ns, B * H), dim3(RT_THREADS), RtSmem::TOTAL + 1024, ctx->stream,
      tmX, images, flags, side, H, dm->pool, L, Lpad, tps, crow, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}

int fs_tc_rowterm(fsharp_ctx* ctx, const void* K, const fsharp_dims* dm, const uint8_t* images, const int* flags, int Lpad,
                  int tiles_per_split, int nsplit, float* crow) {
  (void)tiles_per_split;
  (void)nsplit;
  return fs_tc_rowterm_side(ctx, K, dm, 2, images, flags, Lpad, crow);
}
