// Set statistics of Theorems 4.2 and 4.3 on the tensor cores, for bf16 tokens with d = 64:
// M1 = L^-1 sum x x^T, M2 = L^-1 sum y y^T, mu4 = mean x, mu5 = mean y.
//
// A 128-token tile X [128 x 64] sits in shared memory once (TMA, 128-byte swizzle) and is read
// by the MMA as both operands: D = [X | E]^T X with E the constant tile whose first column is 1.
// Rows 0..63 of D are the tile's Gram matrix, row 64 its column sums.  Products of bf16 values
// are exact in fp32; the fp32 sums of ST_FOLD tiles at a time are folded into fp64 registers (the fold, 64
// conversions and additions per thread, is what a tile's arrival rate from HBM has to cover), and the
// blocks of one group are combined with fp64 atomics.  The kernel is bound by the HBM read of Q and K.
// d = 128 (WIDE): the Gram matrix is four 64 x 64 blocks G_ab = X_a^T X_b over the column halves a, b of the tokens; a
// block of the grid computes one of them from the two 64-column panels of a token tile, D = [X_a | E]^T X_b (row 64:
// the column sums of X_b, kept when a = b).
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int ST_STAGES = 4;                 // ring of token tiles in flight (two blocks share an SM: eight tiles per SM)
constexpr int ST_FOLD = 2;                   // tiles summed in one fp32 accumulator before it is folded into fp64
constexpr int ST_EPI_WARPS = 3;              // rows 0..95 of D; only 0..64 carry data
constexpr int ST_WARP_TMA = 3, ST_WARP_MMA = 4, ST_THREADS = 160;
constexpr uint32_t ST_TMEM_COLS = 128;       // two accumulators of 64 columns

template <bool WIDE>
struct StSmemT {
  static constexpr uint32_t STAGE = (WIDE ? 2u : 1u) * TILE_BYTES;     // WIDE: panel a, then panel b
  static constexpr int NST = WIDE ? 2 : ST_STAGES;                    // (two blocks of either kind fit an SM)
  static constexpr uint32_t X0 = 0, ONES = NST * STAGE, MISC = ONES + TILE_BYTES, TOTAL = MISC + 256;
};
using StSmem = StSmemT<false>;
struct StMisc {
  uint64_t full[ST_STAGES], empty[ST_STAGES], acc_full[2], acc_free[2];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(StMisc) <= 256, "misc block");

template <bool WIDE>
__global__ void __launch_bounds__(ST_THREADS, 2)
tc_stats_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, int H, int Lq, int Lk,
                int pool, int Bpool, double qk_scale, int tiles_per_split, double* __restrict__ stats,
                int* __restrict__ status) {
  using StSmem = StSmemT<WIDE>;
  constexpr int DD = WIDE ? 2 * TC_D : TC_D;          // head dimension
  constexpr int NST = StSmem::NST;
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  StMisc* misc = reinterpret_cast<StMisc*>(sm + StSmem::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // WIDE: blockIdx.z = 4 side + 2 a + b, the column halves of the A and the B operand
  const int side = WIDE ? blockIdx.z >> 2 : blockIdx.z, ha = WIDE ? (blockIdx.z >> 1) & 1 : 0, hb = WIDE ? blockIdx.z & 1 : 0;
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int L = side ? Lk : Lq;
  const CUtensorMap* tm = side ? &tmK : &tmQ;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = blockIdx.x * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NST; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&misc->acc_full[i], 1); mbar_init(&misc->acc_free[i], ST_EPI_WARPS); }
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  for (int i = threadIdx.x; i < TILE_BYTES / 16; i += ST_THREADS) reinterpret_cast<uint4*>(sm + StSmem::ONES)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (threadIdx.x < TILE)
    *reinterpret_cast<__nv_bfloat16*>(sm + StSmem::ONES + sw128_offset(threadIdx.x, 0)) = __float2bfloat16(1.f);
  fence_proxy_async_smem();
  if (warp == ST_WARP_MMA) {
    tmem_alloc(&misc->tmem_base, ST_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == ST_WARP_TMA) {
    if (lane == 0) {
      prefetch_tmap(tm);
      int issued = 0;
      for (int it = 0; it < ntiles; it++) {
        const int st = it % NST;
        if (!mbar_wait(&misc->empty[st], ((it / NST) & 1) ^ 1, abortp, status)) break;
        mbar_expect_tx(&misc->full[st], StSmem::STAGE);
        tma_load_4d(sm + StSmem::X0 + st * StSmem::STAGE, tm, &misc->full[st], 64 * ha, (tile0 + it) * TILE, h, b);
        if (WIDE) tma_load_4d(sm + StSmem::X0 + st * StSmem::STAGE + TILE_BYTES, tm, &misc->full[st], 64 * hb, (tile0 + it) * TILE, h, b);
        issued = it + 1;
      }
      // no copy of this block may still be in flight when it exits
      for (int it = max(0, issued - NST); it < issued; it++)
        mbar_wait(&misc->full[it % NST], (it / NST) & 1, abortp, status, false);
    }
  } else if (warp == ST_WARP_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues.
    // An MMA issued by a single lane of a diverged warp costs its thread two to three times as long.
    constexpr uint32_t ID = idesc_bf16(128, TC_D, 1, 1);      // both operands MN-major (feature index contiguous)
    const uint32_t sX0 = smem_u32(sm + StSmem::X0), sOnes = smem_u32(sm + StSmem::ONES);
    for (int it = 0; it < ntiles; it++) {
      const int st = it % NST, grp = it / ST_FOLD, buf = grp & 1, sub = it % ST_FOLD;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[st], (it / NST) & 1, abortp, status))) break;
      if (sub == 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->acc_free[buf], ((grp >> 1) & 1) ^ 1, abortp, status))) break;
      tcgen05_fence_after();
      const uint32_t sX = sX0 + st * StSmem::STAGE, sXb = WIDE ? sX + TILE_BYTES : sX;
      // A = [X | E]: block 0 the tile, block 1 the constant tile (leading offset = their distance); a step's
      // descriptors are the tile's plus a constant in the low word (start address / 16)
      const uint64_t dA = smem_desc(sX, sOnes - sX, 1024, SWZ_128B);
      const uint64_t dB = smem_desc(sXb, TILE_BYTES, 1024, SWZ_128B);
      uint32_t al = (uint32_t)dA, bl = (uint32_t)dB;
      const uint32_t ah = (uint32_t)(dA >> 32), bh = (uint32_t)(dB >> 32);
      opaque(al); opaque(bl);
      // (a fixed lane, not an elected one: with two of these blocks on an SM the elected form gave wrong products now and then)
      if (lane == 0) {
#pragma unroll
        for (int k = 0; k < TILE / 16; k++)
          mma_bf16_lh(tmem + buf * TC_D, al + k * 128, ah, bl + k * 128, bh, ID, (k > 0 || sub > 0) ? 1u : 0u);
        if (sub == ST_FOLD - 1 || it == ntiles - 1) mma_commit(&misc->acc_full[buf]);
        mma_commit(&misc->empty[st]);
      }
      __syncwarp();
    }
  } else {
    // epilogue: thread = row of D (rows 0..63 Gram, row 64 column sums), 64 columns
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    double acc[TC_D];
#pragma unroll
    for (int j = 0; j < TC_D; j++) acc[j] = 0.0;
    bool alive = true;
    const int ngroups = (ntiles + ST_FOLD - 1) / ST_FOLD;
    for (int it = 0; it < ngroups && alive; it++) {
      const int buf = it & 1;
      if (!mbar_wait(&misc->acc_full[buf], (it >> 1) & 1, abortp, status, false)) { alive = false; break; }
      __syncwarp();
      tcgen05_fence_after();
#pragma unroll
      for (int c = 0; c < TC_D / 16; c++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + buf * TC_D + c * 16, t);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j++) acc[c * 16 + j] += (double)__uint_as_float(t[j]);
      }
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->acc_free[buf], lane);
    }
    if (alive && row <= TC_D) {
      const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
      const double inv = 1.0 / ((double)L * (double)Bpool);
      StatsLayout sl{DD};
      double* out = stats + (size_t)g * sl.total();
      bool bad = false;
      if (row < TC_D) {
        // the Gram matrix is symmetric: row `row` is stored as column `row`, so a warp's atomics coalesce
        // (entry (64 a + row, 64 b + j) of the matrix goes to row 64 b + j, column 64 a + row)
        double* Mo = out + sl.M(side + 1) + (size_t)(TC_D * hb) * DD + TC_D * ha;
        const double f = inv * qk_scale * qk_scale;
#pragma unroll
        for (int j = 0; j < TC_D; j++) {
          if (!isfinite(acc[j])) bad = true;
          atomicAdd(&Mo[(size_t)j * DD + row], acc[j] * f);
        }
      } else if (ha == hb) {
        double* mu = out + sl.mu(side + 4) + TC_D * hb;
        const double f = inv * qk_scale;
#pragma unroll
        for (int j = 0; j < TC_D; j++) {
          if (!isfinite(acc[j])) bad = true;
          atomicAdd(&mu[j], acc[j] * f);
        }
      }
      if (bad) atomicExch(status, FSHARP_E_NONFINITE);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == ST_WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, ST_TMEM_COLS);
  }
}

bool aligned16(const void* p, TensorAddr a) {
  return (reinterpret_cast<uintptr_t>(p) & 15) == 0 && a.sl % 8 == 0 && a.sh % 8 == 0 && a.sb % 8 == 0;
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}

int fs_tc_stats_supported(const void* Q, const void* K, const fsharp_dims* dm, int dtype) {
  if (dtype != FSHARP_BF16 || (dm->d != TC_D && dm->d != 2 * TC_D) || dm->Lq <= 0 || dm->Lk <= 0) return 0;
  return aligned16(Q, fs_addr(dm->q_stride, dm->H, dm->Lq, dm->d)) && aligned16(K, fs_addr(dm->k_stride, dm->H, dm->Lk, dm->d));
}

// The statistics block must already be zero (the blocks add into it).
int fs_tc_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dm, float qk_scale, double* stats) {
  const int B = dm->B, H = dm->H, BH = B * H;
  const int Lmax = dm->Lq > dm->Lk ? dm->Lq : dm->Lk;
  const int tiles = (Lmax + TILE - 1) / TILE;
  const bool wide = dm->d == 2 * TC_D;
  // two blocks per SM (each block has one MMA-issuing thread, and issuing is what bounds a block): the split of
  // the token range with the fewest (waves x tiles per block)
  int best = 1, best_cost = 0x7fffffff, tps = tiles;
  for (int ns = 1; ns <= tiles; ns++) {
    const int t = (tiles + ns - 1) / ns;
    if ((tiles + t - 1) / t != ns) continue;
    const long long blocks = (wide ? 8LL : 2LL) * BH * ns;
    const int waves = (int)((blocks + 2 * ctx->sm_count - 1) / (2 * ctx->sm_count));
    const int cost = waves * (t + 6);        // fill, drain and the final atomics cost about six tiles
    if (cost < best_cost) { best_cost = cost; best = ns; tps = t; }
  }
  CUtensorMap tmQ, tmK;
  FS_TRY(tchost::make_map_tokens(&tmQ, Q, fs_addr(dm->q_stride, H, dm->Lq, dm->d), B, H, dm->Lq, dm->d));
  FS_TRY(tchost::make_map_tokens(&tmK, K, fs_addr(dm->k_stride, H, dm->Lk, dm->d), B, H, dm->Lk, dm->d));
  const int Bpool = dm->pool == FSHARP_POOL_PER_BH ? 1 : B;
  if (wide) {
    FS_CUDA_OK(cudaFuncSetAttribute(tc_stats_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)StSmemT<true>::TOTAL + 1024));
    FS_TIME_BEGIN(ctx, FS_K_TC_STATS);
    (void)fs_launch_chained(tc_stats_kernel<true>, dim3(best, BH, 8), dim3(ST_THREADS), StSmemT<true>::TOTAL + 1024, ctx->stream,
        tmQ, tmK, H, dm->Lq, dm->Lk, dm->pool, Bpool, (double)qk_scale, tps, stats, ctx->d_status);
    FS_TIME_END(ctx);
  } else {
    FS_CUDA_OK(cudaFuncSetAttribute(tc_stats_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)StSmem::TOTAL + 1024));
    FS_TIME_BEGIN(ctx, FS_K_TC_STATS);
    (void)fs_launch_chained(tc_stats_kernel<false>, dim3(best, BH, 2), dim3(ST_THREADS), StSmem::TOTAL + 1024, ctx->stream,
        tmQ, tmK, H, dm->Lq, dm->Lk, dm->pool, Bpool, (double)qk_scale, tps, stats, ctx->d_status);
    FS_TIME_END(ctx);
  }
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
