// Feature exponents (Section 4: log f = w^T A w + w^T B x + x^T C x + log D) for bf16 tokens with d = 128 on the
// tensor cores:  e_im = bias + a_m + w_m . x_i + c_i  as fp32 [B*H][L][M], the input of the fp32 path's shift /
// exponential kernels (the d = 128 shapes have no fused attention kernel; this replaces their largest fp32 product).
//
// One block = (token split, block of 128 features, (batch, head)).  It turns its 128 rows of W = Omega B
// (fp32, scaled by qk_scale) into two bf16 operand images, the rounded value and the remainder, so that the
// product carries 16 significant bits of W (the tokens are exact in bf16); a token tile [128 x 128] arrives by TMA
// as two 64-column panels (128-byte swizzle), and D = X W^T is 16 MMAs of N = 128 (two panels x four K steps,
// value image then remainder image) into one of two accumulators in tensor memory.  The epilogue adds the
// per-feature and per-token terms and writes the rows.
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int LG_D = 128, LG_NF = 128, LG_STAGES = 3;
constexpr int LG_EPI_THREADS = 128, LG_WARP_TMA = 4, LG_WARP_MMA = 5, LG_THREADS = 192;
constexpr uint32_t LG_TMEM_COLS = 256;                 // two accumulators of 128 columns
constexpr uint32_t LG_XBYTES = 2 * TILE_BYTES;         // token tile: two panels [128 rows x 64 columns]
constexpr uint32_t LG_WBYTES = 2 * TILE_BYTES;         // feature block: two panels [128 features x 64 columns]

struct LgSmem {
  static constexpr uint32_t X0 = 0, WHI = LG_STAGES * LG_XBYTES, WLO = WHI + LG_WBYTES, AV = WLO + LG_WBYTES,
                            MISC = AV + LG_NF * 4, TOTAL = MISC + 256;
};
struct LgMisc {
  uint64_t full[LG_STAGES], empty[LG_STAGES], t_full[2], t_free[2];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(LgMisc) <= 256, "misc block");
static_assert(LgSmem::TOTAL + 1024 <= 232448, "shared memory budget");

__global__ void __launch_bounds__(LG_THREADS, 1)
tc_logits128_kernel(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ prep, const float* __restrict__ rowc,
                    float* __restrict__ phi, int H, int pool, int L, int M, int side, float qk_scale, int tiles_per_split,
                    int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  LgMisc* misc = reinterpret_cast<LgMisc*>(sm + LgSmem::MISC);
  float* a_s = reinterpret_cast<float*>(sm + LgSmem::AV);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int fblk = blockIdx.y, bh = blockIdx.z, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = blockIdx.x * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  volatile int* abortp = &misc->abort_flag;
  PrepLayout pr{LG_D, M};
  const float* pp = prep + ((size_t)g * 2 + (side - 1)) * pr.total();
  const float* W = pp + pr.W() + (size_t)fblk * LG_NF * LG_D;
  const float* av = pp + pr.a() + (size_t)fblk * LG_NF;
  const float bias = pp[pr.scal() + PS_BIAS];

  if (threadIdx.x == 0) {
    for (int i = 0; i < LG_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&misc->t_full[i], 1); mbar_init(&misc->t_free[i], LG_EPI_THREADS / 32); }
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  // operand images of this feature block: feature f, columns 8 c .. 8 c + 7 -> panel c / 8, 16-byte piece (c % 8) ^ (f % 8)
  // of row f (the 128-byte swizzle of a K-major operand)
  for (int e = threadIdx.x; e < LG_NF * (LG_D / 8); e += LG_THREADS) {
    const int f = e / (LG_D / 8), c = e % (LG_D / 8);
    const float4 w0 = *reinterpret_cast<const float4*>(W + (size_t)f * LG_D + 8 * c);
    const float4 w1 = *reinterpret_cast<const float4*>(W + (size_t)f * LG_D + 8 * c + 4);
    const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const float x0 = qk_scale * w[2 * j], x1 = qk_scale * w[2 * j + 1];
      const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
      hi[j] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lo[j] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    const uint32_t off = (uint32_t)(c >> 3) * TILE_BYTES + (uint32_t)f * 128u + (uint32_t)(((c & 7) ^ (f & 7)) << 4);
    *reinterpret_cast<uint4*>(sm + LgSmem::WHI + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(sm + LgSmem::WLO + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
  if (threadIdx.x < LG_NF) a_s[threadIdx.x] = av[threadIdx.x] + bias;
  fence_proxy_async_smem();
  if (warp == LG_WARP_MMA) {
    tmem_alloc(&misc->tmem_base, LG_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == LG_WARP_TMA) {
    if (lane == 0) {
      prefetch_tmap(&tmX);
      int issued = 0;
      for (int it = 0; it < ntiles; it++) {
        const int st = it % LG_STAGES;
        if (!mbar_wait(&misc->empty[st], ((it / LG_STAGES) & 1) ^ 1, abortp, status)) break;
        mbar_expect_tx(&misc->full[st], LG_XBYTES);
        tma_load_4d(sm + LgSmem::X0 + st * LG_XBYTES, &tmX, &misc->full[st], 0, (tile0 + it) * TILE, h, b);
        tma_load_4d(sm + LgSmem::X0 + st * LG_XBYTES + TILE_BYTES, &tmX, &misc->full[st], 64, (tile0 + it) * TILE, h, b);
        issued = it + 1;
      }
      // no copy of this block may still be in flight when it exits
      for (int it = max(0, issued - LG_STAGES); it < issued; it++)
        mbar_wait(&misc->full[it % LG_STAGES], (it / LG_STAGES) & 1, abortp, status, false);
    }
  } else if (warp == LG_WARP_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues.
    constexpr uint32_t ID = idesc_bf16(128, LG_NF, 0, 0);
    const uint64_t dX0 = smem_desc(smem_u32(sm + LgSmem::X0), 16, 1024, SWZ_128B);
    const uint64_t dWh = smem_desc(smem_u32(sm + LgSmem::WHI), 16, 1024, SWZ_128B);
    const uint64_t dWl = smem_desc(smem_u32(sm + LgSmem::WLO), 16, 1024, SWZ_128B);
    uint32_t xl0 = (uint32_t)dX0, whl = (uint32_t)dWh, wll = (uint32_t)dWl;
    const uint32_t xh = (uint32_t)(dX0 >> 32), wh = (uint32_t)(dWh >> 32);
    for (int it = 0; it < ntiles; it++) {
      const int st = it % LG_STAGES, buf = it & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[st], (it / LG_STAGES) & 1, abortp, status))) break;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->t_free[buf], ((it >> 1) & 1) ^ 1, abortp, status))) break;
      tcgen05_fence_after();
      opaque(xl0); opaque(whl); opaque(wll);
      const uint32_t xl = xl0 + st * (LG_XBYTES / 16);
      if (lane == 0) {
#pragma unroll
        for (int p = 0; p < 2; p++)
#pragma unroll
          for (int k = 0; k < 4; k++)
            mma_bf16_lh(tmem + buf * LG_NF, xl + p * (TILE_BYTES / 16) + 2 * k, xh, whl + p * (TILE_BYTES / 16) + 2 * k, wh, ID,
                        (p | k) ? 1u : 0u);
#pragma unroll
        for (int p = 0; p < 2; p++)
#pragma unroll
          for (int k = 0; k < 4; k++)
            mma_bf16_lh(tmem + buf * LG_NF, xl + p * (TILE_BYTES / 16) + 2 * k, xh, wll + p * (TILE_BYTES / 16) + 2 * k, wh, ID, 1u);
        mma_commit(&misc->t_full[buf]);
        mma_commit(&misc->empty[st]);       // the token tile has no other reader
      }
      __syncwarp();
    }
  } else {
    // epilogue: one token row per thread
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    for (int it = 0; it < ntiles; it++) {
      const int buf = it & 1;
      const int64_t tok = (int64_t)(tile0 + it) * TILE + row;
      const float ci = tok < L ? rowc[(int64_t)bh * L + tok] : 0.f;
      if (!mbar_wait(&misc->t_full[buf], (it >> 1) & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      float* out = phi + ((int64_t)bh * L + tok) * M + (int64_t)fblk * LG_NF;
#pragma unroll
      for (int c = 0; c < LG_NF / 16; c++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + buf * LG_NF + c * 16, t);
        tmem_wait_ld();
        if (tok < L) {
#pragma unroll
          for (int j = 0; j < 4; j++)
            *reinterpret_cast<float4*>(out + c * 16 + 4 * j) =
                make_float4(__uint_as_float(t[4 * j]) + a_s[c * 16 + 4 * j] + ci, __uint_as_float(t[4 * j + 1]) + a_s[c * 16 + 4 * j + 1] + ci,
                            __uint_as_float(t[4 * j + 2]) + a_s[c * 16 + 4 * j + 2] + ci, __uint_as_float(t[4 * j + 3]) + a_s[c * 16 + 4 * j + 3] + ci);
        }
      }
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->t_free[buf], lane);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == LG_WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, LG_TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}

// bf16 tokens with d = 128, M a multiple of 128, 16-byte aligned rows
int fs_tc_logits128_supported(const void* X, int dtype, TensorAddr ax, int L, int d, int M) {
  if (dtype != FSHARP_BF16 || d != LG_D || M % LG_NF != 0 || L <= 0) return 0;
  if (reinterpret_cast<uintptr_t>(X) % 16 != 0) return 0;
  if ((ax.sl * 2) % 16 != 0 || (ax.sh * 2) % 16 != 0 || (ax.sb * 2) % 16 != 0) return 0;
  return 1;
}

// phi [B*H][L][M] fp32 <- bias + a_m + w_m . (qk_scale x_i) + rowc_i;  rowc [B*H][L] (the x^T C x term)
int fs_tc_logits128(fsharp_ctx* ctx, const void* X, TensorAddr ax, int B, int H, int L, int M, int pool, const float* prep,
                    int side, float qk_scale, const float* rowc, float* phi) {
  CUtensorMap tmX;
  FS_TRY(tchost::make_map_tokens(&tmX, X, ax, B, H, L, LG_D));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_logits128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LgSmem::TOTAL + 1024));
  // every block builds its operand images first (64 KB of W), so few, long blocks: about one per SM
  const int total = (L + TILE - 1) / TILE, nq = M / LG_NF, BH = B * H;
  int ns = ctx->sm_count / (BH * nq);
  ns = ns < 1 ? 1 : (ns > total ? total : ns);
  const int tps = (total + ns - 1) / ns;
  ns = (total + tps - 1) / tps;
  FS_TIME_BEGIN(ctx, FS_K_TC_LOGITS128);
  tc_logits128_kernel<<<dim3(ns, nq, BH), LG_THREADS, LgSmem::TOTAL + 1024, ctx->stream>>>(
      tmX, prep, rowc, phi, H, pool, L, M, side, qk_scale, tps, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
