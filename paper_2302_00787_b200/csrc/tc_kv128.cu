// Per-chunk key-side sums of the causal form, S_c^T [V_c | 1] (Section 2.1's O(L M n) order, chunk by chunk), on the
// tensor cores for the shapes that have no fused kernel: bf16 copy of phi(K) [B*H][L][M], V [B,H,L,128] bf16.
// Output st [B*H * L/C][129][M] fp32, column index first (feature index contiguous), so that a warp's stores coalesce
// and the query-side product finds the feature index contiguous.
//
// One block = (range of chunks, block of 128 features, (batch, head)).  Tokens are the contraction: a stage holds
// 128 tokens of the feature block (two 64-feature panels) and of V (two 64-column panels), all "MN-major" operands
// (the contracted index is the row of the tile).  Per 16 tokens: D[:, 0..127] += phi^T V (N = 128) and
// D[:, 128..143] += phi^T E with E the constant tile whose first column is 1 (N = 16).  Two accumulators in tensor
// memory: the epilogue writes chunk c while chunk c + 1 is multiplied.
#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int KV_ST = 2;
constexpr int KVE_THREADS = 128, KVW_TMA = 4, KVW_MMA = 5, KVT = 192;
constexpr uint32_t KV_ACC_COLS = 160;                  // 128 + 16, kept apart by a multiple of 32
constexpr uint32_t KV_TMEM_COLS = 512;                 // two accumulators (power of two)
constexpr uint32_t KV_STAGE = 4 * TILE_BYTES;          // feature panels 0, 1, then V panels 0, 1

struct KvSm {
  static constexpr uint32_t A0 = 0, ONES = KV_ST * KV_STAGE, MISC = ONES + TILE_BYTES, TOTAL = MISC + 256;
};
struct KvMs {
  uint64_t full[KV_ST], empty[KV_ST], acc_full[2], acc_free[2];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(KvMs) <= 256, "misc block");
static_assert(KvSm::TOTAL + 1024 <= 232448, "shared memory budget");

__global__ void __launch_bounds__(KVT, 1)
tc_kv128_kernel(const __grid_constant__ CUtensorMap tmP, const __grid_constant__ CUtensorMap tmV, float* __restrict__ st,
                int H, int M, int C, int nch, int chunks_per_split, int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  KvMs* misc = reinterpret_cast<KvMs*>(sm + KvSm::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int fblk = blockIdx.y, bh = blockIdx.z, b = bh / H, h = bh % H;
  const int c0 = blockIdx.x * chunks_per_split;
  const int ncs = min(chunks_per_split, nch - c0);
  if (ncs <= 0) return;                        // uniform over the block, before anything is allocated
  const int tpc = C / TILE;                    // token tiles per chunk
  const int ntiles = ncs * tpc;
  volatile int* abortp = &misc->abort_flag;
  constexpr int N = 129;

  if (threadIdx.x == 0) {
    for (int i = 0; i < KV_ST; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&misc->acc_full[i], 1); mbar_init(&misc->acc_free[i], KVE_THREADS / 32); }
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  for (int i = threadIdx.x; i < (int)(TILE_BYTES / 16); i += KVT) reinterpret_cast<uint4*>(sm + KvSm::ONES)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (threadIdx.x < TILE)
    *reinterpret_cast<__nv_bfloat16*>(sm + KvSm::ONES + sw128_offset(threadIdx.x, 0)) = __float2bfloat16(1.f);
  fence_proxy_async_smem();
  if (warp == KVW_MMA) {
    tmem_alloc(&misc->tmem_base, KV_TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp == KVW_TMA) {
    if (lane == 0) {
      prefetch_tmap(&tmP);
      prefetch_tmap(&tmV);
      int issued = 0;
      for (int it = 0; it < ntiles; it++) {
        const int s = it % KV_ST;
        const int tok = (c0 * tpc + it) * TILE;
        if (!mbar_wait(&misc->empty[s], ((it / KV_ST) & 1) ^ 1, abortp, status)) break;
        uint8_t* base = sm + KvSm::A0 + s * KV_STAGE;
        mbar_expect_tx(&misc->full[s], KV_STAGE);
        tma_load_4d(base, &tmP, &misc->full[s], fblk * 128, tok, bh, 0);
        tma_load_4d(base + TILE_BYTES, &tmP, &misc->full[s], fblk * 128 + 64, tok, bh, 0);
        tma_load_4d(base + 2 * TILE_BYTES, &tmV, &misc->full[s], 0, tok, h, b);
        tma_load_4d(base + 3 * TILE_BYTES, &tmV, &misc->full[s], 64, tok, h, b);
        issued = it + 1;
      }
      // no copy of this block may still be in flight when it exits
      for (int it = max(0, issued - KV_ST); it < issued; it++)
        mbar_wait(&misc->full[it % KV_ST], (it / KV_ST) & 1, abortp, status, false);
    }
  } else if (warp == KVW_MMA) {
    // The whole warp walks the schedule (waits and descriptor arithmetic stay warp-uniform); lane 0 issues.
    constexpr uint32_t ID_V = idesc_bf16(128, 128, 1, 1), ID_E = idesc_bf16(128, 16, 1, 1);   // both operands MN-major
    const uint32_t sA0 = smem_u32(sm + KvSm::A0), sOnes = smem_u32(sm + KvSm::ONES);
    for (int it = 0; it < ntiles; it++) {
      const int s = it % KV_ST, ch = it / tpc, sub = it % tpc, buf = ch & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[s], (it / KV_ST) & 1, abortp, status))) break;
      if (sub == 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->acc_free[buf], ((ch >> 1) & 1) ^ 1, abortp, status))) break;
      tcgen05_fence_after();
      const uint32_t sP = sA0 + s * KV_STAGE, sV = sP + 2 * TILE_BYTES;
      // operands of 128 (features / columns) = two 64-wide panels: the leading offset is the panels' distance
      const uint64_t dA = smem_desc(sP, TILE_BYTES, 1024, SWZ_128B);
      const uint64_t dB = smem_desc(sV, TILE_BYTES, 1024, SWZ_128B);
      const uint64_t dE = smem_desc(sOnes, TILE_BYTES, 1024, SWZ_128B);
      uint32_t al = (uint32_t)dA, bl = (uint32_t)dB, el = (uint32_t)dE;
      const uint32_t ah = (uint32_t)(dA >> 32), bhh = (uint32_t)(dB >> 32), eh = (uint32_t)(dE >> 32);
      opaque(al); opaque(bl); opaque(el);
      if (lane == 0) {
        const uint32_t acc = tmem + buf * KV_ACC_COLS;
#pragma unroll
        for (int k = 0; k < TILE / 16; k++) {
          mma_bf16_lh(acc, al + k * 128, ah, bl + k * 128, bhh, ID_V, (k > 0 || sub > 0) ? 1u : 0u);
          mma_bf16_lh(acc + 128, al + k * 128, ah, el + k * 128, eh, ID_E, (k > 0 || sub > 0) ? 1u : 0u);
        }
        if (sub == tpc - 1) mma_commit(&misc->acc_full[buf]);
        mma_commit(&misc->empty[s]);
      }
      __syncwarp();
    }
  } else {
    // epilogue: thread = feature row of D; columns 0..127 the V part, column 128 the ones column
    const int row = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    for (int ch = 0; ch < ncs; ch++) {
      const int buf = ch & 1;
      if (!mbar_wait(&misc->acc_full[buf], (ch >> 1) & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      float* out = st + ((size_t)bh * nch + c0 + ch) * (size_t)N * M + (size_t)fblk * 128 + row;
#pragma unroll
      for (int cc = 0; cc < 8; cc++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + buf * KV_ACC_COLS + cc * 16, t);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j++) out[(size_t)(cc * 16 + j) * M] = __uint_as_float(t[j]);
      }
      {
        uint32_t t[8];
        tmem_ld8(lane_addr + buf * KV_ACC_COLS + 128, t);
        tmem_wait_ld();
        out[(size_t)128 * M] = __uint_as_float(t[0]);
      }
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->acc_free[buf], lane);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == KVW_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, KV_TMEM_COLS);
  }
}

}  // namespace

namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}

// bf16 tensors, dv = 128, M a multiple of 128, chunks of 128 or 256 tokens, 16-byte aligned V rows
int fs_tc_kv128_supported(const void* V, TensorAddr av, int dv, int M, int C) {
  if (dv != 128 || M % 128 != 0 || (C != 128 && C != 256)) return 0;
  if (reinterpret_cast<uintptr_t>(V) % 16 != 0) return 0;
  return (av.sl * 2) % 16 == 0 && (av.sh * 2) % 16 == 0 && (av.sb * 2) % 16 == 0;
}

// phiK16 [BH][L][M] bf16, V [B,H,L,128] bf16 (strides av), st [BH * L / C][129][M] fp32 (feature index contiguous)
int fs_tc_kv128(fsharp_ctx* ctx, const void* phiK16, const void* V, TensorAddr av, int B, int H, int L, int M, int C, float* st) {
  const int BH = B * H, nch = L / C, nq = M / 128;
  CUtensorMap tmP, tmV;
  TensorAddr ap{(int64_t)BH * L * M, (int64_t)L * M, (int64_t)M};
  FS_TRY(tchost::make_map_tokens(&tmP, phiK16, ap, 1, BH, L, M));
  FS_TRY(tchost::make_map_tokens(&tmV, V, av, B, H, L, 128));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_kv128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)KvSm::TOTAL + 1024));
  // about two blocks per SM's worth of work in the grid, each walking a range of chunks
  int ns = (2 * ctx->sm_count + BH * nq - 1) / (BH * nq);
  ns = ns < 1 ? 1 : (ns > nch ? nch : ns);
  const int cps = (nch + ns - 1) / ns;
  ns = (nch + cps - 1) / cps;
  FS_TIME_BEGIN(ctx, FS_K_TC_KV128);
  tc_kv128_kernel<<<dim3(ns, nq, BH), KVT, KvSm::TOTAL + 1024, ctx->stream>>>(tmP, tmV, st, H, M, C, nch, cps, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
