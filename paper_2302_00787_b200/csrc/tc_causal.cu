// Tensor-core path, causal attention (Section 2.2's formula with a lower-triangular mask) for
// bf16, d = dv = 64, M = 256, chunk = 128 tokens:
//
//   Y_c = [ phiQ_c P_c  +  tril(phiQ_c phiK_c^T) [V_c | 1] ]  (numerator | denominator),
//   P_c = sum over earlier chunks c' of phiK_c'^T [V_c' | 1].
//
//   tc_kv_kernel (tc_bidir.cu), every tile a chunk: chunk states and the chunk's bf16 key features
//   tc_featq_kernel:          bf16 query features, each row shifted by its own maximum
//   tc_causal_prefix_kernel:  exclusive scan of the chunk states -> bf16 prefixes P_c, every
//                             chunk brought to a scale of its own that also weighs the in-chunk term
//   tc_causal_out_kernel:     per chunk  D = phiQ P_c^T, S = phiQ phiK^T (TMEM),
//                             S masked, scaled, rounded to bf16 into shared memory,
//                             D += S V, denominator += row sums of S, Y = num / den
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

// ------------------------------------------------------------------------------------------
// query features
// ------------------------------------------------------------------------------------------
constexpr int FQ_STAGES = 3;
// The feature tile leaves as four 64-feature blocks (16 KB each, one bulk store each) from a ring of six block
// slots: block j of tile t sits in slot (4 t + j) % 6, so a tile only reuses slots whose stores were issued at least
// one and a half tiles earlier and the stores of a tile's last two blocks may still be reading when the next is written.
constexpr int FQ_PHI_SLOTS = 6;
struct FqSmem {
  static constexpr uint32_t X0 = 0, W = FQ_STAGES * TILE_BYTES, WLO = W + IMG_W_BYTES, PHI = WLO + IMG_W_BYTES,
                            ROWMAX = PHI + FQ_PHI_SLOTS * TILE_BYTES,
                            AH = ROWMAX + 2 * 2 * TILE * 4, MISC = AH + TC_M * 4, TOTAL = MISC + 256;
};
struct FqMisc {
  uint64_t full[FQ_STAGES], empty[FQ_STAGES], logits_full[2], logits_free[2], const_bar;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_featq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmPhi,
                const uint8_t* __restrict__ images, int H, int pool, int L, int tiles_per_split, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  FqMisc* misc = reinterpret_cast<FqMisc*>(sm + FqSmem::MISC);
  float* rowmax = reinterpret_cast<float*>(sm + FqSmem::ROWMAX);   // [tile & 1][half][row]
  float* ah = reinterpret_cast<float*>(sm + FqSmem::AH);           // the query side's share a2 / 2 of the per-feature term
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = blockIdx.x * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  const uint8_t* img = images + ((size_t)g * 2 + 0) * IMG_BYTES;        // side 1 (queries)
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < FQ_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->empty[i], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&misc->logits_full[i], 1); mbar_init(&misc->logits_free[i], EPI_THREADS / 32); }
    mbar_init(&misc->const_bar, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  if (threadIdx.x < TC_M) ah[threadIdx.x] = 0.5f * reinterpret_cast<const float*>(img + IMG_A2)[threadIdx.x];
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
        prefetch_tmap(&tmQ);
        mbar_expect_tx(&misc->const_bar, 2 * IMG_W_BYTES);
        bulk_load(sm + FqSmem::W, img + IMG_W, IMG_W_BYTES, &misc->const_bar);
        bulk_load(sm + FqSmem::WLO, img + IMG_WLO, IMG_W_BYTES, &misc->const_bar);
        int issued = 0;
        for (int it = 0; it < ntiles; it++) {
          const int st = it % FQ_STAGES;
          if (!mbar_wait(&misc->empty[st], ((it / FQ_STAGES) & 1) ^ 1, abortp, status)) break;
          mbar_expect_tx(&misc->full[st], TILE_BYTES);
          tma_load_4d(sm + FqSmem::X0 + st * TILE_BYTES, &tmQ, &misc->full[st], 0, (tile0 + it) * TILE, h, b);
          issued = it + 1;
        }
        // no copy of this block may still be in flight when it exits
        mbar_wait(&misc->const_bar, 0, abortp, status, false);
        for (int it = max(0, issued - FQ_STAGES); it < issued; it++)
          mbar_wait(&misc->full[it % FQ_STAGES], (it / FQ_STAGES) & 1, abortp, status, false);
      }
    } else if (warp == WARP_MMA) {
      if (lane == 0) {
        constexpr uint32_t ID_LOGITS = idesc_bf16(128, TC_M, 0, 0);
        const uint64_t dX0 = smem_desc(smem_u32(sm + FqSmem::X0), 16, 1024, SWZ_128B);
        const uint64_t dW = smem_desc(smem_u32(sm + FqSmem::W), 16, 1024, SWZ_128B);
        const uint64_t dWlo = smem_desc(smem_u32(sm + FqSmem::WLO), 16, 1024, SWZ_128B);
        bool ok = mbar_wait(&misc->const_bar, 0, abortp, status);
        for (int it = 0; ok && it < ntiles; it++) {
          const int st = it % FQ_STAGES, buf = it & 1;
          if (!mbar_wait(&misc->full[st], (it / FQ_STAGES) & 1, abortp, status)) break;
          if (!mbar_wait(&misc->logits_free[buf], ((it >> 1) & 1) ^ 1, abortp, status)) break;
          tcgen05_fence_after();
          const uint64_t dX = desc_advance(dX0, st * TILE_BYTES);
#pragma unroll
          for (int k = 0; k < TC_D / 16; k++)
            mma_bf16(tmem + buf * TC_M, desc_advance(dX, 32 * k), desc_advance(dW, 32 * k), ID_LOGITS, k > 0);
#pragma unroll
          for (int k = 0; k < TC_D / 16; k++)
            mma_bf16(tmem + buf * TC_M, desc_advance(dX, 32 * k), desc_advance(dWlo, 32 * k), ID_LOGITS, 1);
          mma_commit(&misc->logits_full[buf]);
          mma_commit(&misc->empty[st]);
        }
      }
    }
  } else {
    regs_acquire<REGS_EPILOGUE>();
    // one query row per thread, 128 of the 256 features; the two threads of a row agree on the row maximum
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    for (int it = 0; it < ntiles; it++) {
      const int buf = it & 1;
      if (!mbar_wait(&misc->logits_full[buf], (it >> 1) & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      uint32_t v[128];
#pragma unroll
      for (int c = 0; c < 8; c++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + buf * TC_M + hf * 128 + c * 16, t);
#pragma unroll
        for (int j = 0; j < 16; j++) v[c * 16 + j] = t[j];
      }
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->logits_free[buf], lane);
      float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < 128; i += 4) {
        const float4 a4 = *reinterpret_cast<const float4*>(ah + hf * 128 + i);
        v[i] = __float_as_uint(__uint_as_float(v[i]) + a4.x);
        v[i + 1] = __float_as_uint(__uint_as_float(v[i + 1]) + a4.y);
        v[i + 2] = __float_as_uint(__uint_as_float(v[i + 2]) + a4.z);
        v[i + 3] = __float_as_uint(__uint_as_float(v[i + 3]) + a4.w);
      }
#pragma unroll
      for (int i = 0; i < 128; i++) mxp[i & 3] = fmaxf(mxp[i & 3], __uint_as_float(v[i]));
      float mx = fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3]));
      float* rm = rowmax + buf * 2 * TILE;
      rm[hf * TILE + row] = mx;
      if (threadIdx.x == 0 && it > 0) bulk_wait_read2();      // all stores but the previous tile's last two have read their slots
      named_bar_sync(1, EPI_THREADS);
      mx = fmaxf(mx, rm[(hf ^ 1) * TILE + row]);
      // the tile goes to shared memory in the layout of an MMA operand and leaves as one TMA store per
      // 64-feature block
      const int slot0 = (4 * it + 2 * hf) % FQ_PHI_SLOTS, slot1 = (4 * it + 2 * hf + 1) % FQ_PHI_SLOTS;
      uint8_t* prow0 = sm + FqSmem::PHI + slot0 * TILE_BYTES + row * 128;
      uint8_t* prow1 = sm + FqSmem::PHI + slot1 * TILE_BYTES + row * 128;
#pragma unroll
      for (int c = 0; c < 16; c++) {
        uint32_t p[4];
#pragma unroll
        for (int j = 0; j < 4; j++)
          p[j] = pack_bf16(ex2(__uint_as_float(v[c * 8 + 2 * j]) - mx), ex2(__uint_as_float(v[c * 8 + 2 * j + 1]) - mx));
        *reinterpret_cast<uint4*>((c < 8 ? prow0 : prow1) + (((c & 7) ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
      }
      fence_proxy_async_smem();
      named_bar_sync(2, EPI_THREADS);
      if (threadIdx.x == 0) {
#pragma unroll
        for (int fb = 0; fb < TC_M / 64; fb++) {
          tma_store_3d(&tmPhi, sm + FqSmem::PHI + ((4 * it + fb) % FQ_PHI_SLOTS) * TILE_BYTES, fb * 64, (tile0 + it) * TILE, bh);
          bulk_commit();
        }
      }
    }
    if (threadIdx.x == 0) bulk_wait0();
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------
// exclusive scan over chunks
// ------------------------------------------------------------------------------------------
// state[bh][c]: [80][256] bf16, chunk c's [V | 1]^T phiK with phiK = 2^(exponent - s_c); pmax its largest
// magnitude.  For every chunk c the kernel writes
//   prefix[bh][c] = alpha_c 2^(-e_c) sum_{c' < c} 2^(s_c' - sigma_c) state[c']   (bf16),
//   beta[bh][c],
// where sigma_c = max_{c' < c} s_c', e_c brings the sum to order 2^14, and (alpha_c, beta_c) <= 1 put the
// prefix term (true scale 2^(sigma_c + e_c)) and the in-chunk term (true scale 2^(s_c)) on one scale.
constexpr int PFX_SLICES = 10;               // 80 x 256 elements = 10 x 256 threads x 8
constexpr int PFX_MAXCH = 1024;
__global__ void __launch_bounds__(256)
tc_causal_prefix_kernel(const __nv_bfloat16* __restrict__ state, const float* __restrict__ shifts, const int* __restrict__ pmax,
                        int nch, __nv_bfloat16* __restrict__ prefix, float* __restrict__ beta) {
  __shared__ float up[PFX_MAXCH], add[PFX_MAXCH], oscale[PFX_MAXCH];
  const int bh = blockIdx.y;
  if (threadIdx.x == 0) {
    float sigma = -INFINITY, bound = 0.f;
    for (int c = 0; c < nch; c++) {
      const size_t i2 = ((size_t)bh * nch + c) * 2;
      const float sc = shifts[i2];            // both halves carry the same shift
      const float pm = fmaxf(__int_as_float(pmax[i2]), __int_as_float(pmax[i2 + 1]));
      float os = 0.f, bt = 1.f;
      if (c > 0 && bound > 0.f && isfinite(bound)) {
        int ex = 0;
        frexpf(bound, &ex);
        const float t_inter = sigma + (float)(ex - 14), tau = fmaxf(t_inter, sc);
        os = exp2f((float)(14 - ex)) * exp2f(t_inter - tau);
        bt = exp2f(sc - tau);
      }
      oscale[c] = os;
      if (blockIdx.x == 0) beta[(size_t)bh * nch + c] = bt;
      const float sn = fmaxf(sigma, sc);
      up[c] = sigma == -INFINITY ? 0.f : exp2f(sigma - sn);
      add[c] = exp2f(sc - sn);
      bound = bound * up[c] + add[c] * pm;
      sigma = sn;
    }
  }
  __syncthreads();
  // thread t of slice x owns columns 2 (t % 128), 2 (t % 128) + 1 of rows 8x + 4 (t / 128) .. + 3: states come in
  // and prefixes go out as bf16 pairs (4-byte accesses, a warp's access = 128 contiguous bytes)
  const int cp = threadIdx.x & 127, n0 = blockIdx.x * 8 + (threadIdx.x >> 7) * 4;
  const uint32_t* sb = reinterpret_cast<const uint32_t*>(state + (size_t)bh * nch * TC_NV * TC_M) + cp;
  uint32_t* pb = reinterpret_cast<uint32_t*>(prefix + (size_t)bh * nch * TC_NV * TC_M) + cp;
  float R[4][2];
#pragma unroll
  for (int u = 0; u < 4; u++) R[u][0] = R[u][1] = 0.f;
  // eight chunks per trip: their loads are issued together, then the running sums move on
  for (int c0 = 0; c0 < nch; c0 += 8) {
    uint32_t kv[8][4];
#pragma unroll
    for (int k = 0; k < 8; k++)
#pragma unroll
      for (int u = 0; u < 4; u++)
        kv[k][u] = (c0 + k < nch && n0 + u <= TC_DV) ? sb[((size_t)(c0 + k) * TC_NV + n0 + u) * (TC_M / 2)] : 0u;
#pragma unroll
    for (int k = 0; k < 8; k++) {
      const int c = c0 + k;
      if (c < nch) {
        const float os = oscale[c], upc = up[c], adc = add[c];
#pragma unroll
        for (int u = 0; u < 4; u++) {
          pb[((size_t)c * TC_NV + n0 + u) * (TC_M / 2)] = pack_bf16(R[u][0] * os, R[u][1] * os);
          R[u][0] = fmaf(R[u][0], upc, adc * __uint_as_float(kv[k][u] << 16));
          R[u][1] = fmaf(R[u][1], upc, adc * __uint_as_float(kv[k][u] & 0xffff0000u));
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// causal query side
// ------------------------------------------------------------------------------------------
struct CoSmem {
  // PHIK doubles as the masked score tile S (bf16, two 64-key blocks) once the score MMAs have read it
  static constexpr uint32_t PHIQ = 0, PHIK = 4 * TILE_BYTES, PFX = 8 * TILE_BYTES, V = PFX + KVT_BYTES, STAGE = V + TILE_BYTES,
                            RSUM = STAGE + (EPI_THREADS / 32) * 2048, MISC = RSUM + 2 * TILE * 4, TOTAL = MISC + 256;
};
static_assert(CoSmem::PFX % 1024 == 0 && CoSmem::V % 1024 == 0, "swizzled tiles need 1024-byte alignment");
static_assert(CoSmem::TOTAL + 1024 <= 232448, "shared memory budget");
struct CoMisc {
  uint64_t full, s_ready, s_full, out_done, chunk_free;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr uint32_t CO_COL_OUT = 0, CO_COL_S = 128, CO_TMEM_COLS = 256;
constexpr uint32_t CO_CHUNK_BYTES = 8 * TILE_BYTES + KVT_BYTES + TILE_BYTES;

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_causal_out_kernel(const __grid_constant__ CUtensorMap tmPhiQ, const __grid_constant__ CUtensorMap tmPhiK,
                     const __grid_constant__ CUtensorMap tmPfx, const __grid_constant__ CUtensorMap tmV,
                     const float* __restrict__ beta, int H, int L, int nch, int chunks_per_block,
                     __nv_bfloat16* __restrict__ Y, TensorAddr ay, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  CoMisc* misc = reinterpret_cast<CoMisc*>(sm + CoSmem::MISC);
  float* rsum = reinterpret_cast<float*>(sm + CoSmem::RSUM);      // [half][row]: row sums of the rounded masked scores
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int c0 = blockIdx.x * chunks_per_block;
  const int nmine = min(chunks_per_block, nch - c0);
  if (nmine <= 0) return;                     // uniform over the block, before anything is allocated
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&misc->full, 1);
    mbar_init(&misc->s_ready, 1);
    mbar_init(&misc->s_full, EPI_THREADS / 32);
    mbar_init(&misc->out_done, 1);
    mbar_init(&misc->chunk_free, EPI_THREADS / 32);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == WARP_MMA) {
    tmem_alloc(&misc->tmem_base, CO_TMEM_COLS);
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
        prefetch_tmap(&tmPhiQ);
        prefetch_tmap(&tmPhiK);
        prefetch_tmap(&tmPfx);
        prefetch_tmap(&tmV);
        int issued = 0;
        for (int it = 0; it < nmine; it++) {
          const int c = c0 + it;
          if (it > 0 && !mbar_wait(&misc->chunk_free, (it - 1) & 1, abortp, status)) break;
          mbar_expect_tx(&misc->full, CO_CHUNK_BYTES);
#pragma unroll
          for (int fb = 0; fb < TC_M / 64; fb++) {
            tma_load_3d(sm + CoSmem::PHIQ + fb * TILE_BYTES, &tmPhiQ, &misc->full, fb * 64, c * TILE, bh);
            tma_load_3d(sm + CoSmem::PHIK + fb * TILE_BYTES, &tmPhiK, &misc->full, fb * 64, c * TILE, bh);
            tma_load_3d(sm + CoSmem::PFX + fb * KVT_BLOCK_BYTES, &tmPfx, &misc->full, fb * 64, 0, bh * nch + c);
          }
          tma_load_4d(sm + CoSmem::V, &tmV, &misc->full, 0, c * TILE, h, b);
          issued = it + 1;
          if (it + 1 < nmine) {           // the next chunk's operands: into L2 while this one is worked on
#pragma unroll
            for (int fb = 0; fb < TC_M / 64; fb++) {
              tma_prefetch_3d(&tmPhiQ, fb * 64, (c + 1) * TILE, bh);
              tma_prefetch_3d(&tmPhiK, fb * 64, (c + 1) * TILE, bh);
              tma_prefetch_3d(&tmPfx, fb * 64, 0, bh * nch + c + 1);
            }
            tma_prefetch_4d(&tmV, 0, (c + 1) * TILE, h, b);
          }
        }
        // no copy of this block may still be in flight when it exits
        if (issued > 0) mbar_wait(&misc->full, (issued - 1) & 1, abortp, status, false);
      }
    } else if (warp == WARP_MMA) {
      if (lane == 0) {
        constexpr uint32_t ID_INTER = idesc_bf16(128, TC_NV, 0, 0);      // phiQ P^T
        constexpr uint32_t ID_SCORE = idesc_bf16(128, 128, 0, 0);        // phiQ phiK^T
        constexpr uint32_t ID_SV = idesc_bf16(128, TC_DV, 0, 1);        // S V (V with the value index contiguous)
        const uint64_t dQ = smem_desc(smem_u32(sm + CoSmem::PHIQ), 16, 1024, SWZ_128B);
        const uint64_t dK = smem_desc(smem_u32(sm + CoSmem::PHIK), 16, 1024, SWZ_128B);
        const uint64_t dP = smem_desc(smem_u32(sm + CoSmem::PFX), 16, 1024, SWZ_128B);
        const uint64_t dV = smem_desc(smem_u32(sm + CoSmem::V), TILE_BYTES, 1024, SWZ_128B);
        for (int it = 0; it < nmine; it++) {
          if (!mbar_wait(&misc->full, it & 1, abortp, status)) break;
          tcgen05_fence_after();
#pragma unroll 1
          for (int fb = 0; fb < TC_M / 64; fb++) {
#pragma unroll
            for (int k = 0; k < 4; k++)
              mma_bf16(tmem + CO_COL_OUT, desc_advance(dQ, fb * TILE_BYTES + 32 * k), desc_advance(dP, fb * KVT_BLOCK_BYTES + 32 * k),
                       ID_INTER, (fb | k) ? 1u : 0u);
          }
#pragma unroll 1
          for (int fb = 0; fb < TC_M / 64; fb++) {
#pragma unroll
            for (int k = 0; k < 4; k++)
              mma_bf16(tmem + CO_COL_S, desc_advance(dQ, fb * TILE_BYTES + 32 * k), desc_advance(dK, fb * TILE_BYTES + 32 * k),
                       ID_SCORE, (fb | k) ? 1u : 0u);
          }
          mma_commit(&misc->s_ready);
          if (!mbar_wait(&misc->s_full, it & 1, abortp, status)) break;
          tcgen05_fence_after();
          // S tile: [128 queries x 128 keys] bf16 in the phiK region, two 64-key blocks
#pragma unroll 2
          for (int j = 0; j < TILE / 16; j++)
            mma_bf16(tmem + CO_COL_OUT, desc_advance(dK, (j >> 2) * TILE_BYTES + 32 * (j & 3)), desc_advance(dV, j * 2048), ID_SV, 1u);
          mma_commit(&misc->out_done);
        }
      }
    }
  } else {
    regs_acquire<REGS_EPILOGUE>();
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    __nv_bfloat16* Yb = Y + b * ay.sb + h * ay.sh;
    for (int it = 0; it < nmine; it++) {
      const int c = c0 + it;
      const float bt = beta[(size_t)bh * nch + c];
      if (!mbar_wait(&misc->s_ready, it & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      // this thread's 64 keys of its query row: mask (key <= query), scale, round to bf16
      float sum = 0.f;
      uint8_t* srow = sm + CoSmem::PHIK + hf * TILE_BYTES + row * 128;
#pragma unroll
      for (int cc = 0; cc < 4; cc++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + CO_COL_S + hf * 64 + cc * 16, t);
        tmem_wait_ld();
        uint32_t p[8];
#pragma unroll
        for (int j = 0; j < 8; j++) {
          const int k0 = hf * 64 + cc * 16 + 2 * j;
          const float s0 = k0 <= row ? __uint_as_float(t[2 * j]) * bt : 0.f;
          const float s1 = k0 + 1 <= row ? __uint_as_float(t[2 * j + 1]) * bt : 0.f;
          p[j] = pack_bf16(s0, s1);
          sum += __uint_as_float(p[j] << 16) + __uint_as_float(p[j] & 0xffff0000u);
        }
        *reinterpret_cast<uint4*>(srow + (((2 * cc) ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
        *reinterpret_cast<uint4*>(srow + (((2 * cc + 1) ^ (row & 7)) << 4)) = make_uint4(p[4], p[5], p[6], p[7]);
      }
      rsum[hf * TILE + row] = sum;
      fence_proxy_async_smem();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->s_full, lane);
      if (!mbar_wait(&misc->out_done, it & 1, abortp, status, false)) break;
      __syncwarp();
      tcgen05_fence_after();
      uint32_t n0[32], d0[16];
      tmem_ld16(lane_addr + CO_COL_OUT + hf * 32, reinterpret_cast<uint32_t(&)[16]>(n0[0]));
      tmem_ld16(lane_addr + CO_COL_OUT + hf * 32 + 16, reinterpret_cast<uint32_t(&)[16]>(n0[16]));
      tmem_ld16(lane_addr + CO_COL_OUT + TC_DV, d0);
      tmem_wait_ld();
      const float den = __uint_as_float(d0[0]) + rsum[row] + rsum[TILE + row];
      const int64_t r0 = (int64_t)c * TILE + q * 32;                  // first row of this warp
      if (r0 + lane < L && (!(den > 0.f) || !isfinite(den))) atomicExch(status, FSHARP_E_NONFINITE);
      const float inv = 1.f / den;
      uint8_t* stg = sm + CoSmem::STAGE + warp * 2048;
#pragma unroll
      for (int i = 0; i < 4; i++) {
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; e++)
          o[e] = pack_bf16(inv * __uint_as_float(n0[8 * i + 2 * e]), inv * __uint_as_float(n0[8 * i + 2 * e + 1]));
        *reinterpret_cast<uint4*>(stg + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 4; i++) {
        const int rr = (lane >> 2) + 8 * i, cw = lane & 3;
        const uint4 val = *reinterpret_cast<const uint4*>(stg + rr * 64 + ((cw ^ ((rr >> 1) & 3)) << 4));
        if (r0 + rr < L) *reinterpret_cast<uint4*>(Yb + (r0 + rr) * ay.sl + hf * 32 + cw * 8) = val;
      }
      __syncwarp();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->chunk_free, lane);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, CO_TMEM_COLS);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
int make_map_kvt(CUtensorMap* map, const void* base, int BH, int bf16);
int make_map_feat(CUtensorMap* map, const void* base, int BH, int Lpad);
}  // namespace tchost
int fs_tc_key_side(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                   const int* flags, int tiles_per_split, int nsplit, float* crow, float* partial, float* shifts, int* pmax,
                   __nv_bfloat16* phik);
int fs_tc_causal_supported(const fsharp_dims* dm, int chunk);
size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                 const int* flags, void* Y, WsAlloc* ws);

int fs_tc_causal_supported(const fsharp_dims* dm, int chunk) {
  if (chunk != TILE || dm->Lq != dm->Lk || dm->Lq <= 0) return 0;
  const int nch = (dm->Lq + TILE - 1) / TILE;
  return nch <= PFX_MAXCH;
}

size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm) {
  (void)ctx;
  const size_t BH = (size_t)dm->B * dm->H, G = fs_groups(dm);
  const size_t nch = (dm->Lk + TILE - 1) / TILE, Lpad = nch * TILE;
  return ws_round(G * 2 * IMG_BYTES) + ws_round(G * 2 * FLAG_WORDS * 4 + 64) + ws_round(BH * nch * TC_M * TC_NV * 4) +
         2 * ws_round(BH * nch * 2 * 4) + ws_round(BH * Lpad * 4) + 2 * ws_round(BH * Lpad * TC_M * 2) +
         ws_round(BH * nch * TC_NV * TC_M * 2) + ws_round(BH * nch * 4);
}

int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                 const int* flags, void* Y, WsAlloc* ws) {
  const int B = dm->B, H = dm->H, BH = B * H, L = dm->Lq;
  const int nch = (L + TILE - 1) / TILE, Lpad = nch * TILE;
  __nv_bfloat16* state = ws->take<__nv_bfloat16>((size_t)BH * nch * TC_M * TC_NV);     // chunk states, bf16
  float* shifts = ws->take<float>((size_t)BH * nch * 2);
  int* pmax = ws->take<int>((size_t)BH * nch * 2);
  float* crow = ws->take<float>((size_t)BH * Lpad);
  __nv_bfloat16* phik16 = ws->take<__nv_bfloat16>((size_t)BH * Lpad * TC_M);
  __nv_bfloat16* phiq16 = ws->take<__nv_bfloat16>((size_t)BH * Lpad * TC_M);
  __nv_bfloat16* prefix = ws->take<__nv_bfloat16>((size_t)BH * nch * TC_NV * TC_M);
  float* beta = ws->take<float>((size_t)BH * nch);
  FS_CUDA_OK(cudaMemsetAsync(pmax, 0, (size_t)BH * nch * 2 * sizeof(int), ctx->stream));

  // query features
  CUtensorMap tmQ, tmPhiQ, tmPhiK, tmPfx, tmV;
  FS_TRY(tchost::make_map_tokens(&tmQ, Q, fs_addr(dm->q_stride, H, L, dm->d), B, H, L, dm->d));
  FS_TRY(tchost::make_map_tokens(&tmV, V, fs_addr(dm->v_stride, H, L, dm->dv), B, H, L, dm->dv));
  FS_TRY(tchost::make_map_feat(&tmPhiQ, phiq16, BH, Lpad));
  FS_TRY(tchost::make_map_feat(&tmPhiK, phik16, BH, Lpad));
  FS_TRY(tchost::make_map_kvt(&tmPfx, prefix, BH * nch, 1));
  // blocks of equal tile count: (waves of blocks) x (tiles per block + fill and drain)
  auto split = [&](int overhead, int* per) {
    int best = 1, best_cost = 0x7fffffff, best_per = nch;
    for (int ns = 1; ns <= nch; ns++) {
      const int t = (nch + ns - 1) / ns;
      if ((nch + t - 1) / t != ns) continue;
      const long long blocks = (long long)BH * ns;
      const int cost = (int)((blocks + ctx->sm_count - 1) / ctx->sm_count) * (t + overhead);
      if (cost < best_cost) { best_cost = cost; best = ns; best_per = t; }
    }
    *per = best_per;
    return best;
  };
  // key side: chunk states and bf16 key features
  int kper = 0;
  const int ksplit = split(4, &kper);
  FS_TRY(fs_tc_key_side(ctx, K, V, dm, images, flags, kper, ksplit, crow, reinterpret_cast<float*>(state), shifts, pmax, phik16));
  int qper = 0;
  const int qsplit = split(4, &qper);
  FS_CUDA_OK(cudaFuncSetAttribute(tc_featq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FqSmem::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_FEATQ);
  tc_featq_kernel<<<dim3(qsplit, BH), TC_THREADS, FqSmem::TOTAL + 1024, ctx->stream>>>(tmQ, tmPhiQ, images, H, dm->pool, L, qper,
                                                                                       ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);

  FS_TIME_BEGIN(ctx, FS_K_TC_CAUSAL_PREFIX);
  tc_causal_prefix_kernel<<<dim3(PFX_SLICES, BH), 256, 0, ctx->stream>>>(state, shifts, pmax, nch, prefix, beta);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);

  int cper = 0;
  const int csplit = split(2, &cper);
  FS_CUDA_OK(cudaFuncSetAttribute(tc_causal_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CoSmem::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_CAUSAL_OUT);
  tc_causal_out_kernel<<<dim3(csplit, BH), TC_THREADS, CoSmem::TOTAL + 1024, ctx->stream>>>(
      tmPhiQ, tmPhiK, tmPfx, tmV, beta, H, L, nch, cper, (__nv_bfloat16*)Y, fs_addr(dm->y_stride, H, L, dm->dv), ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
