// Tensor-core path, causal attention (Section 2.2's formula with a lower-triangular mask) for
// bf16, d = dv = 64, M = 256.  With P = phi(Q), S = phi(K) (Section 2.1) and tiles of 128 tokens,
//
//   [num | den]_c = P_c T_{c-1} + tril(P_c S_c^T) [V_c | 1],      T_c = T_{c-1} + S_c^T [V_c | 1],
//
// evaluated by ONE kernel per segment of consecutive tiles: the features of a tile are computed in the
// kernel and never leave the SM, and the state T is carried from tile to tile in tensor memory.
//
//   tc_kv_kernel (tc_bidir.cu)  totals S^T [V | 1] of the segments that have a successor (fp32 partials)
//   tc_causal_kernel            one block per (segment, batch, head): starts from the sum of the earlier
//                               segments' totals and walks its tiles
//
// Per tile (tensor memory columns in brackets):
//   logits of the keys, then of the queries, 128 features at a time  X Wh^T         [L: 128 columns]
//   phi(K) -> bf16 tile in shared memory (the B operand of the scores, the A operand of the state update)
//   phi(Q) -> bf16, written back over its own logits [L] and read from there as the A operand
//   [scores | inter-tile output] = phi(Q) [phi(K)^T | bf16(T)]      one MMA stream, N = 208   [S: 128][O: 80]
//   scores masked (key <= query), rounded to bf16 over their own columns
//   O += masked scores (from tensor memory) [V | 1]: column 64 collects the denominators       [O]
//   T += phi(K)^T [V | 1], 128 features per accumulator                                       [T: 2 x 80]
//   bf16(T) for the next tile: the accumulators are read back and written to shared memory
//   Y rows of the previous tile: [O] normalised, staged in the idle token tile, one TMA store per warp
// A block may also start from handed-in totals of keys that precede its whole sequence (sequence parallelism).
// The token tiles are converted from bf16 to fp16 in shared memory (exact for |x| in [2^-14, 65504]), so the
// logits need one fp16 image of W (11 significant bits) instead of a bf16 value and its remainder.
// The keys of a segment share one running shift (raised, with the state rescaled, when a tile's largest
// exponent exceeds it by the headroom); it cancels between numerator and denominator.
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

// Warps 0-3 are the producer warpgroup (0: TMA copies, 1: all MMAs; 0, 2 and 3: token tiles to fp16), warps 4-11
// the epilogue.  Every scheduler thus carries one producer warp and two epilogue warps: the epilogue warps of a
// tile meet at barriers several times per tile, so the slowest scheduler sets the pace.
constexpr int CF_WARP_TMA = 0, CF_WARP_MMA = 1, CF_WARP_CVT0 = 2, CF_PRODUCER_WARPS = 4;
constexpr int CVT_THREADS = 96;       // warps 0, 2 and 3 (each shares its scheduler with two epilogue warps; so does the MMA warp)
// Of every four pairs of exponentials, this many are evaluated on the multiply-add pipe (exp2_poly2), the others
// by the special-function unit, whose 16 results per clock would otherwise bound the kernel.
constexpr int CF_POLY_PAIRS_K = 1, CF_POLY_PAIRS_Q = 1;     // key features, query features (2 for either is slower here)
// The MMA-issuing thread of this kernel keeps more descriptors alive than those of the other kernels:
// 128 x 64 + 256 x 216 registers (of the 384 x 168 the block is launched with).
constexpr int CF_REGS_PRODUCER = 64, CF_REGS_EPILOGUE = 216;

struct CfSmem {
  // KP: four blocks of 64 features, each [phi(K) 128 keys x 64 | bf16(T) 80 rows x 64], so that one K-major
  // operand of 208 rows covers both
  static constexpr uint32_t W1 = 0, W2 = IMG_W_BYTES, X = 2 * IMG_W_BYTES, V = X + TILE_BYTES, ONES = V + TILE_BYTES,
                            KP = ONES + TILE_BYTES, BLK = TILE_BYTES + KVT_BLOCK_BYTES,
                            // row maxima of the query logits, exchanged between the two threads of a row: [2][128] floats
                            ROWMAX = KP + 4 * BLK,
                            // per-feature term as an MMA operand: [256 features x 16] fp16, no swizzle (8 x 16-byte core
                            // matrices: the two 16-byte K pieces of a row 128 bytes apart, 8-row groups 256 bytes apart)
                            A2OP = ROWMAX + 2 * TILE * 4, A2OP_BYTES = TC_M * 32, MISC = A2OP + A2OP_BYTES, TOTAL = MISC + 256;
};
static_assert(CfSmem::KP % 1024 == 0 && CfSmem::BLK % 1024 == 0 && CfSmem::X % 1024 == 0, "swizzled tiles need 1024-byte alignment");
static_assert(CfSmem::TOTAL + 1024 <= 232448, "shared memory budget");

struct CfMisc {
  uint64_t const_bar, x_full, x_ready, x_free, v_full, v_free, lg_full, lg_free, phik_full[2], phiq_full[5], p_full,
      s_ready, sm_full, o_ready, o_free, st_ready,
      stage_free;   // the output rows staged in the token tile have been read by their copies to global memory
  // meeting points of the epilogue warps (the two warps of a row quarter; all eight): mbarriers, so that these
  // waits are bounded like every other
  uint64_t pair_bar[4], all_bar;
  uint32_t tmem_base;
  int abort_flag;
  int chunk_max[3];
};
static_assert(sizeof(CfMisc) <= 256, "misc block");

// tensor memory columns; CF_ONE: an A operand of one K step whose first two K elements are 1 (fp16) in every row
constexpr uint32_t CF_L = 0, CF_S = 128, CF_O = 256, CF_T = 336, CF_ONE = 496;

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_causal_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmY,
                 const uint8_t* __restrict__ images,
                 const float* __restrict__ crow, const float* __restrict__ partial, const float* __restrict__ shifts,
                 int nsplit1, int nprefix, int H, int pool, int L, int Lpad, int tiles_per_seg, int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  CfMisc* misc = reinterpret_cast<CfMisc*>(sm + CfSmem::MISC);
  float* rowmax = reinterpret_cast<float*>(sm + CfSmem::ROWMAX);   // [half][row]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seg = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = seg * tiles_per_seg;
  const int ntiles = min(tiles_per_seg, total_tiles - tile0);
  if (ntiles <= 0) return;                    // uniform over the block, before anything is allocated
  const uint8_t* img1 = images + ((size_t)g * 2 + 0) * IMG_BYTES;        // side 1 (queries)
  const uint8_t* img2 = images + ((size_t)g * 2 + 1) * IMG_BYTES;        // side 2 (keys)
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&misc->const_bar, 1);
    mbar_init(&misc->x_full, 1);
    mbar_init(&misc->x_ready, CVT_THREADS / 32);
    mbar_init(&misc->x_free, 1);
    mbar_init(&misc->v_full, 1);
    mbar_init(&misc->v_free, 1);
    mbar_init(&misc->lg_full, 1);
    mbar_init(&misc->lg_free, EPI_THREADS / 32);
    for (int i = 0; i < 2; i++) mbar_init(&misc->phik_full[i], EPI_THREADS / 32);
    for (int i = 0; i < 5; i++) mbar_init(&misc->phiq_full[i], EPI_THREADS / 32);
    mbar_init(&misc->p_full, EPI_THREADS / 32);
    mbar_init(&misc->s_ready, 1);
    mbar_init(&misc->sm_full, EPI_THREADS / 32);
    mbar_init(&misc->o_ready, 1);
    mbar_init(&misc->o_free, EPI_THREADS / 32);
    mbar_init(&misc->st_ready, 1);
    mbar_init(&misc->stage_free, EPI_THREADS / 32);
    for (int i = 0; i < 4; i++) mbar_init(&misc->pair_bar[i], 2);
    mbar_init(&misc->all_bar, EPI_THREADS / 32);
    for (int j = 0; j < 3; j++) misc->chunk_max[j] = f2ord(-INFINITY);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  // constants written by the block itself: the second 64-column block of [V | 1] (a one in its first column) and
  // the zero rows 65..79 of bf16(T) (rows 0..64 are rewritten for every tile)
  for (int i = threadIdx.x; i < (int)(TILE_BYTES / 16); i += TC_THREADS) reinterpret_cast<uint4*>(sm + CfSmem::ONES)[i] = make_uint4(0, 0, 0, 0);
  for (int i = threadIdx.x; i < 4 * (int)(KVT_BLOCK_BYTES / 16); i += TC_THREADS)
    reinterpret_cast<uint4*>(sm + CfSmem::KP + (i / (KVT_BLOCK_BYTES / 16)) * CfSmem::BLK + TILE_BYTES)[i % (KVT_BLOCK_BYTES / 16)] =
        make_uint4(0, 0, 0, 0);
  // The per-feature term a2 = 2 log2e w^T A w of both sides joins the query logits inside their MMA: one more K step
  // whose A operand is [1, 1, 0, ...] in every row and whose B operand holds a2 as an fp16 value and its fp16 remainder.
  if (threadIdx.x < TC_M) {
    const float a2 = reinterpret_cast<const float*>(img1 + IMG_A2)[threadIdx.x];
    const __half hi = __float2half_rn(a2), lo = __float2half_rn(a2 - __half2float(hi));
    uint8_t* rowp = sm + CfSmem::A2OP + (threadIdx.x >> 3) * 256 + (threadIdx.x & 7) * 16;
    *reinterpret_cast<uint4*>(rowp) = make_uint4((uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16), 0, 0, 0);
    *reinterpret_cast<uint4*>(rowp + 128) = make_uint4(0, 0, 0, 0);
  }
  __syncthreads();
  if (threadIdx.x < TILE)
    *reinterpret_cast<__nv_bfloat16*>(sm + CfSmem::ONES + sw128_offset(threadIdx.x, 0)) = __float2bfloat16(1.f);
  fence_proxy_async_smem();
  if (warp == CF_WARP_MMA) {
    tmem_alloc(&misc->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = misc->tmem_base;

  if (warp < CF_PRODUCER_WARPS) {
    regs_release<CF_REGS_PRODUCER>();
    // bf16 -> fp16 of token tile n, in place (16-byte pieces keep their swizzled positions); t: 0 .. CVT_THREADS - 1
    auto convert_tile = [&](int n, int t) -> bool {
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->x_full, n & 1, abortp, status, false))) return false;    // warp-uniform
      uint4* xt = reinterpret_cast<uint4*>(sm + CfSmem::X);
#pragma unroll 4
      for (int i = t; i < (int)(TILE_BYTES / 16); i += CVT_THREADS) {
        uint4 u = xt[i];
        u.x = pack_f16(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
        u.y = pack_f16(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
        u.z = pack_f16(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
        u.w = pack_f16(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
        xt[i] = u;
      }
      fence_proxy_async_smem();
      mbar_arrive_warp(&misc->x_ready, lane);
      return true;
    };
    if (warp == CF_WARP_TMA) {
      // The whole warp walks the schedule (it also converts a third of every token tile); lane 0 issues the copies.
      if (lane == 0) {
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
        prefetch_tmap(&tmY);
        mbar_expect_tx(&misc->const_bar, 2 * IMG_W_BYTES);
        bulk_load(sm + CfSmem::W1, img1 + IMG_WH, IMG_W_BYTES, &misc->const_bar);
        bulk_load(sm + CfSmem::W2, img2 + IMG_WH, IMG_W_BYTES, &misc->const_bar);
      }
      // One token tile in shared memory serves keys and queries in turn: load 2 it is the key tile of tile it
      // (free once the second half of the key logits has been computed), load 2 it + 1 its query tile.
      int nx = 0, nv = 0;
      for (int it = 0; it < ntiles; it++) {
        const int tok = (tile0 + it) * TILE;
        if (nx > 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->x_free, (nx - 1) & 1, abortp, status))) break;
        // (between its query logits and this load the token tile staged the output rows of tile it - 2)
        if (it >= 2 && !__all_sync(0xffffffffu, mbar_wait(&misc->stage_free, (it - 2) & 1, abortp, status))) break;
        if (lane == 0) {
          mbar_expect_tx(&misc->x_full, TILE_BYTES);
          tma_load_4d(sm + CfSmem::X, &tmK, &misc->x_full, 0, tok, h, b);
          if (it + 1 < ntiles) {             // the next tile's operands: into L2 while this one is worked on
            tma_prefetch_4d(&tmK, 0, tok + TILE, h, b);
            tma_prefetch_4d(&tmQ, 0, tok + TILE, h, b);
            tma_prefetch_4d(&tmV, 0, tok + TILE, h, b);
          }
        }
        nx++;
        if (!convert_tile(nx - 1, lane)) break;
        if (nv > 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->v_free, (nv - 1) & 1, abortp, status))) break;
        if (lane == 0) {
          mbar_expect_tx(&misc->v_full, TILE_BYTES);
          tma_load_4d(sm + CfSmem::V, &tmV, &misc->v_full, 0, tok, h, b);
        }
        nv++;
        if (!__all_sync(0xffffffffu, mbar_wait(&misc->x_free, (nx - 1) & 1, abortp, status))) break;
        if (lane == 0) {
          mbar_expect_tx(&misc->x_full, TILE_BYTES);
          tma_load_4d(sm + CfSmem::X, &tmQ, &misc->x_full, 0, tok, h, b);
        }
        nx++;
        if (!convert_tile(nx - 1, lane)) break;
      }
      // no copy of this block may still be in flight when it exits
      if (lane == 0) {
        mbar_wait(&misc->const_bar, 0, abortp, status, false);
        if (nx > 0) mbar_wait(&misc->x_full, (nx - 1) & 1, abortp, status, false);
        if (nv > 0) mbar_wait(&misc->v_full, (nv - 1) & 1, abortp, status, false);
      }
    } else if (warp == CF_WARP_MMA) {
      // ---------------- all MMAs of the block.  The whole warp walks the schedule (descriptor arithmetic and waits
      // stay warp-uniform); one elected lane issues the MMAs and their commits.
      {
        constexpr uint32_t ID_LOGITS = idesc_f16(128, 128, 0, 0);            // X Wh^T, 128 features
        constexpr uint32_t ID_STATE = idesc_bf16(128, TC_NV, 1, 1);          // phi(K)_h^T [V | 1]
        constexpr uint32_t ID_SO = idesc_bf16(128, 128 + TC_NV, 0, 0);       // phi(Q) [phi(K)^T | bf16(T)]
        constexpr uint32_t ID_SV = idesc_bf16(128, TC_NV, 0, 1);             // masked scores x [V | 1]: the ones column adds the row sums
        const uint64_t dX = smem_desc(smem_u32(sm + CfSmem::X), 16, 1024, SWZ_128B);
        const uint64_t dW1 = smem_desc(smem_u32(sm + CfSmem::W1), 16, 1024, SWZ_128B);
        const uint64_t dW2 = smem_desc(smem_u32(sm + CfSmem::W2), 16, 1024, SWZ_128B);
        const uint32_t sV = smem_u32(sm + CfSmem::V), sOnes = smem_u32(sm + CfSmem::ONES);
        const uint64_t dKP = smem_desc(smem_u32(sm + CfSmem::KP), 16, 1024, SWZ_128B);             // K-major, 208 rows per block
        const uint64_t dPhiMN = smem_desc(smem_u32(sm + CfSmem::KP), CfSmem::BLK, 1024, SWZ_128B); // features contiguous
        const uint64_t dV1 = smem_desc(sV, sOnes - sV, 1024, SWZ_128B);                            // [V | 1], value index contiguous
        // low words (start address / 16) and high words of the descriptors; the low words are made opaque once per
        // tile so that the offsets are added next to each MMA
        uint32_t xl = (uint32_t)dX, w1l = (uint32_t)dW1, w2l = (uint32_t)dW2, kpl = (uint32_t)dKP, pml = (uint32_t)dPhiMN, v1l = (uint32_t)dV1;
        const uint32_t xh = (uint32_t)(dX >> 32), wh = (uint32_t)(dW1 >> 32), kph = (uint32_t)(dKP >> 32), pmh = (uint32_t)(dPhiMN >> 32),
                       v1h = (uint32_t)(dV1 >> 32);
        const uint64_t dA2 = smem_desc(smem_u32(sm + CfSmem::A2OP), 128, 256, SWZ_NONE);
        uint32_t a2l = (uint32_t)dA2;
        const uint32_t a2h = (uint32_t)(dA2 >> 32);
        auto issue_logits = [&](uint32_t wl, int half, bool with_a2) {
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < TC_D / 16; k++)
              mma_bf16_lh(tmem + CF_L, xl + 2 * k, xh, wl + half * (IMG_W_BYTES / 32) + 2 * k, wh, ID_LOGITS, k > 0);
            if (with_a2) mma_bf16_ta_lh(tmem + CF_L, tmem + CF_ONE, a2l + half * (128 * 32 / 16), a2h, ID_LOGITS, 1u);
            mma_commit(&misc->lg_full);
          }
          __syncwarp();
        };
        int nlg = 0, nxr = 0;                 // logits halves handed over so far, token tiles consumed so far
        bool ok = mbar_wait(&misc->const_bar, 0, abortp, status);
        if (ok) ok = mbar_wait(&misc->x_ready, nxr & 1, abortp, status);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
          tcgen05_fence_after();
          issue_logits(w2l, 0, false);
        }
        // a wait that gave up in one lane ends the schedule for the whole warp
#define CF_WAIT(bar, par) if (!__all_sync(0xffffffffu, mbar_wait((bar), (par), abortp, status))) break
        for (int it = 0; ok && it < ntiles; it++) {
          opaque(a2l); opaque(xl); opaque(w1l); opaque(w2l); opaque(kpl); opaque(pml); opaque(v1l);
          // second half of the key logits once the epilogue has taken the first out of tensor memory
          CF_WAIT(&misc->lg_free, nlg & 1);
          nlg++;
          tcgen05_fence_after();
          issue_logits(w2l, 1, false);
          if (elect_one()) mma_commit(&misc->x_free);
          __syncwarp();
          nxr++;
          // query logits
          CF_WAIT(&misc->lg_free, nlg & 1);
          nlg++;
          CF_WAIT(&misc->x_ready, nxr & 1);
          tcgen05_fence_after();
          issue_logits(w1l, 0, true);
          CF_WAIT(&misc->lg_free, nlg & 1);
          nlg++;
          tcgen05_fence_after();
          issue_logits(w1l, 1, true);
          if (elect_one()) mma_commit(&misc->x_free);
          __syncwarp();
          nxr++;
          // state update T_h += phi(K)_h^T [V | 1], once the epilogue has taken its bf16 copy of the state BEFORE this
          // tile (it does so between the two halves of the query logits); runs while it takes the row maxima
          CF_WAIT(&misc->v_full, it & 1);
          CF_WAIT(&misc->phik_full[0], it & 1);
          CF_WAIT(&misc->phik_full[1], it & 1);
          CF_WAIT(&misc->p_full, it & 1);
          tcgen05_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int j = 0; j < 2 * (TILE / 16); j++) {
              const int hh = j >> 3, k = j & 7;
              mma_bf16_lh(tmem + CF_T + hh * TC_NV, pml + hh * 2 * (CfSmem::BLK / 16) + k * 128, pmh, v1l + k * 128, v1h, ID_STATE, 1u);
            }
            mma_commit(&misc->st_ready);
          }
          __syncwarp();
          // scores and inter-tile output, 32 features (two K steps) of two blocks at a time
          if (it > 0) CF_WAIT(&misc->o_free, (it - 1) & 1);
          bool ok2 = true;
#pragma unroll
          for (int qt = 0; qt < 5; qt++) {
            // hand-over qt < 3: features 32 (qt % 2) .. + 32 of the blocks 2 (qt / 2), 2 (qt / 2) + 1 (two K steps each);
            // the last 32 features come in two hand-overs of one K step, so that little is left when the exponentials end
            if (!__all_sync(0xffffffffu, mbar_wait(&misc->phiq_full[qt], it & 1, abortp, status))) { ok2 = false; break; }
            tcgen05_fence_after();
            if (elect_one()) {
#pragma unroll
              for (int j = 0; j < (qt < 3 ? 4 : 2); j++) {
                const int fb = qt < 3 ? 2 * (qt >> 1) + (j >> 1) : 2 + j;
                const int k = qt < 3 ? 2 * (qt & 1) + (j & 1) : qt - 1;
                mma_bf16_ta_lh(tmem + CF_S, tmem + CF_L + fb * 32 + k * 8, kpl + fb * (CfSmem::BLK / 16) + 2 * k, kph, ID_SO,
                               (qt | j) ? 1u : 0u);
              }
              if (qt == 4) mma_commit(&misc->s_ready);
            }
            __syncwarp();
          }
          if (!ok2) break;
          // the next tile's first key logits go ahead of the masked-score product: they only need the columns that
          // the MMAs above have finished reading by the time they run (the pipe keeps issue order)
          CF_WAIT(&misc->lg_free, nlg & 1);      // (long since: the query logits were taken)
          nlg++;
          if (it + 1 < ntiles) {
            CF_WAIT(&misc->x_ready, nxr & 1);
            tcgen05_fence_after();
            issue_logits(w2l, 0, false);
          }
          CF_WAIT(&misc->sm_full, it & 1);
          tcgen05_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < TILE / 16; k++)
              mma_bf16_ta_lh(tmem + CF_O, tmem + CF_S + k * 8, v1l + k * 128, v1h, ID_SV, 1u);
            mma_commit(&misc->o_ready);
            mma_commit(&misc->v_free);
          }
          __syncwarp();
        }
#undef CF_WAIT
      }
    } else {
      // ---------------- bf16 -> fp16 of the token tiles, with the copying warp
      const int t = (warp - CF_WARP_CVT0 + 1) * 32 + lane;
      for (int n = 0; n < 2 * ntiles; n++)
        if (!convert_tile(n, t)) break;
    }
  } else {
    regs_acquire<CF_REGS_EPILOGUE>();
    // ---------------- epilogue warps.  As a token's thread: row = 32 q + lane, feature blocks hf and 2 + hf (64
    // features each; block hf comes out of the first logits half, block 2 + hf out of the second).  As a
    // feature's thread (state, bf16(T)): feature m = 128 hf + row, lane `row` of accumulator hf.
    const int q = warp & 3, hf = (warp - CF_PRODUCER_WARPS) >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const int m = hf * 128 + row;
    uint8_t* blk0 = sm + CfSmem::KP + hf * CfSmem::BLK;              // phi(K) block hf
    uint8_t* blk1 = sm + CfSmem::KP + (2 + hf) * CfSmem::BLK;        // phi(K) block 2 + hf
    // bf16(T): column m of T is column m % 64 of the 80-row block of feature block m / 64; row n of a 128-byte-swizzled
    // block keeps its 16-byte piece p at position p ^ (n % 8): one base address per value of n % 8
    uint32_t pcol[8];
#pragma unroll
    for (int k = 0; k < 8; k++)
      pcol[k] = smem_u32(sm + CfSmem::KP + (m >> 6) * CfSmem::BLK + TILE_BYTES) + (((((uint32_t)m & 63u) >> 3) ^ (uint32_t)k) << 4) +
                (((uint32_t)m & 7u) << 1);
    float s = -INFINITY;                                              // the keys' running shift
    bool alive = true;
    int npair = 0, nall = 0;
    // all threads of the two warps of row quarter q (resp. of all eight warps) have reached this point
    auto sync_pair = [&]() {
      mbar_arrive_warp(&misc->pair_bar[q], lane);
      if (!mbar_wait(&misc->pair_bar[q], npair & 1, abortp, status, false)) alive = false;
      npair++;
    };
    auto sync_all = [&]() {
      mbar_arrive_warp(&misc->all_bar, lane);
      if (!mbar_wait(&misc->all_bar, nall & 1, abortp, status, false)) alive = false;
      nall++;
    };
    // ---- the state before this segment: sum of the earlier segments' totals, brought to one shift
    {
      // key-side splits are segments; the first nprefix totals belong to keys that precede the whole sequence
      const int np = min(nsplit1, nprefix + seg);
      float val[TC_NV];
#pragma unroll
      for (int n = 0; n < TC_NV; n++) val[n] = 0.f;
      if (np > 0) {
        const float* sh = shifts + (size_t)bh * nsplit1 * 2;
        float smax = -INFINITY;
        for (int p = 0; p < 2 * np; p++) smax = fmaxf(smax, sh[p]);
        s = smax;
        const float* base = partial + (size_t)bh * nsplit1 * TC_NV * TC_M + m;
        for (int p = 0; p < np; p++) {
          const float f = exp2f(sh[2 * p + hf] - s);
          const float* bp = base + (size_t)p * TC_NV * TC_M;
#pragma unroll
          for (int n = 0; n <= TC_DV; n++) val[n] = fmaf(bp[n * TC_M], f, val[n]);
        }
      }
#pragma unroll
      for (int c = 0; c < TC_NV / 16; c++) {
        uint32_t a[16];
#pragma unroll
        for (int j = 0; j < 16; j++) a[j] = __float_as_uint(val[c * 16 + j]);
        tmem_st16(lane_addr + CF_T + hf * TC_NV + c * 16, a);
      }
      if (hf == 0) {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %2, %2, %2, %2, %2, %2};" ::"r"(lane_addr + CF_ONE),
                     "r"(0x3C003C00u), "r"(0u) : "memory");
      }
      tmem_wait_st();
      tcgen05_fence_before();
    }
    const float* cptr = crow + (size_t)bh * Lpad + (size_t)tile0 * TILE + row;
    float cj = cptr[0];

    // Y rows of tile j (all its MMAs have completed): 32 of the 64 columns per thread.  A warp's 32 rows x 64 bytes are
    // staged in its eighth of the token tile (idle between the query logits of a tile and the next tile's keys) with
    // the 64-byte swizzle and leave as one TMA store, which also drops the rows past the end of the sequence.
    auto write_out = [&](int j) {
      __syncwarp();
      tcgen05_fence_after();
      uint32_t n0[32], d0[8];
      tmem_ld16(lane_addr + CF_O + hf * 32, reinterpret_cast<uint32_t(&)[16]>(n0[0]));
      tmem_ld16(lane_addr + CF_O + hf * 32 + 16, reinterpret_cast<uint32_t(&)[16]>(n0[16]));
      tmem_ld8(lane_addr + CF_O + TC_DV, d0);
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->o_free, lane);
      const float den = __uint_as_float(d0[0]);
      const int r0 = (tile0 + j) * TILE + q * 32;                    // first row of this warp
      if (r0 + lane < L && (!(den > 0.f) || !isfinite(den))) atomicExch(status, FSHARP_E_NONFINITE);
      const float inv = 1.f / den;
      uint8_t* stg = sm + CfSmem::X + (warp - CF_PRODUCER_WARPS) * 2048;
#pragma unroll
      for (int i = 0; i < 4; i++) {
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; e++)
          o[e] = pack_bf16(inv * __uint_as_float(n0[8 * i + 2 * e]), inv * __uint_as_float(n0[8 * i + 2 * e + 1]));
        *reinterpret_cast<uint4*>(stg + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_4d(&tmY, stg, hf * 32, r0, h, b);
        bulk_commit();
      }
    };

    int nlg = 0;
    for (int it = 0; it < ntiles && alive; it++) {
      FS_DBG(tile0 + it < total_tiles && (size_t)tile0 * TILE + (size_t)(it + 1) * TILE <= (size_t)Lpad, status);
      FS_DBG(CF_T + hf * TC_NV + TC_NV <= CF_ONE && CF_ONE + 8 <= TMEM_COLS && CF_L + 2 * 64 <= CF_S, status);
      FS_DBG(pcol[7] + (uint32_t)TC_DV * 128u + 2u <= smem_u32(sm) + CfSmem::KP + 4 * CfSmem::BLK, status);
      FS_DBG(blk1 + row * 128 + 128 <= sm + CfSmem::KP + 4 * CfSmem::BLK && row < TILE, status);
      const float cnext = it + 1 < ntiles ? cptr[(size_t)(it + 1) * TILE] : 0.f;     // in flight during this tile
      uint32_t v[128];
      // ---- key logits, first half
      if (!mbar_wait(&misc->lg_full, nlg & 1, abortp, status, false)) { alive = false; break; }
      nlg++;
      __syncwarp();
      tcgen05_fence_after();
#pragma unroll
      for (int c = 0; c < 4; c++) tmem_ld16(lane_addr + CF_L + hf * 64 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->lg_free, lane);
      // ---- while the second half is computed: the maximum of the first
      float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < 64; i += 8) {
        mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
        mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
        mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
        mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
      }
      // the previous tile's state update has completed: nothing reads the previous phi(K) tile any more
      if (it > 0 && !mbar_wait(&misc->st_ready, (it - 1) & 1, abortp, status, false)) { alive = false; break; }
      // ---- key logits, second half
      if (!mbar_wait(&misc->lg_full, nlg & 1, abortp, status, false)) { alive = false; break; }
      nlg++;
      __syncwarp();
      tcgen05_fence_after();
#pragma unroll
      for (int c = 0; c < 4; c++) tmem_ld16(lane_addr + CF_L + hf * 64 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[64 + c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->lg_free, lane);
      const bool valid = (tile0 + it) * TILE + row < L;
      // ---- exact maximum of the tile's exponents, one value for the block
      float tm;
      {
#pragma unroll
        for (int i = 64; i < 128; i += 8) {
          mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
          mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
          mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
        }
        float mx = valid ? fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3])) + cj : -INFINITY;
        const int wm = __reduce_max_sync(0xffffffffu, f2ord(mx));       // one instruction for the warp's maximum
        if (lane == 0) atomicMax(&misc->chunk_max[it % 3], wm);
        if (threadIdx.x == CF_PRODUCER_WARPS * 32) misc->chunk_max[(it + 1) % 3] = f2ord(-INFINITY);   // next tile's slot; idle since tile it - 2
        sync_all();
        if (!alive) break;
        tm = ord2f(misc->chunk_max[it % 3]);
      }
      if (s == -INFINITY) {
        s = tm;                      // first keys of the sequence: the state is still zero
      } else if (tm - s > SHIFT_HEADROOM_LOG2) {
        // rare: the shift moves up to this tile's maximum and the state with it (the previous tile's update of the
        // state has completed: st_ready was waited for above)
        __syncwarp();
        tcgen05_fence_after();
        const float f = ex2(s - tm);
#pragma unroll
        for (int c = 0; c < TC_NV / 16; c++) {
          uint32_t a[16];
          tmem_ld16(lane_addr + CF_T + hf * TC_NV + c * 16, a);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; j++) a[j] = __float_as_uint(__uint_as_float(a[j]) * f);
          tmem_st16(lane_addr + CF_T + hf * TC_NV + c * 16, a);
        }
        tmem_wait_st();
        tcgen05_fence_before();
        s = tm;
      }
      // ---- phi(K): 2^(exponent - s), bf16, 64 features at a time.  Rows past the end of the sequence (last tile only)
      // are not zeroed: the mask removes their scores, and the state after the last tile is not used.
      {
        const float rc = cj - s;
#pragma unroll
        for (int half = 0; half < 2; half++) {
          uint8_t* prow = (half ? blk1 : blk0) + row * 128;
#pragma unroll
          for (int c = 0; c < 8; c++) {
            uint32_t p[4];
#pragma unroll
            for (int j = 0; j < 4; j++) {
              uint32_t& e0 = v[half * 64 + c * 8 + 2 * j];
              uint32_t& e1 = v[half * 64 + c * 8 + 2 * j + 1];
              add2(e0, e1, rc, rc);
              if (j < CF_POLY_PAIRS_K) {
                exp2_poly2(e0, e1);
                p[j] = pack_bf16(__uint_as_float(e0), __uint_as_float(e1));
              } else {
                p[j] = pack_bf16(ex2(__uint_as_float(e0)), ex2(__uint_as_float(e1)));
              }
            }
            *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
          }
          fence_proxy_async_smem();
          mbar_arrive_warp(&misc->phik_full[half], lane);
          if (*abortp) { alive = false; goto after_keys; }
        }
      }
    after_keys:
      if (!alive) break;
      // ---- query logits
      if (!mbar_wait(&misc->lg_full, nlg & 1, abortp, status, false)) { alive = false; break; }
      nlg++;
      __syncwarp();
      tcgen05_fence_after();
#pragma unroll
      for (int c = 0; c < 4; c++) tmem_ld16(lane_addr + CF_L + hf * 64 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->lg_free, lane);
      // ---- while the second half of the query logits is computed: bf16(T) of the state before this tile: row `row` of accumulator hf = column m of T.  The previous
      // tile's MMAs that read the old copy have completed (its scores were taken out of tensor memory).
      {
        __syncwarp();
        tcgen05_fence_after();
#pragma unroll
        for (int c = 0; c < TC_NV / 16; c++) {
          uint32_t a[16];
          tmem_ld16(lane_addr + CF_T + hf * TC_NV + c * 16, a);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; j++)
            if (c * 16 + j <= TC_DV) {
              const uint16_t hb = __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(a[j])));
              asm volatile("st.shared.u16 [%0], %1;" ::"r"(pcol[j & 7] + (uint32_t)(c * 16 + j) * 128u), "h"(hb) : "memory");
            }
        }
        tcgen05_fence_before();
        fence_proxy_async_smem();
        mbar_arrive_warp(&misc->p_full, lane);
      }
      if (!mbar_wait(&misc->lg_full, nlg & 1, abortp, status, false)) { alive = false; break; }
      nlg++;
      __syncwarp();
      tcgen05_fence_after();
#pragma unroll
      for (int c = 0; c < 4; c++) tmem_ld16(lane_addr + CF_L + hf * 64 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[64 + c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->lg_free, lane);
      // ---- the previous tile's output: its masked-score product has long completed (the scores of this tile wait for
      // it), and the query logits just taken were the last readers of the token tile
      if (it > 0) {
        if (!mbar_wait(&misc->o_ready, (it - 1) & 1, abortp, status, false)) { alive = false; break; }
        write_out(it - 1);
      }
      float mx;
      {
        float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
          mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
          mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
          mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
        }
        mx = fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3]));
        // the row's other thread sits in warp q of the other warpgroup; after this barrier both have also taken
        // their logits out of tensor memory, whose columns the features now overwrite
        rowmax[hf * TILE + row] = mx;
        sync_pair();
        if (!alive) break;
        mx = fmaxf(mx, rowmax[(hf ^ 1) * TILE + row]);
      }
      if (it > 0) {                    // the staged rows have been read: the token tile may take the next keys
        if (lane == 0) bulk_wait_read0();
        mbar_arrive_warp(&misc->stage_free, lane);
      }
      // ---- phi(Q): 2^(exponent - row maximum), bf16 pairs over the logits' columns: block fb at columns 32 fb
#pragma unroll
      for (int half = 0; half < 2; half++) {
        const int fb = 2 * half + hf;
#pragma unroll
        for (int c = 0; c < 2; c++) {
          uint32_t p[16];
#pragma unroll
          for (int j = 0; j < 16; j++) {
            uint32_t& e0 = v[half * 64 + c * 32 + 2 * j];
            uint32_t& e1 = v[half * 64 + c * 32 + 2 * j + 1];
            add2(e0, e1, -mx, -mx);
            if ((j & 3) < CF_POLY_PAIRS_Q) {
              exp2_poly2(e0, e1);
              p[j] = pack_bf16(__uint_as_float(e0), __uint_as_float(e1));
            } else {
              p[j] = pack_bf16(ex2(__uint_as_float(e0)), ex2(__uint_as_float(e1)));
            }
          }
          if (half == 1 && c == 1) {
            // columns of K step 2, then of K step 3
            uint32_t lo8[8], hi8[8];
#pragma unroll
            for (int j = 0; j < 8; j++) { lo8[j] = p[j]; hi8[j] = p[8 + j]; }
            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(lane_addr + CF_L + fb * 32 + 16),
                         "r"(lo8[0]), "r"(lo8[1]), "r"(lo8[2]), "r"(lo8[3]), "r"(lo8[4]), "r"(lo8[5]), "r"(lo8[6]), "r"(lo8[7]) : "memory");
            tmem_wait_st();
            tcgen05_fence_before();
            mbar_arrive_warp(&misc->phiq_full[3], lane);
            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(lane_addr + CF_L + fb * 32 + 24),
                         "r"(hi8[0]), "r"(hi8[1]), "r"(hi8[2]), "r"(hi8[3]), "r"(hi8[4]), "r"(hi8[5]), "r"(hi8[6]), "r"(hi8[7]) : "memory");
            tmem_wait_st();
            tcgen05_fence_before();
            mbar_arrive_warp(&misc->phiq_full[4], lane);
          } else {
            tmem_st16(lane_addr + CF_L + fb * 32 + c * 16, p);
            tmem_wait_st();
            tcgen05_fence_before();
            mbar_arrive_warp(&misc->phiq_full[2 * half + c], lane);
          }
          // A real branch after every hand-over: without one the instruction scheduler moves the (side-effect-free)
          // exponentials of the chunks that follow ahead of the hand-over, and all hand-overs bunch at the end.
          if (*abortp) { alive = false; goto after_queries; }
        }
      }
    after_queries:
      if (!alive) break;
      // ---- scores: mask (key <= query) and round to bf16 over their own columns (their row sums come out of the
      // product with [V | 1])
      if (!mbar_wait(&misc->s_ready, it & 1, abortp, status, false)) { alive = false; break; }
      __syncwarp();
      tcgen05_fence_after();
      {
        uint32_t pm[32];
#pragma unroll
        for (int cc = 0; cc < 2; cc++) {
          uint32_t t[32];
          tmem_ld16(lane_addr + CF_S + hf * 64 + cc * 32, reinterpret_cast<uint32_t(&)[16]>(t[0]));
          tmem_ld16(lane_addr + CF_S + hf * 64 + cc * 32 + 16, reinterpret_cast<uint32_t(&)[16]>(t[16]));
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; j++) {
            const int k0 = hf * 64 + cc * 32 + 2 * j;
            const float s0 = k0 <= row ? __uint_as_float(t[2 * j]) : 0.f;
            const float s1 = k0 + 1 <= row ? __uint_as_float(t[2 * j + 1]) : 0.f;
            pm[cc * 16 + j] = pack_bf16(s0, s1);
          }
        }
        // the packed scores of the row's second thread land on columns its first thread reads: both have read
        sync_pair();
        if (!alive) break;
        tmem_st16(lane_addr + CF_S + hf * 32, reinterpret_cast<uint32_t(&)[16]>(pm[0]));
        tmem_st16(lane_addr + CF_S + hf * 32 + 16, reinterpret_cast<uint32_t(&)[16]>(pm[16]));
        tmem_wait_st();
        tcgen05_fence_before();
        mbar_arrive_warp(&misc->sm_full, lane);
      }
      cj = cnext;
    }
    if (alive && mbar_wait(&misc->st_ready, (ntiles - 1) & 1, abortp, status, false) &&
        mbar_wait(&misc->o_ready, (ntiles - 1) & 1, abortp, status, false)) {
      write_out(ntiles - 1);
      if (lane == 0) bulk_wait0();                 // the block's shared memory outlives its copies
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == CF_WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
int make_map_out(CUtensorMap* map, void* base, TensorAddr a, int B, int H, int L, int inner);
}  // namespace tchost
int fs_tc_rowterm(fsharp_ctx* ctx, const void* K, const fsharp_dims* dm, const uint8_t* images, const int* flags, int Lpad,
                  int tiles_per_split, int nsplit, float* crow);
int fs_tc_key_side(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                   const int* flags, int tiles_per_split, int nsplit, float* crow, float* partial, float* shifts);
int fs_tc_causal_supported(const fsharp_dims* dm, int chunk);
size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                 const int* flags, void* Y, WsAlloc* ws);
size_t fs_tc_causal_prefix_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm, int nprefix);
int fs_tc_causal_prefix(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                        const int* flags, const float* pre_state, const float* pre_shifts, int nprefix, void* Y, WsAlloc* ws);

namespace {
constexpr int CF_MAX_SEG = 64;

// Segments of equal tile count per (batch, head).  A segment's block walks its tiles one after the other (about 2.2
// times a key-side tile each); every segment but the last also costs a key-side pass over its tiles.
int pick_segments(int units, int tiles, int sms, int* tiles_per_seg) {
  int best = 1, best_per = tiles;
  double best_cost = 1e300;
  for (int ns = 1; ns <= tiles && ns <= CF_MAX_SEG; ns++) {
    const int per = (tiles + ns - 1) / ns;
    if ((tiles + per - 1) / per != ns) continue;
    const long long b2 = (long long)units * ns, b1 = (long long)units * (ns - 1);
    double cost = (double)((b2 + sms - 1) / sms) * (2.2 * per + 3.0);
    if (ns > 1) cost += (double)((b1 + sms - 1) / sms) * (per + 4.0);
    if (cost < best_cost) { best_cost = cost; best = ns; best_per = per; }
  }
  *tiles_per_seg = best_per;
  return best;
}
}  // namespace

// The mask is applied token by token, so the result does not depend on `chunk`: the kernel always walks 128-token tiles.
int fs_tc_causal_supported(const fsharp_dims* dm, int chunk) {
  (void)chunk;
  return dm->Lq == dm->Lk && dm->Lq > 0;
}

size_t fs_tc_causal_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm) {
  (void)ctx;
  const size_t BH = (size_t)dm->B * dm->H, G = fs_groups(dm);
  const size_t nch = (dm->Lk + TILE - 1) / TILE, Lpad = nch * TILE;
  return ws_round(G * 2 * IMG_BYTES) + ws_round(G * 2 * FLAG_WORDS * 4 + 64) + ws_round(BH * CF_MAX_SEG * TC_M * TC_NV * 4) +
         2 * ws_round(BH * CF_MAX_SEG * 2 * 4) + ws_round(BH * Lpad * 4);
}

int fs_tc_causal(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                 const int* flags, void* Y, WsAlloc* ws) {
  return fs_tc_causal_prefix(ctx, Q, K, V, dm, images, flags, nullptr, nullptr, 0, Y, ws);
}

size_t fs_tc_causal_prefix_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm, int nprefix) {
  const size_t BH = (size_t)dm->B * dm->H;
  return fs_tc_causal_scratch_bytes(ctx, dm) + ws_round(BH * (size_t)(nprefix + CF_MAX_SEG) * TC_M * TC_NV * 4) +
         ws_round(BH * (size_t)(nprefix + CF_MAX_SEG) * 2 * 4);
}

// pre_state [B*H][nprefix][80][256], pre_shifts [B*H][nprefix][2]: key-side sums (in the layout of the key-side kernel's
// partials) of keys that precede every token of this call; nprefix = 0: none.
int fs_tc_causal_prefix(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                        const int* flags, const float* pre_state, const float* pre_shifts, int nprefix, void* Y, WsAlloc* ws) {
  FS_RANGE("causal segments");
  const int B = dm->B, H = dm->H, BH = B * H, L = dm->Lq;
  const int nch = (L + TILE - 1) / TILE, Lpad = nch * TILE;
  float* partial = ws->take<float>((size_t)BH * CF_MAX_SEG * TC_M * TC_NV);
  float* shifts = ws->take<float>((size_t)BH * CF_MAX_SEG * 2);
  float* crow = ws->take<float>((size_t)BH * Lpad);
  int per = 0;
  const int nseg = pick_segments(BH, nch, ctx->sm_count, &per);
  // key side: the per-key quadratic term of every key, and the totals of the segments that have a successor
  if (nseg > 1) {
    FS_TRY(fs_tc_key_side(ctx, K, V, dm, images, flags, per, nseg - 1, crow, partial, shifts));
  } else {
    FS_TRY(fs_tc_rowterm(ctx, K, dm, images, flags, Lpad, per, 1, crow));
  }
  int ntot = nseg - 1;
  if (nprefix > 0) {
    // one list per (batch, head): the totals that precede the sequence, then those of this call's segments
    ntot = nprefix + nseg - 1;
    float* all = ws->take<float>((size_t)BH * ntot * TC_M * TC_NV);
    float* allsh = ws->take<float>((size_t)BH * ntot * 2);
    const size_t one = (size_t)TC_M * TC_NV * sizeof(float), onesh = 2 * sizeof(float);
    FS_CUDA_OK(cudaMemcpy2DAsync(all, ntot * one, pre_state, nprefix * one, nprefix * one, BH, cudaMemcpyDeviceToDevice, ctx->stream));
    FS_CUDA_OK(cudaMemcpy2DAsync(allsh, ntot * onesh, pre_shifts, nprefix * onesh, nprefix * onesh, BH, cudaMemcpyDeviceToDevice, ctx->stream));
    if (nseg > 1) {
      FS_CUDA_OK(cudaMemcpy2DAsync(all + (size_t)nprefix * TC_M * TC_NV, ntot * one, partial, (nseg - 1) * one, (nseg - 1) * one, BH,
                                   cudaMemcpyDeviceToDevice, ctx->stream));
      FS_CUDA_OK(cudaMemcpy2DAsync(allsh + (size_t)nprefix * 2, ntot * onesh, shifts, (nseg - 1) * onesh, (nseg - 1) * onesh, BH,
                                   cudaMemcpyDeviceToDevice, ctx->stream));
    }
    partial = all;
    shifts = allsh;
  }
  CUtensorMap tmQ, tmK, tmV, tmY;
  FS_TRY(tchost::make_map_tokens(&tmQ, Q, fs_addr(dm->q_stride, H, L, dm->d), B, H, L, dm->d));
  FS_TRY(tchost::make_map_tokens(&tmK, K, fs_addr(dm->k_stride, H, L, dm->d), B, H, L, dm->d));
  FS_TRY(tchost::make_map_tokens(&tmV, V, fs_addr(dm->v_stride, H, L, dm->dv), B, H, L, dm->dv));
  FS_TRY(tchost::make_map_out(&tmY, Y, fs_addr(dm->y_stride, H, L, dm->dv), B, H, L, dm->dv));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_causal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CfSmem::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_CAUSAL);
  (void)fs_launch_chained(tc_causal_kernel, dim3(nseg, BH), dim3(TC_THREADS), CfSmem::TOTAL + 1024, ctx->stream,
      tmQ, tmK, tmV, tmY, images, crow, partial, shifts, ntot, nprefix, H, dm->pool, L, Lpad, per, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
