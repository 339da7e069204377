// Tensor-core path, bidirectional attention (Sections 2.1 / 2.2) for bf16, d = dv = 64, M = 256.
//
//   key side   (tc_kv_kernel):  per 128-key tile   logits = Y W2^T           (tcgen05, TMEM)
//                               phi = 2^(logits + c_j - s)  -> bf16 tile in shared memory
//                               KV^T += [V | 1]^T phi                        (tcgen05, TMEM)
//                               (c_j, the key's quadratic term, comes from tc_rowterm_kernel)
//   query side (tc_out_kernel): first the merge of the key-side partials of its (batch, head): common
//                               shift, sum, every feature's column scaled to order one (fp16), the
//                               scales' exponents g (with a2) kept for the logits; then per tile
//                               logits + g, phi = 2^(... - max of the half row) in fp16,
//                               [num | den] = phi KV per feature half, halves combined, Y = num / den
//
// The feature tiles never leave the SM.  One block = 8 epilogue warps (exponentials), one
// TMA producer warp and one MMA issuing warp; all exponents are kept in log2 units
// (W and C are pre-multiplied by log2 e), so a feature is one ex2 per element.  The per-feature
// term w^T A w is the same on the query and the key side; the key side leaves it out and the query
// side adds both shares, 2 log2e w_m^T A w_m, to its logits (inside g).
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"
#include "tc_layout.cuh"

using namespace tc;
using namespace tcl;

namespace {

constexpr int MAX_KEY_SPLIT = 64;    // splits of the key range of one (batch, head)
constexpr int PREFETCH_TILES = 4;   // tiles pulled into L2 ahead of the shared-memory ring

// ------------------------------------------------------------------------------------------
// key side
// ------------------------------------------------------------------------------------------
// The two halves of the feature range (128 features each) run as two pipelines of their own:
// four epilogue warps, a phi half tile, a pair of barriers, a running shift and a TMEM
// accumulator per half.  They only share the key / value tiles, the logits MMA and the MMA
// pipe itself, so while the tensor cores contract one half the other half's exponentials run.
// The accumulator of half h is acc_h = phi_h^T [V | 1] (128 feature lanes x 80 columns: the phi half
// tile is the M-side operand, [V | 1] the N = 80 side), so a contraction step costs 80 columns of the
// tensor pipe instead of 128, and every epilogue thread (= one feature) takes part when the state leaves.
constexpr int KV_KSTAGES = 3;       // key tiles in flight (TMA, conversion to fp16, logits MMA)
constexpr bool KV_TURNS = false;    // the two feature halves take turns at the exponentials
constexpr int KV_POLY_PAIRS = 2;    // of every four pairs of exponentials, this many run on the multiply-add pipe (measured: 1 and 3 are slower)
struct KvSmem {
  static constexpr uint32_t X0 = 0, V0 = KV_KSTAGES * TILE_BYTES, ONES = V0 + 2 * TILE_BYTES, W = ONES + TILE_BYTES,
                            PHI = W + IMG_W_BYTES, MISC = PHI + 4 * TILE_BYTES, TOTAL = MISC + 256;
};
static_assert(KvSmem::TOTAL + 1024 <= 232448, "shared memory budget");
static_assert(KvSmem::PHI % 1024 == 0 && KvSmem::W % 1024 == 0 && KvSmem::ONES % 1024 == 0, "swizzled tiles need 1024-byte alignment");

struct KvMisc {
  // key and value tiles have barriers of their own: a key tile is free again once the logits MMA that read it
  // has completed, long before the contraction that reads the value tile of the same stage
  uint64_t fullK[KV_KSTAGES], convK[KV_KSTAGES], emptyK[KV_KSTAGES], fullV[2], emptyV[2], logits_full, logits_free, phi_full[2],
      phi_free[2], const_bar;
  // turn[h]: half h may run its exponentials.  The halves take turns (each arrives on the other's barrier when its
  // exponentials are done), so one half has the exponential unit to itself while the other half's contraction
  // runs on the tensor cores and its warps load and scan the next tile's logits.
  uint64_t turn[2];
  uint32_t tmem_base;
  int abort_flag;
  int tile_max[2][4];     // per half: [0..2] rotating slots of the per-tile maximum
};
static_assert(sizeof(KvMisc) <= 256, "misc block");

constexpr uint32_t KV_COL_LOGITS = 0, KV_COL_ACC = 256;   // TMEM columns; half h accumulates at KV_COL_ACC + 80 h
constexpr int HALF_THREADS = EPI_THREADS / 2;

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_kv_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
             const uint8_t* __restrict__ images, const float* __restrict__ crow, int H, int pool, int L, int Lpad,
             int tiles_per_split, int nsplit, float* __restrict__ partial, float* __restrict__ shifts,
             int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  KvMisc* misc = reinterpret_cast<KvMisc*>(sm + KvSmem::MISC);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = split * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  const uint8_t* img = images + ((size_t)g * 2 + 1) * IMG_BYTES;        // side 2 (keys)
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < KV_KSTAGES; i++) {
      mbar_init(&misc->fullK[i], 1);
      mbar_init(&misc->convK[i], 2);
      mbar_init(&misc->emptyK[i], 1);
    }
    for (int i = 0; i < 2; i++) {
      mbar_init(&misc->fullV[i], 1);
      mbar_init(&misc->emptyV[i], 2);
      mbar_init(&misc->phi_full[i], HALF_THREADS / 32);
      mbar_init(&misc->phi_free[i], 1);
      mbar_init(&misc->turn[i], HALF_THREADS / 32);
      for (int j = 0; j < 4; j++) misc->tile_max[i][j] = f2ord(-INFINITY);
    }
    mbar_init(&misc->logits_full, 1);
    mbar_init(&misc->logits_free, EPI_THREADS / 32);
    mbar_init(&misc->const_bar, 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  // constant tile written by the block itself: the second 64-row block of [V | 1]^T, whose
  // first row is the 1 and whose other rows are zero
  for (int i = threadIdx.x; i < TILE_BYTES / 16; i += TC_THREADS) reinterpret_cast<uint4*>(sm + KvSmem::ONES)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if (threadIdx.x < TILE)
    *reinterpret_cast<__nv_bfloat16*>(sm + KvSmem::ONES + sw128_offset(threadIdx.x, 0)) = __float2bfloat16(1.f);
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
  // bf16 -> fp16 of key tile `it`, in place (16-byte pieces keep their swizzled positions): the logits then need one
  // fp16 image of W (11 significant bits) instead of a bf16 value and its remainder.  Half a tile per call, by the
  // converting warp (part 0) and the copying warp (part 1), which sit on different schedulers.
  auto convert_half = [&](int it, int part) -> bool {
    const int st = it % KV_KSTAGES;
    if (!__all_sync(0xffffffffu, mbar_wait(&misc->fullK[st], (it / KV_KSTAGES) & 1, abortp, status, false))) return false;
    uint4* xt = reinterpret_cast<uint4*>(sm + KvSmem::X0 + st * TILE_BYTES) + part * (int)(TILE_BYTES / 32);
#pragma unroll 4
    for (int i = 0; i < (int)(TILE_BYTES / 32) / 32; i++) {
      uint4 u = xt[lane + i * 32];
      u.x = pack_f16(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
      u.y = pack_f16(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
      u.z = pack_f16(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
      u.w = pack_f16(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
      xt[lane + i * 32] = u;
    }
    fence_proxy_async_smem();
    mbar_arrive_warp(&misc->convK[st], lane);
    return true;
  };
  if (warp == WARP_TMA) {
    // The whole warp walks the schedule; lane 0 issues the copies.
    if (lane == 0) {
      prefetch_tmap(&tmK);
      prefetch_tmap(&tmV);
      mbar_expect_tx(&misc->const_bar, IMG_W_BYTES);
      bulk_load(sm + KvSmem::W, img + IMG_WH, IMG_W_BYTES, &misc->const_bar);
      // tiles ahead of the shared-memory ring are pulled into L2
      for (int it = 0; it < min(ntiles, PREFETCH_TILES); it++) {
        tma_prefetch_4d(&tmK, 0, (tile0 + it) * TILE, h, b);
        tma_prefetch_4d(&tmV, 0, (tile0 + it) * TILE, h, b);
      }
    }
    // Key tile `it` is loaded as soon as the logits MMA of tile it - 3 has completed; the warp then converts its half
    // of key tile it - 1, which has landed meanwhile; the value tile follows one iteration behind (its stage is held
    // until the contraction of tile it - 2 has completed).  So the next tile's logits never wait for a value tile.
    int issuedK = 0, issuedV = 0;
    auto load_v = [&](int j) {
      const int sj = j & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->emptyV[sj], ((j >> 1) & 1) ^ 1, abortp, status))) return false;
      if (lane == 0) {
        mbar_expect_tx(&misc->fullV[sj], TILE_BYTES);
        tma_load_4d(sm + KvSmem::V0 + sj * TILE_BYTES, &tmV, &misc->fullV[sj], 0, (tile0 + j) * TILE, h, b);
      }
      issuedV = j + 1;
      return true;
    };
    bool okp = true;
    for (int it = 0; it < ntiles && okp; it++) {
      const int st = it % KV_KSTAGES;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->emptyK[st], ((it / KV_KSTAGES) & 1) ^ 1, abortp, status))) { okp = false; break; }
      if (lane == 0) {
        if (it + PREFETCH_TILES < ntiles) {
          tma_prefetch_4d(&tmK, 0, (tile0 + it + PREFETCH_TILES) * TILE, h, b);
          tma_prefetch_4d(&tmV, 0, (tile0 + it + PREFETCH_TILES) * TILE, h, b);
        }
        mbar_expect_tx(&misc->fullK[st], TILE_BYTES);
        tma_load_4d(sm + KvSmem::X0 + st * TILE_BYTES, &tmK, &misc->fullK[st], 0, (tile0 + it) * TILE, h, b);
      }
      issuedK = it + 1;
      if (it >= 1) {
        okp = convert_half(it - 1, 1);
        if (okp) okp = load_v(it - 1);
      }
    }
    if (okp && ntiles > 0) {
      okp = convert_half(ntiles - 1, 1);
      if (okp) load_v(ntiles - 1);
    }
    // no copy of this block may still be in flight when it exits
    if (lane == 0) {
      mbar_wait(&misc->const_bar, 0, abortp, status, false);
      for (int it = max(0, issuedK - KV_KSTAGES); it < issuedK; it++)
        mbar_wait(&misc->fullK[it % KV_KSTAGES], (it / KV_KSTAGES) & 1, abortp, status, false);
      for (int it = max(0, issuedV - 2); it < issuedV; it++) mbar_wait(&misc->fullV[it & 1], (it >> 1) & 1, abortp, status, false);
    }
  } else if (warp == WARP_MMA + 2) {
    for (int it = 0; it < ntiles; it++)
      if (!convert_half(it, 0)) break;
  } else if (warp == WARP_MMA) {
    // ---------------- logits MMAs: the whole warp walks the schedule (descriptor arithmetic and waits stay
    // warp-uniform), one elected lane issues
    constexpr uint32_t ID_LOGITS = idesc_f16(128, TC_M, 0, 0);
    const uint64_t dX0 = smem_desc(smem_u32(sm + KvSmem::X0), 16, 1024, SWZ_128B);
    const uint64_t dW = smem_desc(smem_u32(sm + KvSmem::W), 16, 1024, SWZ_128B);
    uint32_t xl = (uint32_t)dX0, wl = (uint32_t)dW;
    const uint32_t xh = (uint32_t)(dX0 >> 32), wh = (uint32_t)(dW >> 32);
    for (int it = 0; it < ntiles; it++) {
      const int st = it % KV_KSTAGES;
      opaque(xl); opaque(wl);
      if (it == 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->const_bar, 0, abortp, status))) break;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->convK[st], (it / KV_KSTAGES) & 1, abortp, status))) break;
      if (it > 0 && !__all_sync(0xffffffffu, mbar_wait(&misc->logits_free, (it - 1) & 1, abortp, status))) break;
      tcgen05_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < TC_D / 16; k++)
          mma_bf16_lh(tmem + KV_COL_LOGITS, xl + st * (TILE_BYTES / 16) + 2 * k, xh, wl + 2 * k, wh, ID_LOGITS, k > 0);
        mma_commit(&misc->logits_full);
        mma_commit(&misc->emptyK[st]);
      }
      __syncwarp();
    }
  } else {
    // ---------------- contractions of both feature halves (the halves take turns, half 0 first, so one static order
    // serves both): phi_h^T [V | 1]
    constexpr uint32_t ID_KV = idesc_bf16(128, TC_NV, 1, 1);
    const uint32_t sV0 = smem_u32(sm + KvSmem::V0), sOnes = smem_u32(sm + KvSmem::ONES);
    // phi half hh as the operand whose 128 features (M) are the contiguous index: two 64-feature blocks
    const uint64_t dPhi = smem_desc(smem_u32(sm + KvSmem::PHI), TILE_BYTES, 1024, SWZ_128B);
    // [V | 1] with the value index (N = 80) contiguous: block 0 = the V tile of the stage, block 1 = the ones
    // tile, of which the first 16 columns are read
    const uint64_t dVst0 = smem_desc(sV0, sOnes - sV0, 1024, SWZ_128B);
    const uint64_t dVst1 = smem_desc(sV0 + TILE_BYTES, sOnes - sV0 - TILE_BYTES, 1024, SWZ_128B);
    uint32_t pl = (uint32_t)dPhi, v0l = (uint32_t)dVst0, v1l = (uint32_t)dVst1;
    const uint32_t ph = (uint32_t)(dPhi >> 32), v0h = (uint32_t)(dVst0 >> 32), v1h = (uint32_t)(dVst1 >> 32);
    bool ok = true;
    for (int it = 0; ok && it < ntiles; it++) {
      const int st = it & 1;
      opaque(pl); opaque(v0l); opaque(v1l);
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->fullV[st], (it >> 1) & 1, abortp, status))) break;
      const uint32_t vl = st ? v1l : v0l, vh = st ? v1h : v0h;
      const uint32_t acc0 = it > 0 ? 1u : 0u;
#pragma unroll
      for (int hh = 0; hh < 2; hh++) {
        if (!__all_sync(0xffffffffu, mbar_wait(&misc->phi_full[hh], it & 1, abortp, status))) { ok = false; break; }
        tcgen05_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < TILE / 16; k++)
            mma_bf16_lh(tmem + KV_COL_ACC + hh * TC_NV, pl + hh * 2 * (TILE_BYTES / 16) + k * 128, ph, vl + k * 128, vh, ID_KV,
                        k > 0 ? 1u : acc0);
          mma_commit(&misc->phi_free[hh]);
          mma_commit(&misc->emptyV[st]);           // the value tile is free once both halves' contractions have completed
        }
        __syncwarp();
      }
    }
  }
  } else {
    regs_acquire<REGS_EPILOGUE>();
    // ---------------- epilogue warps: one key row per thread, the 128 features of its half.
    // The half keeps a running shift s.  Every tile's exact maximum is known before its exponentials
    // start; only when it exceeds s by more than the headroom (rare: the running maximum grows a
    // handful of times per sequence) does s move up, and the accumulated state with it.
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t acc_addr = lane_addr + KV_COL_ACC + hf * TC_NV;      // this thread's lane: feature hf * 128 + row
    int* tmax = misc->tile_max[hf];
    const float* cptr = crow + (size_t)bh * Lpad + (size_t)tile0 * TILE + row;
    float s = 0.f;
    float cj = ntiles > 0 ? cptr[0] : 0.f;
    bool alive = true;
    if (KV_TURNS && hf == 1) mbar_arrive_warp(&misc->turn[0], lane);     // half 0 goes first
    // accumulator of this half -> partial `slot` (the contraction that feeds it has completed)
    auto write_partial = [&](size_t slot) {
      __syncwarp();
      tcgen05_fence_after();
      // thread = feature m: its row of the accumulator is column m of the state [80][256]; a store instruction of
      // the warp covers 32 consecutive features of one state row (128 contiguous bytes).  Rows 65..79 are not written.
      float* out = partial + slot * TC_NV * TC_M + hf * 128 + row;
#pragma unroll
      for (int c = 0; c < 5; c++) {
        uint32_t a[16];
        tmem_ld16(acc_addr + c * 16, a);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j++) {
          if (c * 16 + j <= TC_DV) out[(size_t)(c * 16 + j) * TC_M] = __uint_as_float(a[j]);
        }
      }
      if (q == 0 && lane == 0) shifts[slot * 2 + hf] = s;
      tcgen05_fence_before();
    };
    for (int it = 0; it < ntiles && alive; it++) {
      FS_DBG(tile0 + it < total_tiles && (size_t)tile0 * TILE + (size_t)(it + 1) * TILE <= (size_t)Lpad, status);
      FS_DBG(KV_COL_ACC + hf * TC_NV + TC_NV <= TMEM_COLS && row < TILE, status);
      FS_DBG(KvSmem::PHI + hf * 2 * TILE_BYTES + TILE_BYTES + row * 128 + 128 <= KvSmem::MISC, status);
      const float cnext = it + 1 < ntiles ? cptr[(size_t)(it + 1) * TILE] : 0.f;     // in flight during this tile
      if (!mbar_wait(&misc->logits_full, it & 1, abortp, status, false)) { alive = false; break; }
      __syncwarp();
      tcgen05_fence_after();
      uint32_t v[128];
#pragma unroll
      for (int c = 0; c < 8; c++) {
        uint32_t t[16];
        tmem_ld16(lane_addr + KV_COL_LOGITS + hf * 128 + c * 16, t);
#pragma unroll
        for (int j = 0; j < 16; j++) v[c * 16 + j] = t[j];
      }
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->logits_free, lane);
      const bool valid = (tile0 + it) * TILE + row < L;
      // Exact maximum of this half of the tile, taken BEFORE the exponentials:
      // it overlaps the contraction of the previous tile, and nothing stands between the last exponential and
      // the arrival that starts this tile's contraction.
      float tm;
      {
        float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
          mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
          mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
          mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
        }
        const float hm = fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3]));
        float mx = valid ? hm + cj : -INFINITY;
        const int wm = __reduce_max_sync(0xffffffffu, f2ord(mx));       // one instruction for the warp's maximum
        if (lane == 0) atomicMax(&tmax[it % 3], wm);
        if (q == 0 && lane == 0) tmax[(it + 1) % 3] = f2ord(-INFINITY);           // next tile's slot; idle since tile it-2
        named_bar_sync(1 + hf, HALF_THREADS);
        tm = ord2f(tmax[it % 3]);
      }
      // the previous tile's contraction has read the phi half tile and updated the accumulator
      if (it > 0 && !mbar_wait(&misc->phi_free[hf], (it - 1) & 1, abortp, status, false)) { alive = false; break; }
      if (it == 0) {
        s = tm;                      // first tile: the shift is the exact maximum
      } else if (tm - s > SHIFT_HEADROOM_LOG2) {
        // rare (the running maximum grows a handful of times per sequence): the shift moves up to this tile's
        // maximum and the accumulated [V | 1]^T phi_h is brought along
        __syncwarp();
        tcgen05_fence_after();
        const float f = ex2(s - tm);
#pragma unroll
        for (int c = 0; c < 5; c++) {
          uint32_t a[16];
          tmem_ld16(acc_addr + c * 16, a);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; j++) a[j] = __float_as_uint(__uint_as_float(a[j]) * f);
          tmem_st16(acc_addr + c * 16, a);
        }
        tmem_wait_st();
        s = tm;
      }
      uint8_t* prow = sm + KvSmem::PHI + hf * 2 * TILE_BYTES + row * 128;
      const float rc = cj - s;
      if (KV_TURNS && !mbar_wait(&misc->turn[hf], it & 1, abortp, status, false)) { alive = false; break; }
#pragma unroll
      for (int c = 0; c < 16; c++) {
        uint32_t p[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
          uint32_t& e0 = v[c * 8 + 2 * j];
          uint32_t& e1 = v[c * 8 + 2 * j + 1];
          add2(e0, e1, rc, rc);
          if (j < KV_POLY_PAIRS) {
            exp2_poly2(e0, e1);
            p[j] = pack_bf16(__uint_as_float(e0), __uint_as_float(e1));
          } else {
            p[j] = pack_bf16(ex2(__uint_as_float(e0)), ex2(__uint_as_float(e1)));
          }
        }
        if (!valid) p[0] = p[1] = p[2] = p[3] = 0u;
        *reinterpret_cast<uint4*>(prow + (c >> 3) * TILE_BYTES + (((c & 7) ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
      }
      fence_proxy_async_smem();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->phi_full[hf], lane);
      if (KV_TURNS) mbar_arrive_warp(&misc->turn[hf ^ 1], lane);
      cj = cnext;
    }
    // write this split's partial phi_h^T [V | 1] (rows 0..64 of the state) and its shift
    if (alive && ntiles > 0 && mbar_wait(&misc->phi_free[hf], (ntiles - 1) & 1, abortp, status, false))
      write_partial((size_t)bh * nsplit + split);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------
// query side
// ------------------------------------------------------------------------------------------
// Every block first merges the key-side partials of its (batch, head) into shared memory: common
// shift, sum over the splits, and a scale of its own for every feature.  The query side contracts
// phi(Q) with this state in fp16, whose exponent range is narrow, and what a feature contributes to
// an output is phi(Q)_m times the size of column m of the state.  So every column m is brought to
// order one by a power of two 2^-e_m, and g_m = e_m + a2_m - max a2 (the per-feature term w^T A w
// of both sides rides along) joins the query logits BEFORE the row maximum is taken: a query
// feature near 1 is then one that matters, and what underflows in either operand is negligible by
// construction.  g joins the logits inside their MMA, as one more K step whose A operand is
// [1, 1, 0, ...] in every row (tensor memory) and whose B operand holds g as an fp16 value and its
// fp16 remainder.  The query tile is converted from bf16 to fp16 in shared memory (exact for |x| in
// [2^-14, 65504]), so the logits need one fp16 image of W instead of a bf16 value and its remainder.
constexpr int OUT_STAGES = 3;
constexpr int WARP_OUT_MMA2 = WARP_MMA + 1, WARP_OUT_CVT = WARP_MMA + 2;
// Of every four pairs of exponentials, this many run on the multiply-add pipe (exp2_poly2).
constexpr int OUT_POLY_PAIRS = 1;
struct OutSmem {
  // PHI also serves the merge (shifts and their factors) and, 2 KB per epilogue warp inside the rows that warp
  // itself writes next, the output rows on their way out
  static constexpr uint32_t X0 = 0, WH = OUT_STAGES * TILE_BYTES, PHI = WH + IMG_W_BYTES, KVT = PHI + 4 * TILE_BYTES,
                            ROWMAX = KVT + KVT_BYTES,
                            // g as an MMA operand: [256 features x 16] fp16, no swizzle (the two 16-byte K pieces of a
                            // row 128 bytes apart, 8-row groups 256 bytes apart)
                            GOP = ROWMAX + 2 * 2 * TILE * 4, GOP_BYTES = TC_M * 32, MISC = GOP + GOP_BYTES, TOTAL = MISC + 256;
};
static_assert(OutSmem::PHI % 1024 == 0 && OutSmem::KVT % 1024 == 0 && OutSmem::WH % 1024 == 0, "alignment");
static_assert(OutSmem::TOTAL + 1024 <= 232448, "shared memory budget");

struct OutMisc {
  // full: the tile has landed; conv: it has been converted to fp16; phi_full[f]: the 64-feature block f of the phi
  // tile is written (the four warps of its half arrive); g_ready: the merge has written its operands
  uint64_t full[OUT_STAGES], conv[OUT_STAGES], empty[OUT_STAGES], logits_full, logits_free, phi_full[TC_M / 64], phi_free, const_bar,
      g_ready;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(OutMisc) <= 256, "misc block");
// TMEM columns: logits, then [num | den], then the A operand of the g step
constexpr uint32_t OUT_COL_LOGITS = 0, OUT_COL_OUT = 256, OUT_COL_ONE = 496;

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_out_kernel(const __grid_constant__ CUtensorMap tmQ, const uint8_t* __restrict__ images,
              const float* __restrict__ partial, const float* __restrict__ shifts, int nsplit, int H, int pool, int L,
              int tiles_per_split,
              __nv_bfloat16* __restrict__ Y, TensorAddr ay, int* __restrict__ status) {
  fs_grid_dependency_wait();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  OutMisc* misc = reinterpret_cast<OutMisc*>(sm + OutSmem::MISC);
  float* rowmax = reinterpret_cast<float*>(sm + OutSmem::ROWMAX);   // [tile % 2][half][row]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = pool == FSHARP_POOL_PER_BH ? bh : h;
  const int total_tiles = (L + TILE - 1) / TILE;
  const int tile0 = split * tiles_per_split;
  const int ntiles = min(tiles_per_split, total_tiles - tile0);
  const uint8_t* img = images + ((size_t)g * 2 + 0) * IMG_BYTES;        // side 1 (queries)
  volatile int* abortp = &misc->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < OUT_STAGES; i++) { mbar_init(&misc->full[i], 1); mbar_init(&misc->conv[i], 2); mbar_init(&misc->empty[i], 1); }
    mbar_init(&misc->logits_full, 1);
    mbar_init(&misc->logits_free, EPI_THREADS / 32);
    for (int i = 0; i < TC_M / 64; i++) mbar_init(&misc->phi_full[i], EPI_THREADS / 64);
    mbar_init(&misc->phi_free, 1);
    mbar_init(&misc->const_bar, 1);
    mbar_init(&misc->g_ready, EPI_THREADS / 32);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
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
  // bf16 -> fp16 of query tile `it`, in place (16-byte pieces keep their swizzled positions): half a tile per call,
  // by the converting warp (part 0) and the copying warp (part 1), which sit on different schedulers
  auto convert_half = [&](int it, int part) -> bool {
    const int st = it % OUT_STAGES;
    if (!__all_sync(0xffffffffu, mbar_wait(&misc->full[st], (it / OUT_STAGES) & 1, abortp, status, false))) return false;
    uint4* xt = reinterpret_cast<uint4*>(sm + OutSmem::X0 + st * TILE_BYTES) + part * (int)(TILE_BYTES / 32);
#pragma unroll 4
    for (int i = 0; i < (int)(TILE_BYTES / 32) / 32; i++) {
      uint4 u = xt[lane + i * 32];
      u.x = pack_f16(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
      u.y = pack_f16(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
      u.z = pack_f16(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
      u.w = pack_f16(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
      xt[lane + i * 32] = u;
    }
    fence_proxy_async_smem();
    mbar_arrive_warp(&misc->conv[st], lane);
    return true;
  };
  if (warp == WARP_TMA) {
    // The whole warp walks the schedule; lane 0 issues the copies.  After the copy of tile it has been issued the
    // warp converts its half of tile it - 1, which has landed meanwhile.
    if (lane == 0) {
      prefetch_tmap(&tmQ);
      mbar_expect_tx(&misc->const_bar, IMG_W_BYTES);
      bulk_load(sm + OutSmem::WH, img + IMG_WH, IMG_W_BYTES, &misc->const_bar);
      for (int it = 0; it < min(ntiles, PREFETCH_TILES); it++) tma_prefetch_4d(&tmQ, 0, (tile0 + it) * TILE, h, b);
    }
    int issued = 0;
    bool okp = true;
    for (int it = 0; it < ntiles; it++) {
      const int st = it % OUT_STAGES;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->empty[st], ((it / OUT_STAGES) & 1) ^ 1, abortp, status))) { okp = false; break; }
      if (lane == 0) {
        if (it + PREFETCH_TILES < ntiles) tma_prefetch_4d(&tmQ, 0, (tile0 + it + PREFETCH_TILES) * TILE, h, b);
        mbar_expect_tx(&misc->full[st], TILE_BYTES);
        tma_load_4d(sm + OutSmem::X0 + st * TILE_BYTES, &tmQ, &misc->full[st], 0, (tile0 + it) * TILE, h, b);
      }
      issued = it + 1;
      if (it > 0 && !convert_half(it - 1, 1)) { okp = false; break; }
    }
    if (okp && ntiles > 0) convert_half(ntiles - 1, 1);
    // no copy of this block may still be in flight when it exits
    if (lane == 0) {
      mbar_wait(&misc->const_bar, 0, abortp, status, false);
      for (int it = max(0, issued - OUT_STAGES); it < issued; it++)
        mbar_wait(&misc->full[it % OUT_STAGES], (it / OUT_STAGES) & 1, abortp, status, false);
    }
  } else if (warp == WARP_OUT_CVT) {
    for (int it = 0; it < ntiles; it++)
      if (!convert_half(it, 0)) break;
  } else if (warp == WARP_MMA) {
    // ---------------- logits MMAs: the whole warp walks the schedule, one elected lane issues
    constexpr uint32_t ID_LOGITS = idesc_f16(128, TC_M, 0, 0);
    const uint64_t dX0 = smem_desc(smem_u32(sm + OutSmem::X0), 16, 1024, SWZ_128B);
    const uint64_t dW = smem_desc(smem_u32(sm + OutSmem::WH), 16, 1024, SWZ_128B);
    const uint64_t dG = smem_desc(smem_u32(sm + OutSmem::GOP), 128, 256, SWZ_NONE);
    uint32_t xl = (uint32_t)dX0, wl = (uint32_t)dW, gl = (uint32_t)dG;
    const uint32_t xh = (uint32_t)(dX0 >> 32), wh = (uint32_t)(dW >> 32), gh = (uint32_t)(dG >> 32);
    auto issue_logits = [&](int st) {
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < TC_D / 16; k++)
          mma_bf16_lh(tmem + OUT_COL_LOGITS, xl + st * (TILE_BYTES / 16) + 2 * k, xh, wl + 2 * k, wh, ID_LOGITS, k > 0);
        mma_bf16_ta_lh(tmem + OUT_COL_LOGITS, tmem + OUT_COL_ONE, gl, gh, ID_LOGITS, 1u);
        mma_commit(&misc->logits_full);
        mma_commit(&misc->empty[st]);
      }
      __syncwarp();
    };
#define OUT_WAIT(bar, par) if (!__all_sync(0xffffffffu, mbar_wait((bar), (par), abortp, status))) break
    for (int it = 0; it < ntiles; it++) {
      const int st = it % OUT_STAGES;
      opaque(xl); opaque(wl); opaque(gl);
      if (it == 0) {
        OUT_WAIT(&misc->const_bar, 0);
        OUT_WAIT(&misc->g_ready, 0);
      }
      OUT_WAIT(&misc->conv[st], (it / OUT_STAGES) & 1);
      if (it > 0) OUT_WAIT(&misc->logits_free, (it - 1) & 1);
      // (Every barrier this warp waits on is one whose next phase cannot complete before this warp has moved on: a
      // wait by parity on a barrier that may run two phases ahead of its waiter would never end.  phi_free is such
      // a barrier for this warp, so the logits are not ordered behind the contraction of an earlier tile.)
      tcgen05_fence_after();
      issue_logits(st);
    }
#undef OUT_WAIT
  } else if (warp == WARP_OUT_MMA2) {
    // ---------------- contraction: every 64-feature block of phi is contracted as soon as it is written, first
    // blocks of both halves first, so only the last block's MMAs are left when the exponentials end.  One
    // accumulator [num | den] for all 256 features (the two threads of a row agree on the row's shift).
    constexpr uint32_t ID_OUT = idesc_f16(128, TC_NV, 0, 0);      // fp16: phi(Q) <= 1 and a state of order one per feature
    const uint64_t dPhi = smem_desc(smem_u32(sm + OutSmem::PHI), 16, 1024, SWZ_128B);
    const uint64_t dKvt = smem_desc(smem_u32(sm + OutSmem::KVT), 16, 1024, SWZ_128B);
    uint32_t pl = (uint32_t)dPhi, kl = (uint32_t)dKvt;
    const uint32_t ph = (uint32_t)(dPhi >> 32), kh = (uint32_t)(dKvt >> 32);
    bool ok = true;
    for (int it = 0; ok && it < ntiles; it++) {
      opaque(pl); opaque(kl);
      // An epilogue thread arrives on its half's first block only after it has read the previous tile's output
      // row, so the accumulator may be overwritten once the first blocks of BOTH halves are in.
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->phi_full[0], it & 1, abortp, status))) break;
      if (!__all_sync(0xffffffffu, mbar_wait(&misc->phi_full[2], it & 1, abortp, status))) break;
#pragma unroll
      for (int o = 0; o < TC_M / 64; o++) {
        const int fb = ((o & 1) << 1) | (o >> 1);      // 0, 2, 1, 3
        if (o >= 2 && !__all_sync(0xffffffffu, mbar_wait(&misc->phi_full[fb], it & 1, abortp, status))) { ok = false; break; }
        tcgen05_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 4; k++)
            mma_bf16_lh(tmem + OUT_COL_OUT, pl + fb * (TILE_BYTES / 16) + 2 * k, ph, kl + fb * (KVT_BLOCK_BYTES / 16) + 2 * k, kh, ID_OUT,
                        (o > 0 || k > 0) ? 1u : 0u);
          if (o == TC_M / 64 - 1) mma_commit(&misc->phi_free);
        }
        __syncwarp();
      }
    }
  }
  } else {
    regs_acquire<REGS_EPILOGUE>();
    // ---------------- epilogue warps: one query row per thread, 128 of the 256 features.
    // The two threads of a row exchange the maxima of their half rows (through shared memory, the
    // two warps of a row quarter meeting at a barrier of their own), so the row has one shift and
    // both halves are contracted into one accumulator, read when the next tile's maxima are known.
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    __nv_bfloat16* Yb = Y + b * ay.sb + h * ay.sh;
    bool alive = true;
    {
      // merge (see above); thread = feature m, whose half (m / 128) is also the thread's half below, so the
      // arrivals that release a 64-feature block to the MMA warp cover the writers of that block of the state
      const int m = threadIdx.x, hh = m >> 7;
      float* sft = reinterpret_cast<float*>(sm + OutSmem::PHI);          // shifts, then their factors (the phi tile is idle)
      float* red = sft + 2 * MAX_KEY_SPLIT;
      const float a2m = reinterpret_cast<const float*>(img + IMG_A2)[m];
      float wmx = a2m;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) wmx = fmaxf(wmx, __shfl_xor_sync(0xffffffffu, wmx, o));
      if (lane == 0) red[warp] = wmx;
      if (m < 2 * nsplit) sft[m] = shifts[(size_t)bh * nsplit * 2 + m];
      named_bar_sync(1, EPI_THREADS);
      float a2max = red[0], smax = -INFINITY;
#pragma unroll
      for (int i = 1; i < EPI_THREADS / 32; i++) a2max = fmaxf(a2max, red[i]);
      for (int p = 0; p < 2 * nsplit; p++) smax = fmaxf(smax, sft[p]);
      named_bar_sync(1, EPI_THREADS);
      if (m < 2 * nsplit) sft[m] = exp2f(sft[m] - smax);
      named_bar_sync(1, EPI_THREADS);
      const float* base = partial + (size_t)bh * nsplit * TC_NV * TC_M + m;
      float val[TC_DV + 1];
#pragma unroll
      for (int n = 0; n <= TC_DV; n++) val[n] = 0.f;
      for (int p = 0; p < nsplit; p++) {        // 65 independent loads in flight per split
        const float f = sft[2 * p + hh];
        const float* bp = base + (size_t)p * TC_NV * TC_M;
#pragma unroll
        for (int n = 0; n <= TC_DV; n++) val[n] = fmaf(bp[n * TC_M], f, val[n]);
      }
      float amax = 0.f;
#pragma unroll
      for (int n = 0; n <= TC_DV; n++) amax = fmaxf(amax, fabsf(val[n]));
      int ex = 0;
      if (amax > 0.f && isfinite(amax)) frexpf(amax, &ex);          // amax = f 2^ex, f in [1/2, 1)
      const float sc = exp2f((float)-ex);
      uint8_t* kcol = sm + OutSmem::KVT + (m >> 6) * KVT_BLOCK_BYTES;
#pragma unroll
      for (int n = 0; n < TC_NV; n++)
        *reinterpret_cast<__half*>(kcol + sw128_offset(n, m & 63)) = __float2half_rn(n <= TC_DV ? val[n <= TC_DV ? n : 0] * sc : 0.f);
      // g_m as an fp16 value and its fp16 remainder: K elements 0 and 1 of row m of the operand
      {
        const float gm = (float)ex + a2m - a2max;
        const __half hi = __float2half_rn(gm), lo = __float2half_rn(gm - __half2float(hi));
        uint8_t* rowp = sm + OutSmem::GOP + (m >> 3) * 256 + (m & 7) * 16;
        *reinterpret_cast<uint4*>(rowp) = make_uint4((uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16), 0, 0, 0);
        *reinterpret_cast<uint4*>(rowp + 128) = make_uint4(0, 0, 0, 0);
      }
      // the A operand of that step: 1, 1, 0, ... (fp16) in every row
      if (hf == 0) {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %2, %2, %2, %2, %2, %2};" ::"r"(lane_addr + OUT_COL_ONE),
                     "r"(0x3C003C00u), "r"(0u) : "memory");
        tmem_wait_st();
      }
      named_bar_sync(1, EPI_THREADS);          // the shifts' factors have been read: the phi tile may be written
      fence_proxy_async_smem();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->g_ready, lane);
    }
    // Y rows of tile j (its contraction has completed): 32 of the 64 columns per thread
    auto write_out = [&](int j) {
      __syncwarp();
      tcgen05_fence_after();
      uint32_t n0[32], d0[16];
      const uint32_t base = lane_addr + OUT_COL_OUT;
      tmem_ld16(base + hf * 32, reinterpret_cast<uint32_t(&)[16]>(n0[0]));
      tmem_ld16(base + hf * 32 + 16, reinterpret_cast<uint32_t(&)[16]>(n0[16]));
      tmem_ld16(base + TC_DV, d0);
      tmem_wait_ld();
      const int64_t r0 = (int64_t)(tile0 + j) * TILE + q * 32;       // first row of this warp
      const float den = __uint_as_float(d0[0]);
      if (r0 + lane < L && (!(den > 0.f) || !isfinite(den))) atomicExch(status, FSHARP_E_NONFINITE);
      float inv;                       // outputs are rounded to bf16: the approximate reciprocal (1 ulp) is exact enough
      asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(den));
      // The thread's 64 bytes go through shared memory so that a store instruction of the warp covers 8 rows x 64
      // contiguous bytes.  The staging area lies inside the rows of the phi tile that this warp itself writes next.
      uint8_t* stg = sm + OutSmem::PHI + hf * 2 * TILE_BYTES + q * 4096;
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
        const int rr = (lane >> 2) + 8 * i, c = lane & 3;
        const uint4 val = *reinterpret_cast<const uint4*>(stg + rr * 64 + ((c ^ ((rr >> 1) & 3)) << 4));
        if (r0 + rr < L) *reinterpret_cast<uint4*>(Yb + (r0 + rr) * ay.sl + hf * 32 + c * 8) = val;
      }
      __syncwarp();
    };
    for (int it = 0; it < ntiles && alive; it++) {
      FS_DBG(tile0 + it < total_tiles && OUT_COL_OUT + TC_NV <= OUT_COL_ONE && OUT_COL_ONE + 8 <= TMEM_COLS, status);
      FS_DBG(OutSmem::PHI + hf * 2 * TILE_BYTES + TILE_BYTES + row * 128 + 128 <= OutSmem::KVT && row < TILE, status);
      if (!mbar_wait(&misc->logits_full, it & 1, abortp, status, false)) { alive = false; break; }
      __syncwarp();
      tcgen05_fence_after();
      uint32_t v[128];
#pragma unroll
      for (int c = 0; c < 8; c++) tmem_ld16(lane_addr + OUT_COL_LOGITS + hf * 128 + c * 16, reinterpret_cast<uint32_t(&)[16]>(v[c * 16]));
      tmem_wait_ld();
      tcgen05_fence_before();
      mbar_arrive_warp(&misc->logits_free, lane);
      // (the exponent of feature m's column of the state and w^T A w of both sides are already in the logits)
      float mxp[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < 128; i += 8) {
        mxp[0] = max3(mxp[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
        mxp[1] = max3(mxp[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
        mxp[2] = max3(mxp[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
        mxp[3] = max3(mxp[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
      }
      float mx = fmaxf(fmaxf(mxp[0], mxp[1]), fmaxf(mxp[2], mxp[3]));
      // the other half of the row: its thread sits in warp q of the other warpgroup (slots rotate over two tiles:
      // a slot is rewritten only after both warps have passed the next tile's barrier)
      rowmax[(it & 1) * 2 * TILE + hf * TILE + row] = mx;
      named_bar_sync(2 + q, 64);
      mx = fmaxf(mx, rowmax[(it & 1) * 2 * TILE + (hf ^ 1) * TILE + row]);
      if (it > 0) {
        // contraction of the previous tile done: its phi tile and its outputs are ours again
        if (!mbar_wait(&misc->phi_free, (it - 1) & 1, abortp, status, false)) { alive = false; break; }
        write_out(it - 1);
      }
      uint8_t* prow = sm + OutSmem::PHI + hf * 2 * TILE_BYTES + row * 128;
#pragma unroll
      for (int c = 0; c < 16; c++) {
        uint32_t p[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
          uint32_t& e0 = v[c * 8 + 2 * j];
          uint32_t& e1 = v[c * 8 + 2 * j + 1];
          add2(e0, e1, -mx, -mx);
          if (j < OUT_POLY_PAIRS) {
            exp2_poly2(e0, e1);
            p[j] = pack_f16(__uint_as_float(e0), __uint_as_float(e1));
          } else {
            p[j] = pack_f16(ex2(__uint_as_float(e0)), ex2(__uint_as_float(e1)));
          }
        }
        *reinterpret_cast<uint4*>(prow + (c >> 3) * TILE_BYTES + (((c & 7) ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
        if ((c & 7) == 7) {                     // a 64-feature block of this half is complete
          fence_proxy_async_smem();
          tcgen05_fence_before();
          mbar_arrive_warp(&misc->phi_full[hf * 2 + (c >> 3)], lane);
          // a real branch after the hand-over: the instruction scheduler would otherwise move the (side-effect-free)
          // exponentials of the second block ahead of it
          if (*abortp) { alive = false; break; }
        }
      }
    }
    if (alive && ntiles > 0 && mbar_wait(&misc->phi_free, (ntiles - 1) & 1, abortp, status, false)) write_out(ntiles - 1);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// Splits `tiles` tiles of each of `units` independent units into blocks of equal tile count so that
// (waves of blocks on `sms` SMs) x (tiles per block + fixed overhead) is smallest; ties go to fewer blocks.
int pick_split(int units, int tiles, int sms, int max_split, int* tiles_per_split) {
  int best = 1, best_cost = 0x7fffffff, best_tps = tiles;
  for (int ns = 1; ns <= tiles && ns <= max_split; ns++) {
    int tps = (tiles + ns - 1) / ns;
    int real = (tiles + tps - 1) / tps;
    if (real != ns) continue;
    long long blocks = (long long)units * ns;
    int waves = (int)((blocks + sms - 1) / sms);
    int cost = waves * (tps + 4);    // a block's fill and drain cost about as much as four tiles
    if (cost < best_cost) { best_cost = cost; best = ns; best_tps = tps; }
  }
  *tiles_per_split = best_tps;
  return best;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
namespace tchost {
int make_map_tokens(CUtensorMap* map, const void* base, TensorAddr a, int B, int H, int L, int inner);
}  // namespace tchost
int fs_tc_rowterm(fsharp_ctx* ctx, const void* K, const fsharp_dims* dm, const uint8_t* images, const int* flags, int Lpad,
                  int tiles_per_split, int nsplit, float* crow);
size_t fs_tc_bidir_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_bidir(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                const int* flags, void* Y, WsAlloc* ws);
int fs_tc_key_side(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                   const int* flags, int tiles_per_split, int nsplit, float* crow, float* partial, float* shifts);
int fs_tc_query_side(fsharp_ctx* ctx, const void* Q, const fsharp_dims* dm, const uint8_t* images, const float* partial,
                     const float* shifts, int nsplit, void* Y);
int fs_tc_key_state_splits(const fsharp_ctx* ctx, const fsharp_dims* dm, int* tiles_per_split);
size_t fs_tc_key_state_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_key_state(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                    const int* flags, float* state, float* shifts, WsAlloc* ws);

// The key range of a key-state call is cut into at most this many pieces (each is one [80][256] block to hand on).
constexpr int MAX_STATE_SPLIT = 8;

int fs_tc_key_state_splits(const fsharp_ctx* ctx, const fsharp_dims* dm, int* tiles_per_split) {
  int tps = 0;
  const int ns = pick_split(dm->B * dm->H, (dm->Lk + TILE - 1) / TILE, ctx->sm_count, MAX_STATE_SPLIT, &tps);
  if (tiles_per_split) *tiles_per_split = tps;
  return ns;
}

size_t fs_tc_key_state_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm) {
  (void)ctx;
  const size_t BH = (size_t)dm->B * dm->H, G = fs_groups(dm);
  return ws_round(G * 2 * IMG_BYTES) + ws_round(G * 2 * FLAG_WORDS * 4 + 64) + ws_round(BH * MAX_STATE_SPLIT * 2 * 4) +
         ws_round(BH * (size_t)((dm->Lk + TILE - 1) / TILE) * TILE * 4);
}

// Key side alone, over all keys of the call: state [B*H][ns][80][256], shifts [B*H][ns][2] with ns = fs_tc_key_state_splits.
int fs_tc_key_state(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                    const int* flags, float* state, float* shifts, WsAlloc* ws) {
  const int BH = dm->B * dm->H;
  int tps = 0;
  const int ns = fs_tc_key_state_splits(ctx, dm, &tps);
  float* crow = ws->take<float>((size_t)BH * ((dm->Lk + TILE - 1) / TILE) * TILE);
  return fs_tc_key_side(ctx, K, V, dm, images, flags, tps, ns, crow, state, shifts);
}

size_t fs_tc_bidir_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm) {
  const size_t BH = (size_t)dm->B * dm->H;
  const size_t G = fs_groups(dm);
  return ws_round(G * 2 * IMG_BYTES) + ws_round(G * 2 * FLAG_WORDS * 4 + 64) +
         ws_round(BH * MAX_KEY_SPLIT * TC_M * TC_NV * 4) + 2 * ws_round(BH * MAX_KEY_SPLIT * 2 * 4) +
         ws_round(BH * (size_t)((dm->Lk + TILE - 1) / TILE) * TILE * 4) +
         ws_round(BH * TC_NV * TC_M * 2) + ws_round(BH * TC_M * 4);
}

// Key side: the per-key quadratic term, then the feature / contraction kernel.  crow: [B*H][Lpad] floats,
// Lpad = ceil(Lk / 128) * 128; partial: [B*H][nsplit][80][256] floats; shifts: [B*H][nsplit][2].
// The quadratic term covers every key; the feature / contraction kernel covers the
// first nsplit * tiles_per_split tiles (the causal path asks for the segments that have a successor only).
int fs_tc_key_side(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                   const int* flags, int tiles_per_split, int nsplit, float* crow, float* partial, float* shifts) {
  FS_RANGE("key side");
  const int B = dm->B, H = dm->H, Lk = dm->Lk;
  const int Lpad = (Lk + TILE - 1) / TILE * TILE;
  FS_TRY(fs_tc_rowterm(ctx, K, dm, images, flags, Lpad, tiles_per_split, nsplit, crow));
  CUtensorMap tmK, tmV;
  FS_TRY(tchost::make_map_tokens(&tmK, K, fs_addr(dm->k_stride, H, Lk, dm->d), B, H, Lk, dm->d));
  FS_TRY(tchost::make_map_tokens(&tmV, V, fs_addr(dm->v_stride, H, Lk, dm->dv), B, H, Lk, dm->dv));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)KvSmem::TOTAL + 1024));
  FS_TIME_BEGIN(ctx, FS_K_TC_KV);
  (void)fs_launch_chained(tc_kv_kernel, dim3(nsplit, B * H), dim3(TC_THREADS), KvSmem::TOTAL + 1024, ctx->stream,
      tmK, tmV, images, crow, H, dm->pool, Lk, Lpad, tiles_per_split, nsplit, partial, shifts, ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}

int fs_tc_bidir(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                const int* flags, void* Y, WsAlloc* ws) {
  const int B = dm->B, H = dm->H, BH = B * H, Lq = dm->Lq, Lk = dm->Lk;

  // key side: the split of the key range that minimises (waves of blocks) x (tiles per block)
  const int ktiles = (Lk + TILE - 1) / TILE;
  int tps = 0;
  int nsplit = pick_split(BH, ktiles, ctx->sm_count, MAX_KEY_SPLIT, &tps);
  float* partial = ws->take<float>((size_t)BH * MAX_KEY_SPLIT * TC_M * TC_NV);
  float* shifts = ws->take<float>((size_t)BH * MAX_KEY_SPLIT * 2);
  const int Lpad = ktiles * TILE;
  float* crow = ws->take<float>((size_t)BH * Lpad);
  FS_TRY(fs_tc_key_side(ctx, K, V, dm, images, flags, tps, nsplit, crow, partial, shifts));

  return fs_tc_query_side(ctx, Q, dm, images, partial, shifts, nsplit, Y);
}

// Query side alone: partial [B*H][nsplit][80][256], shifts [B*H][nsplit][2] are key-side sums of disjoint key ranges
// (of this call's key side, or handed in by the caller).
int fs_tc_query_side(fsharp_ctx* ctx, const void* Q, const fsharp_dims* dm, const uint8_t* images, const float* partial,
                     const float* shifts, int nsplit, void* Y) {
  FS_RANGE("query side");
  const int B = dm->B, H = dm->H, BH = B * H, Lq = dm->Lq;
  if (nsplit < 1 || nsplit > MAX_KEY_SPLIT) return FSHARP_E_LIMIT;
  CUtensorMap tmQ;
  FS_TRY(tchost::make_map_tokens(&tmQ, Q, fs_addr(dm->q_stride, H, Lq, dm->d), B, H, Lq, dm->d));
  FS_CUDA_OK(cudaFuncSetAttribute(tc_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)OutSmem::TOTAL + 1024));
  const int qtiles = (Lq + TILE - 1) / TILE;
  int qtps = 0;
  int qsplit = pick_split(BH, qtiles, ctx->sm_count, 1 << 20, &qtps);
  FS_TIME_BEGIN(ctx, FS_K_TC_OUT);
  (void)fs_launch_chained(tc_out_kernel, dim3(qsplit, BH), dim3(TC_THREADS), OutSmem::TOTAL + 1024, ctx->stream,
      tmQ, images, partial, shifts, nsplit, H, dm->pool, Lq, qtps, (__nv_bfloat16*)Y, fs_addr(dm->y_stride, H, Lq, dm->dv), ctx->d_status);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
