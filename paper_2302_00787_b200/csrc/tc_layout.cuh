// Sizes, shared-memory images and flag words shared by the tensor-core kernels and their prep.
#pragma once
#include <stdint.h>

namespace tcl {

constexpr int TC_D = 64, TC_M = 256, TC_DV = 64;
constexpr int TC_NV = 80;          // dv + 1 (the ones column of [V | 1]) padded to a multiple of 16
constexpr int TILE = 128;          // tokens per tile
// Warps 0-7 are the epilogue (two warpgroups); warps 8-11 form the producer warpgroup: warp 8 issues the TMA
// copies, warp 9 the MMAs (in the bidirectional kernels: the logits MMAs, while warps 10 and 11 issue the
// contractions of one feature half each; elsewhere 10-11 only take part in the register hand-over).
// The producer warpgroup shrinks to REGS_PRODUCER registers per thread so that the epilogue
// warpgroups can grow to REGS_EPILOGUE (384 threads x 168 at launch = 128 x 40 + 256 x 232).
constexpr int EPI_THREADS = 256, WARP_TMA = 8, WARP_MMA = 9, TC_THREADS = 384;
constexpr int REGS_PRODUCER = 40, REGS_EPILOGUE = 232;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TILE_BYTES = 16384;          // 128 rows x 128 bytes

// Per (group, side) operand image, already in the shared-memory layouts the MMAs read:
//   Wh    [256 features x 64]  K-major, 128-byte swizzle, fp16(log2e * qk_scale * W): rounded once to 11
//                              significant bits (the token tiles are converted to fp16 as well, so one
//                              operand serves where a bf16 value and its remainder would be needed)
//   Chi   [64 x 64]            K-major, 128-byte swizzle, bf16 of log2e * qk_scale^2 * C (row n, col k = C[k][n])
//   Clo   [64 x 64]            the bf16 remainder of the same matrix
//   a2    [256] fp32           2 log2e w_m^T A w_m: the factor 2^a2 of feature m (it appears once in
//                              phi(Q) and once in phi(K)) is applied to row m of S^T [V | 1] by the merge
constexpr uint32_t IMG_WH = 0, IMG_W_BYTES = 32768, IMG_CHI = 32768, IMG_C_BYTES = 8192, IMG_CLO = 40960, IMG_A2 = 49152,
                   IMG_A2_BYTES = 1024, IMG_BYTES = 50176;
// S^T [V | 1] transposed, fp16: 4 blocks of [80 rows x 64 features], 128-byte swizzle
constexpr uint32_t KVT_BLOCK_BYTES = 10240, KVT_BYTES = 40960;

// Two words per (group, side): [0] flag bits, [1] float bits of gamma (C = gamma I) in log2 units.
constexpr int FLAG_WORDS = 2;
constexpr int FLAG_C_DENSE = 1, FLAG_C_LO = 2;

// The keys' running shift is raised (and the accumulated state rescaled) when a tile's largest
// exponent exceeds it by more than this many powers of two: features stay below 2^57.7 = e^40.
constexpr float SHIFT_HEADROOM_LOG2 = 57.7f;

}  // namespace tcl
