// 64 x 64 x 16 shared-memory tile product on the fp32 CUDA cores, shared by the fp32 kernels.
#pragma once

namespace {

constexpr int TM = 64, TN = 64, TK = 16, NTH = 256;
// Row stride of a staged k-slice in floats: a multiple of 4, so that a thread's four rows (columns) are one
// 16-byte read.
constexpr int TLD = 68;

// Two stages: the next 16-wide k-slice is fetched into registers while the current one is multiplied, and
// stored into the other stage afterwards (one barrier per slice).
struct alignas(16) Tiles {
  float As[2][TK][TLD];
  float Bs[2][TK][TLD];
};

// Position of row (column) r inside a staged k-slice: the four rows ty, ty + 16, ty + 32, ty + 48 of a thread
// sit side by side.
__device__ __forceinline__ int tile_pos(int r) { return ((r & 15) << 2) | (r >> 4); }

// acc[i][j] += sum_k A(row = ty + 16 i, k) * B(k, col = tx + 16 j), k in [0, K).
// fa(row, k), fb(k, col) return 0 outside the operand.  AKF / BKF: k is the contiguous
// index of that operand in memory (decides which index runs fastest across threads).
// K must be the same for all threads of the block.
template <bool AKF, bool BKF, class FA, class FB>
__device__ __forceinline__ void tile_gemm(float (&acc)[4][4], int K, FA fa, FB fb, Tiles& sm) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  if (K <= 0) return;
  float ra[(TM * TK) / NTH], rb[(TN * TK) / NTH];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int u = 0; u < (TM * TK) / NTH; u++) {
      const int e = tid + u * NTH;
      const int k = AKF ? e % TK : e / TM, r = AKF ? e / TK : e % TM;
      ra[u] = (k0 + k < K) ? fa(r, k0 + k) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < (TN * TK) / NTH; u++) {
      const int e = tid + u * NTH;
      const int k = BKF ? e % TK : e / TN, c = BKF ? e / TK : e % TN;
      rb[u] = (k0 + k < K) ? fb(k0 + k, c) : 0.f;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int u = 0; u < (TM * TK) / NTH; u++) {
      const int e = tid + u * NTH;
      const int k = AKF ? e % TK : e / TM, r = AKF ? e / TK : e % TM;
      sm.As[buf][k][tile_pos(r)] = ra[u];
    }
#pragma unroll
    for (int u = 0; u < (TN * TK) / NTH; u++) {
      const int e = tid + u * NTH;
      const int k = BKF ? e % TK : e / TN, c = BKF ? e / TK : e % TN;
      sm.Bs[buf][k][tile_pos(c)] = rb[u];
    }
  };
  // (an earlier call has ended with a barrier after its last reads of either stage)
  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < K; k0 += TK) {
    const bool more = k0 + TK < K;
    if (more) fetch(k0 + TK);
#pragma unroll
    for (int k = 0; k < TK; k++) {
      const float4 a4 = *reinterpret_cast<const float4*>(&sm.As[buf][k][ty << 2]);
      const float4 b4 = *reinterpret_cast<const float4*>(&sm.Bs[buf][k][tx << 2]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) stash(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
}

}  // namespace
