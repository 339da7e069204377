// 64 x 64 x 16 shared-memory tile product on the fp32 CUDA cores, shared by the fp32 kernels.
#pragma once

namespace {

constexpr int TM = 64, TN = 64, TK = 16, NTH = 256;

struct Tiles {
  float As[TK][TM + 1];
  float Bs[TK][TN + 1];
};

// acc[i][j] += sum_k A(row = ty + 16 i, k) * B(k, col = tx + 16 j), k in [0, K).
// fa(row, k), fb(k, col) return 0 outside the operand.  AKF / BKF: k is the contiguous
// index of that operand in memory (decides which index runs fastest across threads).
template <bool AKF, bool BKF, class FA, class FB>
__device__ __forceinline__ void tile_gemm(float (&acc)[4][4], int K, FA fa, FB fb, Tiles& sm) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int u = 0; u < (TM * TK) / NTH; u++) {
      int e = tid + u * NTH;
      int k = AKF ? e % TK : e / TM, r = AKF ? e / TK : e % TM;
      sm.As[k][r] = (k0 + k < K) ? fa(r, k0 + k) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < (TN * TK) / NTH; u++) {
      int e = tid + u * NTH;
      int k = BKF ? e % TK : e / TN, c = BKF ? e / TK : e % TN;
      sm.Bs[k][c] = (k0 + k < K) ? fb(k0 + k, c) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < TK; k++) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; i++) { a[i] = sm.As[k][ty + 16 * i]; b[i] = sm.Bs[k][tx + 16 * i]; }
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

}  // namespace
