// Backward pass of featurize + attend (Section 5.3 trains Transformers through the attention of
// Section 2.2): given dY, the gradients with respect to Q, K and V, the random features Omega and
// the fitted parameters being constants.  fp32 CUDA-core kernels.
//
// With P = phi(Q) (L x M), S = phi(K), [num | den] = P KV_i, KV_i = sum_{j <= i} S_j [V_j | 1]^T
// (all j when bidirectional), Y = num / den:
//   G_i   = [dY_i / den_i | -(dY_i . Y_i) / den_i]                                (L x (dv + 1))
//   dP_i  = G_i KV_i^T,                     dlogP = dP * P
//   R_j   = sum_{i >= j} P_i G_i^T          (M x (dv + 1); all i when bidirectional)
//   dS_j  = [V_j | 1] R_j^T,                dlogS = dS * S,      dV_j = S_j R_j[:, :dv]
//   logit = a_m + w_m^T B x + x^T C x:      dx = dlog W + rowsum(dlog) (C + C^T) x,   dQ = qk_scale dx
// Causal sequences go chunk by chunk: KV_i = (sum over earlier chunks) + the masked part inside the
// chunk, R_j = (sum over later chunks) + the masked part, with tril(P_c S_c^T) and tril(G_c [V_c | 1]^T)
// formed per chunk.  The feature kernels' shifts (per query row, per (batch, head) for the keys)
// cancel in every product above exactly as they do in Y.
#include "common.cuh"
#include "simt_tile.cuh"

namespace {

struct BwdDims {
  int H, Lq, Lk, d, dv, M, N, causal, C, nch;
};

// ---- out[z][m][n] (+)= sum_{j in slice} F[j][m] * R[j][n] --------------------------------------
// FROM_G = false: F = phi(K), R = [V | 1] (typed);  true: F = phi(Q), R = G (fp32, row stride N).
template <typename T, bool FROM_G>
__global__ void __launch_bounds__(NTH)
bwd_state_kernel(const float* __restrict__ F, const T* __restrict__ V, TensorAddr av, const float* __restrict__ G,
                 BwdDims q, int L, int slice_len, int nslices, int per_slice_out, float* __restrict__ out) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z / nslices, sl = blockIdx.z % nslices;
  const int b = bh / q.H, h = bh % q.H;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int j0 = sl * slice_len, j1 = min(L, j0 + slice_len);
  if (j0 >= j1) return;
  const int M = q.M, N = q.N, dv = q.dv;
  const float* Fb = F + (int64_t)bh * L * M;
  const T* Vb = V + b * av.sb + h * av.sh;
  const float* Gb = G + (int64_t)bh * L * N;
  float acc[4][4] = {};
  tile_gemm<false, false>(
      acc, j1 - j0, [&](int r, int k) { return (m0 + r < M) ? Fb[(int64_t)(j0 + k) * M + m0 + r] : 0.f; },
      [&](int k, int c) {
        const int n = n0 + c;
        if (FROM_G) return n < N ? Gb[(int64_t)(j0 + k) * N + n] : 0.f;
        return n < dv ? fs_load(Vb + (int64_t)(j0 + k) * av.sl + n) : (n == dv ? 1.f : 0.f);
      },
      sm);
  float* O = out + (int64_t)(per_slice_out ? blockIdx.z : bh) * M * N;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int m = m0 + ty + 16 * i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int n = n0 + tx + 16 * j;
      if (n < N) {
        if (per_slice_out) O[(int64_t)m * N + n] = acc[i][j];
        else atomicAdd(&O[(int64_t)m * N + n], acc[i][j]);
      }
    }
  }
}

// ---- exclusive running sum over the chunks, forwards (earlier chunks) or backwards (later chunks) ----
__global__ void __launch_bounds__(NTH)
bwd_scan_kernel(float* __restrict__ st, int nchunks, int64_t elems, int reverse) {
  const int bh = blockIdx.y;
  float* base = st + (int64_t)bh * nchunks * elems;
  for (int64_t e = blockIdx.x * (int64_t)NTH + threadIdx.x; e < elems; e += (int64_t)gridDim.x * NTH) {
    float run = 0.f;
    for (int c0 = 0; c0 < nchunks; c0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int c = reverse ? nchunks - 1 - (c0 + u) : c0 + u;
        v[u] = c0 + u < nchunks ? base[c * elems + e] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int c = reverse ? nchunks - 1 - (c0 + u) : c0 + u;
        if (c0 + u < nchunks) base[c * elems + e] = run;
        run += v[u];
      }
    }
  }
}

// ---- masked blocks of a chunk: MODE 0  tril(phiQ_c phiK_c^T);  MODE 1  tril(G_c [V_c | 1]^T) --------
template <typename T, int MODE>
__global__ void __launch_bounds__(NTH)
bwd_tri_kernel(const float* __restrict__ phiQ, const float* __restrict__ phiK, const float* __restrict__ G,
               const T* __restrict__ V, TensorAddr av, BwdDims q, float* __restrict__ out) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z / q.nch, c = blockIdx.z % q.nch;
  const int b = bh / q.H, h = bh % q.H;
  const int i0 = blockIdx.x * TM, j0 = blockIdx.y * TN;
  const int C = q.C, M = q.M, N = q.N, dv = q.dv, L = q.Lq;
  const int64_t row0 = (int64_t)c * C;
  float* S = out + (int64_t)blockIdx.z * C * C;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  if (j0 <= i0) {
    if (MODE == 0) {
      const float* PQ = phiQ + ((int64_t)bh * L + row0) * M;
      const float* PK = phiK + ((int64_t)bh * L + row0) * M;
      tile_gemm<true, true>(
          acc, M, [&](int r, int k) { return PQ[(int64_t)(i0 + r) * M + k]; },
          [&](int k, int cc) { return PK[(int64_t)(j0 + cc) * M + k]; }, sm);
    } else {
      const float* Gc = G + ((int64_t)bh * L + row0) * N;
      const T* Vb = V + b * av.sb + h * av.sh + row0 * av.sl;
      tile_gemm<true, true>(
          acc, N, [&](int r, int k) { return Gc[(int64_t)(i0 + r) * N + k]; },
          [&](int k, int cc) { return k < dv ? fs_load(Vb + (int64_t)(j0 + cc) * av.sl + k) : 1.f; }, sm);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int r = i0 + ty + 16 * i, cc = j0 + tx + 16 * j;
      S[(int64_t)r * C + cc] = (cc <= r) ? acc[i][j] : 0.f;
    }
}

// ---- [num | den] = phiQ KV (+ masked scores times [V_c | 1]) ------------------------------------
template <typename T>
__global__ void __launch_bounds__(NTH)
bwd_numden_kernel(const float* __restrict__ phiQ, const float* __restrict__ KV, const float* __restrict__ sc,
                  const T* __restrict__ V, TensorAddr av, BwdDims q, float* __restrict__ ND) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z, b = bh / q.H, h = bh % q.H;
  const int i0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int C = q.C, M = q.M, N = q.N, dv = q.dv, L = q.Lq;
  const int chunk = q.causal ? i0 / C : 0, ic = q.causal ? i0 - chunk * C : 0;
  const float* PQ = phiQ + (int64_t)bh * L * M;
  const float* S = KV + ((int64_t)bh * q.nch + chunk) * M * N;
  float acc[4][4] = {};
  tile_gemm<true, false>(
      acc, M, [&](int r, int k) { return (i0 + r < L) ? PQ[(int64_t)(i0 + r) * M + k] : 0.f; },
      [&](int k, int c) { return (n0 + c < N) ? S[(int64_t)k * N + n0 + c] : 0.f; }, sm);
  if (q.causal) {
    const float* SC = sc + ((int64_t)bh * q.nch + chunk) * C * C;
    const T* Vb = V + b * av.sb + h * av.sh + (int64_t)chunk * C * av.sl;
    tile_gemm<true, false>(
        acc, min(C, ic + TM), [&](int r, int k) { return SC[(int64_t)(ic + r) * C + k]; },
        [&](int k, int c) {
          const int n = n0 + c;
          return n < dv ? fs_load(Vb + (int64_t)k * av.sl + n) : (n == dv ? 1.f : 0.f);
        },
        sm);
  }
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int r = i0 + ty + 16 * i;
    if (r >= L) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int n = n0 + tx + 16 * j;
      if (n < N) ND[((int64_t)bh * L + r) * N + n] = acc[i][j];
    }
  }
}

// ---- G_i = [dY_i / den_i | -(dY_i . Y_i) / den_i], in place over [num | den]; one warp per row -----
template <typename T>
__global__ void __launch_bounds__(NTH)
bwd_g_kernel(float* __restrict__ ND, const T* __restrict__ dY, TensorAddr ay, BwdDims q, int* __restrict__ status) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bh = blockIdx.y, b = bh / q.H, h = bh % q.H;
  const int dv = q.dv, N = q.N, L = q.Lq;
  const T* dYb = dY + b * ay.sb + h * ay.sh;
  for (int i = blockIdx.x * 8 + warp; i < L; i += gridDim.x * 8) {
    float* row = ND + ((int64_t)bh * L + i) * N;
    const float den = row[dv];
    const float inv = 1.f / den;
    float s = 0.f;
    for (int c = lane; c < dv; c += 32) {
      const float dy = fs_load(dYb + (int64_t)i * ay.sl + c);
      s = fmaf(dy, row[c] * inv, s);
      row[c] = dy * inv;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
      row[dv] = -s * inv;
      if (!(den > 0.f) || !isfinite(den)) atomicExch(status, FSHARP_E_NONFINITE);
    }
  }
}

// ---- E = dphi * phi (the gradient with respect to the exponents) --------------------------------
// SIDE 1: dphiQ_c = G_c KV_c^T + tril(G_c [V_c | 1]^T) phiK_c;   SIDE 2: dphiK_c = [V_c | 1] R_c^T + tril(...)^T phiQ_c
template <typename T, int SIDE>
__global__ void __launch_bounds__(NTH)
bwd_dfeat_kernel(const float* __restrict__ phiQ, const float* __restrict__ phiK, const float* __restrict__ G,
                 const float* __restrict__ St, const float* __restrict__ gv, const T* __restrict__ V, TensorAddr av,
                 BwdDims q, float* __restrict__ E) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z, b = bh / q.H, h = bh % q.H;
  const int i0 = blockIdx.x * TM, m0 = blockIdx.y * TN;
  const int C = q.C, M = q.M, N = q.N, dv = q.dv;
  const int L = SIDE == 1 ? q.Lq : q.Lk;
  const int chunk = q.causal ? i0 / C : 0, ic = q.causal ? i0 - chunk * C : 0;
  const float* S = St + ((int64_t)bh * q.nch + chunk) * M * N;
  const float* GV = q.causal ? gv + ((int64_t)bh * q.nch + chunk) * C * C : nullptr;
  float acc[4][4] = {};
  if (SIDE == 1) {
    const float* Gb = G + (int64_t)bh * L * N;
    tile_gemm<true, true>(
        acc, N, [&](int r, int k) { return (i0 + r < L) ? Gb[(int64_t)(i0 + r) * N + k] : 0.f; },
        [&](int k, int c) { return (m0 + c < M) ? S[(int64_t)(m0 + c) * N + k] : 0.f; }, sm);
    if (q.causal) {
      const float* PK = phiK + ((int64_t)bh * L + (int64_t)chunk * C) * M;
      tile_gemm<true, false>(
          acc, min(C, ic + TM), [&](int r, int k) { return GV[(int64_t)(ic + r) * C + k]; },
          [&](int k, int c) { return (m0 + c < M) ? PK[(int64_t)k * M + m0 + c] : 0.f; }, sm);
    }
  } else {
    const T* Vb = V + b * av.sb + h * av.sh;
    tile_gemm<true, true>(
        acc, N,
        [&](int r, int k) {
          if (i0 + r >= L) return 0.f;
          return k < dv ? fs_load(Vb + (int64_t)(i0 + r) * av.sl + k) : 1.f;
        },
        [&](int k, int c) { return (m0 + c < M) ? S[(int64_t)(m0 + c) * N + k] : 0.f; }, sm);
    if (q.causal) {
      // rows ic + k of the masked block, k >= 0: the queries of this chunk at or after this tile's first key
      const float* PQ = phiQ + ((int64_t)bh * L + (int64_t)chunk * C + ic) * M;
      tile_gemm<false, false>(
          acc, C - ic, [&](int r, int k) { return GV[(int64_t)(ic + k) * C + ic + r]; },
          [&](int k, int c) { return (m0 + c < M) ? PQ[(int64_t)k * M + m0 + c] : 0.f; }, sm);
    }
  }
  const float* Ph = (SIDE == 1 ? phiQ : phiK) + (int64_t)bh * L * M;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int r = i0 + ty + 16 * i;
    if (r >= L) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int m = m0 + tx + 16 * j;
      if (m < M) E[((int64_t)bh * L + r) * M + m] = acc[i][j] * Ph[(int64_t)r * M + m];
    }
  }
}

// ---- dV_c = phiK_c R_c[:, :dv] + tril(phiQ_c phiK_c^T)^T G_c[:, :dv] ------------------------------
template <typename T>
__global__ void __launch_bounds__(NTH)
bwd_dv_kernel(const float* __restrict__ phiK, const float* __restrict__ Rt, const float* __restrict__ sc,
              const float* __restrict__ G, BwdDims q, T* __restrict__ dV, TensorAddr av) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z, b = bh / q.H, h = bh % q.H;
  const int j0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int C = q.C, M = q.M, N = q.N, dv = q.dv, L = q.Lk;
  const int chunk = q.causal ? j0 / C : 0, jc = q.causal ? j0 - chunk * C : 0;
  const float* PK = phiK + (int64_t)bh * L * M;
  const float* R = Rt + ((int64_t)bh * q.nch + chunk) * M * N;
  float acc[4][4] = {};
  tile_gemm<true, false>(
      acc, M, [&](int r, int k) { return (j0 + r < L) ? PK[(int64_t)(j0 + r) * M + k] : 0.f; },
      [&](int k, int c) { return (n0 + c < dv) ? R[(int64_t)k * N + n0 + c] : 0.f; }, sm);
  if (q.causal) {
    const float* SC = sc + ((int64_t)bh * q.nch + chunk) * C * C;
    const float* Gc = G + ((int64_t)bh * L + (int64_t)chunk * C + jc) * N;
    tile_gemm<false, false>(
        acc, C - jc, [&](int r, int k) { return SC[(int64_t)(jc + k) * C + jc + r]; },
        [&](int k, int c) { return (n0 + c < dv) ? Gc[(int64_t)k * N + n0 + c] : 0.f; }, sm);
  }
  T* Ob = dV + b * av.sb + h * av.sh;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int r = j0 + ty + 16 * i;
    if (r >= L) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int n = n0 + tx + 16 * j;
      if (n < dv) fs_store(Ob + (int64_t)r * av.sl + n, acc[i][j]);
    }
  }
}

// ---- dX = qk_scale (E W + rowsum(E) x^T (C + C^T)),  x = qk_scale X ------------------------------
template <typename T>
__global__ void __launch_bounds__(NTH)
bwd_dx_kernel(const float* __restrict__ E, const T* __restrict__ X, TensorAddr ax, int H, int L, int d, int M, int pool,
              int side, const float* __restrict__ prep, float qk_scale, T* __restrict__ dX, int* __restrict__ status) {
  __shared__ Tiles sm;
  __shared__ float rs[TM];
  const int bh = blockIdx.z, b = bh / H, h = bh % H;
  const int i0 = blockIdx.x * TM, c0 = blockIdx.y * TN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  PrepLayout pr{d, M};
  const float* pp = prep + ((size_t)(pool == FSHARP_POOL_PER_BH ? bh : h) * 2 + (side - 1)) * pr.total();
  const float* W = pp + pr.W();
  const float* Cm = pp + pr.Cmat();
  const float* Eb = E + (int64_t)bh * L * M;
  const T* Xb = X + b * ax.sb + h * ax.sh;
  {
    const int r = tid >> 2, part = tid & 3;
    float s = 0.f;
    if (i0 + r < L)
      for (int m = part; m < M; m += 4) s += Eb[(int64_t)(i0 + r) * M + m];
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (part == 0) rs[r] = s;
  }
  __syncthreads();
  float acc[4][4] = {}, quad[4][4] = {};
  tile_gemm<true, false>(
      acc, M, [&](int r, int k) { return (i0 + r < L) ? Eb[(int64_t)(i0 + r) * M + k] : 0.f; },
      [&](int k, int c) { return (c0 + c < d) ? W[(size_t)k * d + c0 + c] : 0.f; }, sm);
  tile_gemm<true, false>(
      quad, d, [&](int r, int k) { return (i0 + r < L) ? qk_scale * fs_load(Xb + (int64_t)(i0 + r) * ax.sl + k) : 0.f; },
      [&](int k, int c) { return (c0 + c < d) ? Cm[(size_t)k * d + c0 + c] + Cm[(size_t)(c0 + c) * d + k] : 0.f; }, sm);
  T* Ob = dX + b * ax.sb + h * ax.sh;
  bool bad = false;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int r = ty + 16 * i;
    if (i0 + r >= L) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int c = c0 + tx + 16 * j;
      if (c < d) {
        const float v = qk_scale * fmaf(rs[r], quad[i][j], acc[i][j]);
        if (!isfinite(v)) bad = true;
        fs_store(Ob + (int64_t)(i0 + r) * ax.sl + c, v);
      }
    }
  }
  if (bad) atomicExch(status, FSHARP_E_NONFINITE);
}

int slices_for(const fsharp_ctx* ctx, int BH, int L, int* slice_len) {
  int nsl = (4 * ctx->sm_count + BH - 1) / BH;
  const int maxsl = (L + 255) / 256;
  if (nsl > maxsl) nsl = maxsl;
  if (nsl > 65535 / BH) nsl = 65535 / BH;
  if (nsl < 1) nsl = 1;
  const int slen = (L + nsl - 1) / nsl;
  *slice_len = slen;
  return (L + slen - 1) / slen;
}

template <typename T>
int backward_t(fsharp_ctx* ctx, const void* Qv, const void* Kv, const void* Vv, const void* dYv, const fsharp_dims* dm,
               int dtype, int causal, int chunk, float qk_scale, const float* prep, void* dQv, void* dKv, void* dVv,
               WsAlloc* ws) {
  const T* Q = (const T*)Qv; const T* K = (const T*)Kv; const T* V = (const T*)Vv; const T* dY = (const T*)dYv;
  const int B = dm->B, H = dm->H, BH = B * H, Lq = dm->Lq, Lk = dm->Lk, d = dm->d, dv = dm->dv, M = dm->M;
  const int N = dv + 1;
  BwdDims q{H, Lq, Lk, d, dv, M, N, causal ? 1 : 0, causal ? chunk : 0, causal ? Lq / chunk : 1};
  const int C = q.C, nch = q.nch;
  TensorAddr aq = fs_addr(dm->q_stride, H, Lq, d), ak = fs_addr(dm->k_stride, H, Lk, d);
  TensorAddr av = fs_addr(dm->v_stride, H, Lk, dv), ay = fs_addr(dm->y_stride, H, Lq, dv);
  float* phiQ = ws->take<float>((size_t)BH * Lq * M);
  float* phiK = ws->take<float>((size_t)BH * Lk * M);
  float* EQ = ws->take<float>((size_t)BH * Lq * M);
  float* EK = ws->take<float>((size_t)BH * Lk * M);
  float* rowc = ws->take<float>((size_t)BH * (Lq > Lk ? Lq : Lk));
  unsigned* gmax = ws->take<unsigned>((size_t)BH);
  float* lsq = ws->take<float>((size_t)BH * Lq);
  float* lsk = ws->take<float>((size_t)BH);
  float* ND = ws->take<float>((size_t)BH * Lq * N);
  float* KV = ws->take<float>((size_t)BH * nch * M * N);
  float* Rt = ws->take<float>((size_t)BH * nch * M * N);
  float* sc = causal ? ws->take<float>((size_t)BH * nch * C * C) : nullptr;
  float* gv = causal ? ws->take<float>((size_t)BH * nch * C * C) : nullptr;
  cudaStream_t st = ctx->stream;

  FS_TRY(fs_simt_featurize(ctx, K, dtype, ak, B, H, Lk, d, M, dm->pool, prep, 2, qk_scale, FSHARP_STAB_GROUP, rowc,
                           gmax, phiK, lsk));
  FS_TRY(fs_simt_featurize(ctx, Q, dtype, aq, B, H, Lq, d, M, dm->pool, prep, 1, qk_scale, FSHARP_STAB_ROW, rowc,
                           gmax, phiQ, lsq));
  const dim3 gstate((M + TM - 1) / TM, (N + TN - 1) / TN, 1);
  const int64_t elems = (int64_t)M * N;
  const dim3 gscan((unsigned)((elems + NTH - 1) / NTH), BH);
  int slen = 0, nsl = 1;
  // 1. key-side sums: the total (bidirectional) or the sum over earlier chunks (causal)
  if (!causal) {
    nsl = slices_for(ctx, BH, Lk, &slen);
    FS_CUDA_OK(cudaMemsetAsync(KV, 0, (size_t)BH * M * N * sizeof(float), st));
    bwd_state_kernel<T, false><<<dim3(gstate.x, gstate.y, BH * nsl), NTH, 0, st>>>(phiK, V, av, nullptr, q, Lk, slen, nsl, 0, KV);
    FS_LAUNCH_CHECK(ctx);
  } else {
    bwd_state_kernel<T, false><<<dim3(gstate.x, gstate.y, BH * nch), NTH, 0, st>>>(phiK, V, av, nullptr, q, Lk, C, nch, 1, KV);
    FS_LAUNCH_CHECK(ctx);
    bwd_scan_kernel<<<gscan, NTH, 0, st>>>(KV, nch, elems, 0);
    FS_LAUNCH_CHECK(ctx);
    bwd_tri_kernel<T, 0><<<dim3(C / TM, C / TN, BH * nch), NTH, 0, st>>>(phiQ, phiK, nullptr, V, av, q, sc);
    FS_LAUNCH_CHECK(ctx);
  }
  // 2. numerators and normalisers, then G in their place
  bwd_numden_kernel<T><<<dim3((Lq + TM - 1) / TM, (N + TN - 1) / TN, BH), NTH, 0, st>>>(phiQ, KV, sc, V, av, q, ND);
  FS_LAUNCH_CHECK(ctx);
  {
    int gx = (Lq + 7) / 8;
    if (gx > 4 * ctx->sm_count) gx = 4 * ctx->sm_count;
    bwd_g_kernel<T><<<dim3(gx, BH), NTH, 0, st>>>(ND, dY, ay, q, ctx->d_status);
    FS_LAUNCH_CHECK(ctx);
  }
  const float* G = ND;
  // 3. query-side sums R: the total, or the sum over later chunks
  if (!causal) {
    nsl = slices_for(ctx, BH, Lq, &slen);
    FS_CUDA_OK(cudaMemsetAsync(Rt, 0, (size_t)BH * M * N * sizeof(float), st));
    bwd_state_kernel<T, true><<<dim3(gstate.x, gstate.y, BH * nsl), NTH, 0, st>>>(phiQ, V, av, G, q, Lq, slen, nsl, 0, Rt);
    FS_LAUNCH_CHECK(ctx);
  } else {
    bwd_state_kernel<T, true><<<dim3(gstate.x, gstate.y, BH * nch), NTH, 0, st>>>(phiQ, V, av, G, q, Lq, C, nch, 1, Rt);
    FS_LAUNCH_CHECK(ctx);
    bwd_scan_kernel<<<gscan, NTH, 0, st>>>(Rt, nch, elems, 1);
    FS_LAUNCH_CHECK(ctx);
    bwd_tri_kernel<T, 1><<<dim3(C / TM, C / TN, BH * nch), NTH, 0, st>>>(phiQ, phiK, G, V, av, q, gv);
    FS_LAUNCH_CHECK(ctx);
  }
  // 4. gradients with respect to the exponents, dV, then dQ and dK
  bwd_dfeat_kernel<T, 1><<<dim3((Lq + TM - 1) / TM, (M + TN - 1) / TN, BH), NTH, 0, st>>>(phiQ, phiK, G, KV, gv, V, av, q, EQ);
  FS_LAUNCH_CHECK(ctx);
  bwd_dfeat_kernel<T, 2><<<dim3((Lk + TM - 1) / TM, (M + TN - 1) / TN, BH), NTH, 0, st>>>(phiQ, phiK, G, Rt, gv, V, av, q, EK);
  FS_LAUNCH_CHECK(ctx);
  bwd_dv_kernel<T><<<dim3((Lk + TM - 1) / TM, (dv + TN - 1) / TN, BH), NTH, 0, st>>>(phiK, Rt, sc, G, q, (T*)dVv, av);
  FS_LAUNCH_CHECK(ctx);
  bwd_dx_kernel<T><<<dim3((Lq + TM - 1) / TM, (d + TN - 1) / TN, BH), NTH, 0, st>>>(EQ, Q, aq, H, Lq, d, M, dm->pool, 1, prep,
                                                                                  qk_scale, (T*)dQv, ctx->d_status);
  FS_LAUNCH_CHECK(ctx);
  bwd_dx_kernel<T><<<dim3((Lk + TM - 1) / TM, (d + TN - 1) / TN, BH), NTH, 0, st>>>(EK, K, ak, H, Lk, d, M, dm->pool, 2, prep,
                                                                                  qk_scale, (T*)dKv, ctx->d_status);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}

}  // namespace

size_t fs_backward_scratch_bytes(const fsharp_dims* dm, int causal, int chunk) {
  const size_t BH = (size_t)dm->B * dm->H, N = dm->dv + 1, M = dm->M;
  const size_t Lq = dm->Lq, Lk = dm->Lk, Lmax = Lq > Lk ? Lq : Lk;
  const size_t nch = causal && chunk > 0 ? Lq / chunk : 1;
  size_t b = 2 * ws_round(BH * Lq * M * 4) + 2 * ws_round(BH * Lk * M * 4) + ws_round(BH * Lmax * 4) + ws_round(BH * 4) +
             ws_round(BH * Lq * 4) + ws_round(BH * 4) + ws_round(BH * Lq * N * 4) + 2 * ws_round(BH * nch * M * N * 4);
  if (causal) b += 2 * ws_round(BH * nch * (size_t)chunk * chunk * 4);
  return b;
}

int fs_backward(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const void* dY, const fsharp_dims* dm,
                int dtype, int causal, int chunk, float qk_scale, const float* prep, void* dQ, void* dK, void* dV,
                WsAlloc* ws) {
  if (dtype == FSHARP_F32)
    return backward_t<float>(ctx, Q, K, V, dY, dm, dtype, causal, chunk, qk_scale, prep, dQ, dK, dV, ws);
  return backward_t<__nv_bfloat16>(ctx, Q, K, V, dY, dm, dtype, causal, chunk, qk_scale, prep, dQ, dK, dV, ws);
}
