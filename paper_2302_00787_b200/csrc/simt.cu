// fp32 CUDA-core path: features (Section 4 definition with Section 2.1's M^-1/2) and the
// linear-attention contraction (Sections 2.1 / 2.2), bidirectional and causal-chunked.
// Used for fp32 inputs, for shapes the tensor-core path does not take, and on request.
//
// Scratch (from the context workspace): the two feature matrices, the per-token
// quadratic term, S^T [V | 1] (per (batch, head); per chunk when causal) and, when
// causal, the masked in-chunk score blocks.
#include "common.cuh"
#include "simt_tile.cuh"

namespace {

__device__ __forceinline__ int group_of(int bh, int H, int pool) { return pool == FSHARP_POOL_PER_BH ? bh : bh % H; }

// ---- per-token quadratic term c_i = x_i^T C x_i --------------------------------------
template <typename T>
__global__ void __launch_bounds__(NTH)
rowterm_kernel(const T* __restrict__ X, TensorAddr ax, int H, int L, int d, int M, int pool, int side,
               const float* __restrict__ prep, float qk_scale, float* __restrict__ rowc) {
  extern __shared__ float smf[];
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  PrepLayout pr{d, M};
  const float* pp = prep + ((size_t)group_of(bh, H, pool) * 2 + (side - 1)) * pr.total();
  const float* scal = pp + pr.scal();
  const bool cscalar = scal[PS_CSCALAR] != 0.f;
  const float gamma = scal[PS_CGAMMA];
  float* Cs = smf;                   // d*d (only when C is dense)
  float* xs = smf + (cscalar ? 0 : d * d);   // 8 warps * d
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (!cscalar) {
    const float* Cm = pp + pr.Cmat();
    for (int e = tid; e < d * d; e += NTH) Cs[e] = Cm[e];
  }
  __syncthreads();
  const T* Xb = X + b * ax.sb + h * ax.sh;
  float* xw = xs + warp * d;
  for (int i = blockIdx.x * 8 + warp; i < L; i += gridDim.x * 8) {
    for (int j = lane; j < d; j += 32) xw[j] = qk_scale * fs_load(Xb + (int64_t)i * ax.sl + j);
    __syncwarp();
    float s = 0.f;
    if (cscalar) {
      for (int j = lane; j < d; j += 32) s = fmaf(xw[j], xw[j], s);
      s *= gamma;
    } else {
      for (int j = lane; j < d; j += 32) {
        float t = 0.f;
        for (int k = 0; k < d; k++) t = fmaf(xw[k], Cs[k * d + j], t);
        s = fmaf(t, xw[j], s);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) rowc[(int64_t)bh * L + i] = s;
    __syncwarp();
  }
}

// ---- exponents e_im = bias + a_m + w_m . x_i + c_i -----------------------------------
template <typename T>
__global__ void __launch_bounds__(NTH)
logits_kernel(const T* __restrict__ X, TensorAddr ax, int H, int L, int d, int M, int pool, int side,
              const float* __restrict__ prep, float qk_scale, const float* __restrict__ rowc,
              float* __restrict__ phi) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z, b = bh / H, h = bh % H;
  const int i0 = blockIdx.x * TM, m0 = blockIdx.y * TN;
  PrepLayout pr{d, M};
  const float* pp = prep + ((size_t)group_of(bh, H, pool) * 2 + (side - 1)) * pr.total();
  const float* W = pp + pr.W();
  const float* av = pp + pr.a();
  const float bias = pp[pr.scal() + PS_BIAS];
  const T* Xb = X + b * ax.sb + h * ax.sh;
  float acc[4][4] = {};
  tile_gemm<true, true>(
      acc, d,
      [&](int r, int k) { return (i0 + r < L) ? qk_scale * fs_load(Xb + (int64_t)(i0 + r) * ax.sl + k) : 0.f; },
      [&](int k, int c) { return (m0 + c < M) ? W[(size_t)(m0 + c) * d + k] : 0.f; }, sm);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    int row = i0 + ty + 16 * i;
    if (row >= L) continue;
    float ci = rowc[(int64_t)bh * L + row] + bias;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      int m = m0 + tx + 16 * j;
      if (m < M) phi[((int64_t)bh * L + row) * M + m] = acc[i][j] + av[m] + ci;
    }
  }
}

// Order-preserving map float -> unsigned, so that atomicMax on words gives the float maximum.
__device__ __forceinline__ unsigned f2ord(float f) {
  unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord2f(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// ---- largest exponent of each (batch, head) --------------------------------------------
__global__ void __launch_bounds__(NTH)
groupmax_kernel(const float* __restrict__ phi, int64_t per_bh, unsigned* __restrict__ gmax) {
  __shared__ float red[NTH / 32];
  const int bh = blockIdx.y;
  const float* p = phi + (int64_t)bh * per_bh;
  float mx = -3.0e38f;
  for (int64_t e = blockIdx.x * (int64_t)NTH + threadIdx.x; e < per_bh; e += (int64_t)gridDim.x * NTH)
    mx = fmaxf(mx, p[e]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < NTH / 32; i++) mx = fmaxf(mx, red[i]);
    atomicMax(&gmax[bh], f2ord(mx));
  }
}

// ---- phi = exp(e - shift), one warp per row ------------------------------------------
// shift: the row's largest exponent (ROW), the (batch, head)'s largest exponent (GROUP), or 0.
__global__ void __launch_bounds__(NTH)
expshift_kernel(float* __restrict__ phi, int L, int M, int stab, const unsigned* __restrict__ gmax,
                float* __restrict__ logscale, __nv_bfloat16* __restrict__ phi16, int keep32, int* __restrict__ status) {
  // keep32 == 0 (only with phi16): the fp32 features have no reader, only the bf16 copy is written
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bh = blockIdx.y;
  const float gshift = stab == FSHARP_STAB_GROUP ? ord2f(gmax[bh]) : 0.f;
  for (int i = blockIdx.x * 8 + warp; i < L; i += gridDim.x * 8) {
    float* row = phi + ((int64_t)bh * L + i) * M;
    float s = 0.f;
    if (stab == FSHARP_STAB_ROW) {
      float mx = -3.0e38f;
      for (int m = lane; m < M; m += 32) mx = fmaxf(mx, row[m]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      s = mx;
    } else if (stab == FSHARP_STAB_GROUP) {
      s = gshift;
    }
    bool bad = false;
    for (int m = lane; m < M; m += 32) {
      float e = row[m];
      if (!isfinite(e)) bad = true;
      const float f = expf(e - s);
      if (keep32) row[m] = f;
      if (phi16) phi16[((int64_t)bh * L + i) * M + m] = __float2bfloat16_rn(f);     // (a copy for the tensor-core score kernel)
    }
    if (bad) atomicExch(status, FSHARP_E_NONFINITE);
    if (logscale && lane == 0) {
      if (stab == FSHARP_STAB_ROW) logscale[(int64_t)bh * L + i] = s;
      else if (stab == FSHARP_STAB_GROUP && i == 0) logscale[bh] = s;
    }
  }
}

// ---- S^T [V | 1]: out[slot][m][n] += sum_{j in slice} phiK[j][m] * V1[j][n] -------------
template <typename T>
__global__ void __launch_bounds__(NTH)
kv_kernel(const float* __restrict__ phiK, const T* __restrict__ V, TensorAddr av, int H, int L, int M, int dv,
          int slice_len, int nslices, int per_slice_out, float* __restrict__ out) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z / nslices, sl = blockIdx.z % nslices;
  const int b = bh / H, h = bh % H;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int j0 = sl * slice_len, j1 = min(L, j0 + slice_len);
  if (j0 >= j1) return;
  const int N = dv + 1;
  const float* P = phiK + (int64_t)bh * L * M;
  const T* Vb = V + b * av.sb + h * av.sh;
  float acc[4][4] = {};
  tile_gemm<false, false>(
      acc, j1 - j0,
      [&](int r, int k) { return (m0 + r < M) ? P[(int64_t)(j0 + k) * M + m0 + r] : 0.f; },
      [&](int k, int c) {
        int n = n0 + c;
        return n < dv ? fs_load(Vb + (int64_t)(j0 + k) * av.sl + n) : (n == dv ? 1.f : 0.f);
      },
      sm);
  float* O = out + (int64_t)(per_slice_out ? blockIdx.z : bh) * M * N;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    int m = m0 + ty + 16 * i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      int n = n0 + tx + 16 * j;
      if (n < N) {
        if (per_slice_out) O[(int64_t)m * N + n] = acc[i][j];
        else atomicAdd(&O[(int64_t)m * N + n], acc[i][j]);
      }
    }
  }
}

// ---- exclusive prefix over chunks of the per-chunk S^T [V | 1] ---------------------------
__global__ void __launch_bounds__(NTH)
prefix_kernel(float* __restrict__ st, int nchunks, int64_t elems, __nv_bfloat16* __restrict__ st16) {
  const int bh = blockIdx.y;
  float* base = st + (int64_t)bh * nchunks * elems;
  for (int64_t e = blockIdx.x * (int64_t)NTH + threadIdx.x; e < elems; e += (int64_t)gridDim.x * NTH) {
    float run = 0.f;
    // eight chunks at a time: the loads are issued together, then the running sums are stored
    for (int c0 = 0; c0 < nchunks; c0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; u++) v[u] = c0 + u < nchunks ? base[(c0 + u) * elems + e] : 0.f;
#pragma unroll
      for (int u = 0; u < 8; u++) {
        if (c0 + u < nchunks) {
          base[(c0 + u) * elems + e] = run;
          if (st16) st16[((int64_t)bh * nchunks + c0 + u) * elems + e] = __float2bfloat16_rn(run);   // (for the tensor-core query side)
        }
        run += v[u];
      }
    }
  }
}

// ---- masked in-chunk scores: sc[bh, c][i][j] = (j <= i) phiQ_i . phiK_j -------------------
__global__ void __launch_bounds__(NTH)
scores_kernel(const float* __restrict__ phiQ, const float* __restrict__ phiK, int L, int M, int C, int nchunks,
              float* __restrict__ sc) {
  __shared__ Tiles sm;
  const int bh = blockIdx.z / nchunks, c = blockIdx.z % nchunks;
  const int i0 = blockIdx.x * TM, j0 = blockIdx.y * TN;
  float* S = sc + (int64_t)blockIdx.z * C * C;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  if (j0 <= i0) {
    const float* PQ = phiQ + ((int64_t)bh * L + (int64_t)c * C) * M;
    const float* PK = phiK + ((int64_t)bh * L + (int64_t)c * C) * M;
    tile_gemm<true, true>(
        acc, M, [&](int r, int k) { return PQ[(int64_t)(i0 + r) * M + k]; },
        [&](int k, int cc) { return PK[(int64_t)(j0 + cc) * M + k]; }, sm);
  }
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) {
      int r = i0 + ty + 16 * i, cc = j0 + tx + 16 * j;
      S[(int64_t)r * C + cc] = (cc <= r) ? acc[i][j] : 0.f;
    }
}

// ---- Y = num / den -------------------------------------------------------------------
// Bidirectional: [num | den] = phiQ (S^T [V | 1]).  Causal: per chunk, phiQ_c times the
// prefix state plus the masked scores times [V_c | 1].
template <typename T>
__global__ void __launch_bounds__(NTH)
out_kernel(const float* __restrict__ phiQ, const float* __restrict__ KV, const float* __restrict__ sc,
           const T* __restrict__ V, TensorAddr av, T* __restrict__ Y, TensorAddr ay, int H, int L, int M, int dv,
           int causal, int C, int nchunks, const float* __restrict__ lsq, const float* __restrict__ lsk,
           int st_t, int* __restrict__ status) {
  // st_t != 0: the states are stored column index first, [dv + 1][M] (the tensor-core key-side kernel writes them so)
  // lsq != nullptr: the unnormalised operator Khat C of Section 2.1 is wanted: row i of the numerator times
  // exp(lsq[i] + lsk[bh]), the shifts that the feature kernels took out of phi(Q) and phi(K)
  __shared__ Tiles sm;
  __shared__ float den[TM];
  const int bh = blockIdx.z, b = bh / H, h = bh % H;
  const int i0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int N = dv + 1;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const float* PQ = phiQ + (int64_t)bh * L * M;
  const int chunk = causal ? i0 / C : 0;
  const float* S = KV + (int64_t)(causal ? bh * nchunks + chunk : bh) * M * N;
  const float* SC = causal ? sc + ((int64_t)bh * nchunks + chunk) * C * C : nullptr;
  const int ic = causal ? i0 - chunk * C : 0;   // row offset inside the chunk
  const T* Vb = V + b * av.sb + h * av.sh;

  // denominators: 4 threads per row
  {
    int r = tid >> 2, part = tid & 3;
    float s = 0.f;
    if (i0 + r < L) {
      for (int m = part; m < M; m += 4) s = fmaf(PQ[(int64_t)(i0 + r) * M + m], st_t ? S[(int64_t)dv * M + m] : S[(int64_t)m * N + dv], s);
      if (causal)
        for (int j = part; j < C; j += 4) s += SC[(int64_t)(ic + r) * C + j];
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (part == 0) den[r] = s;
  }
  __syncthreads();
  float acc[4][4] = {};
  if (st_t)
    tile_gemm<true, true>(
        acc, M, [&](int r, int k) { return (i0 + r < L) ? PQ[(int64_t)(i0 + r) * M + k] : 0.f; },
        [&](int k, int c) { return (n0 + c < dv) ? S[(int64_t)(n0 + c) * M + k] : 0.f; }, sm);
  else
    tile_gemm<true, false>(
        acc, M, [&](int r, int k) { return (i0 + r < L) ? PQ[(int64_t)(i0 + r) * M + k] : 0.f; },
        [&](int k, int c) { return (n0 + c < dv) ? S[(int64_t)k * N + n0 + c] : 0.f; }, sm);
  if (causal) {
    const int jmax = min(C, ic + TM);   // columns beyond the tile's last row are masked to zero
    tile_gemm<true, false>(
        acc, jmax, [&](int r, int k) { return SC[(int64_t)(ic + r) * C + k]; },
        [&](int k, int c) {
          return (n0 + c < dv) ? fs_load(Vb + (int64_t)(chunk * C + k) * av.sl + n0 + c) : 0.f;
        },
        sm);
  }
  T* Yb = Y + b * ay.sb + h * ay.sh;
  bool bad = false;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    int r = ty + 16 * i;
    if (i0 + r >= L) continue;
    float dn = den[r];
    float inv;
    if (lsq != nullptr) {
      inv = expf(lsq[(int64_t)bh * L + i0 + r] + lsk[bh]);
    } else {
      if (!(dn > 0.f) || !isfinite(dn)) bad = true;
      inv = 1.f / dn;
    }
#pragma unroll
    for (int j = 0; j < 4; j++) {
      int n = n0 + tx + 16 * j;
      if (n < dv) fs_store(Yb + (int64_t)(i0 + r) * ay.sl + n, acc[i][j] * inv);
    }
  }
  if (bad) atomicExch(status, FSHARP_E_NONFINITE);
}

template <typename T>
int featurize_t(fsharp_ctx* ctx, const void* X, TensorAddr ax, int B, int H, int L, int d, int M, int pool,
                const float* prep, int side, float qk_scale, int stab, float* rowc, unsigned* gmax, float* phi,
                float* logscale, __nv_bfloat16* phi16 = nullptr, bool keep32 = true) {
  const int BH = B * H;
  if (BH == 0 || L == 0) return FSHARP_OK;
  {
    int gx = (L + 7) / 8;
    if (gx > 4 * ctx->sm_count) gx = 4 * ctx->sm_count;
    // shared memory: dense C (d*d) + one x per warp; sized for the dense case
    size_t smem = ((size_t)d * d + 8 * (size_t)d) * sizeof(float);
    FS_CUDA_OK(cudaFuncSetAttribute(rowterm_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    FS_TIME_BEGIN(ctx, FS_K_ROWTERM);
    rowterm_kernel<T><<<dim3(gx, BH), NTH, smem, ctx->stream>>>((const T*)X, ax, H, L, d, M, pool, side, prep,
                                                               qk_scale, rowc);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
  }
  // bf16 tokens with d = 128 (no fused attention kernel takes them): the exponents' product on the tensor cores
  if (ctx->impl != FSHARP_IMPL_SIMT && fs_tc_logits128_supported(X, sizeof(T) == 2 ? FSHARP_BF16 : FSHARP_F32, ax, L, d, M)) {
    FS_TRY(fs_tc_logits128(ctx, X, ax, B, H, L, M, pool, prep, side, qk_scale, rowc, phi));
  } else {
    FS_TIME_BEGIN(ctx, FS_K_LOGITS);
    logits_kernel<T><<<dim3((L + TM - 1) / TM, (M + TN - 1) / TN, BH), NTH, 0, ctx->stream>>>(
        (const T*)X, ax, H, L, d, M, pool, side, prep, qk_scale, rowc, phi);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
  }
  {
    int gx = (L + 7) / 8;
    if (gx > 4 * ctx->sm_count) gx = 4 * ctx->sm_count;
    if (stab == FSHARP_STAB_GROUP) {
      FS_CUDA_OK(cudaMemsetAsync(gmax, 0, (size_t)BH * sizeof(unsigned), ctx->stream));
      int64_t per_bh = (int64_t)L * M;
      int gm = (int)((per_bh + 16 * NTH - 1) / (16 * NTH));
      if (gm > 64) gm = 64;
      FS_TIME_BEGIN(ctx, FS_K_GROUPMAX);
      groupmax_kernel<<<dim3(gm, BH), NTH, 0, ctx->stream>>>(phi, per_bh, gmax);
      FS_TIME_END(ctx);
      FS_LAUNCH_CHECK(ctx);
    }
    FS_TIME_BEGIN(ctx, FS_K_EXPSHIFT);
    expshift_kernel<<<dim3(gx, BH), NTH, 0, ctx->stream>>>(phi, L, M, stab, gmax, logscale, phi16, (keep32 || !phi16) ? 1 : 0, ctx->d_status);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
  }
  return FSHARP_OK;
}

template <typename T>
int attend_t(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, int causal,
             int chunk, float qk_scale, const float* prep, void* Y, WsAlloc* ws, bool unnormalised) {
  const int B = dm->B, H = dm->H, BH = B * H, Lq = dm->Lq, Lk = dm->Lk, d = dm->d, dv = dm->dv, M = dm->M;
  const int N = dv + 1;
  TensorAddr aq = fs_addr(dm->q_stride, H, Lq, d), ak = fs_addr(dm->k_stride, H, Lk, d);
  TensorAddr av = fs_addr(dm->v_stride, H, Lk, dv), ay = fs_addr(dm->y_stride, H, Lq, dv);
  float* phiQ = ws->take<float>((size_t)BH * Lq * M);
  float* phiK = ws->take<float>((size_t)BH * Lk * M);
  float* rowc = ws->take<float>((size_t)BH * (Lq > Lk ? Lq : Lk));
  unsigned* gmax = ws->take<unsigned>((size_t)BH);
  float* lsq = unnormalised ? ws->take<float>((size_t)BH * Lq) : nullptr;
  float* lsk = unnormalised ? ws->take<float>((size_t)BH) : nullptr;
  // causal, bf16 tensors: the in-chunk scores come from the tensor cores, from bf16 copies of the features
  const bool tc_scores = causal && !unnormalised && sizeof(T) == 2 && ctx->impl != FSHARP_IMPL_SIMT &&
                         fs_tc_scores128_supported(M, chunk);
  // (with the bf16 copy of phi(K) at hand: the per-chunk sums on the tensor cores, stored column index first; and then
  // the query side as well, from bf16 copies of the running sums and of the scores)
  const bool tc_kv = tc_scores && fs_tc_kv128_supported(V, av, dv, M, chunk);
  const bool tc_out = tc_kv && fs_tc_out128_supported(Y, ay);
  __nv_bfloat16* phiQ16 = tc_scores ? ws->take<__nv_bfloat16>((size_t)BH * Lq * M) : nullptr;
  __nv_bfloat16* phiK16 = tc_scores ? ws->take<__nv_bfloat16>((size_t)BH * Lk * M) : nullptr;
  FS_TRY(featurize_t<T>(ctx, K, ak, B, H, Lk, d, M, dm->pool, prep, 2, qk_scale, FSHARP_STAB_GROUP, rowc, gmax,
                        phiK, lsk, phiK16, !tc_kv));
  FS_TRY(featurize_t<T>(ctx, Q, aq, B, H, Lq, d, M, dm->pool, prep, 1, qk_scale, FSHARP_STAB_ROW, rowc, gmax,
                        phiQ, lsq, phiQ16, !tc_out));
  dim3 gout((Lq + TM - 1) / TM, (dv + TN - 1) / TN, BH);
  if (!causal) {
    float* KV = ws->take<float>((size_t)BH * M * N);
    FS_CUDA_OK(cudaMemsetAsync(KV, 0, (size_t)BH * M * N * sizeof(float), ctx->stream));
    int nsl = (4 * ctx->sm_count + BH - 1) / BH;
    int maxsl = (Lk + 255) / 256;
    if (nsl > maxsl) nsl = maxsl;
    if (nsl > 65535 / BH) nsl = 65535 / BH;          // the (unit, slice) index is a grid z coordinate
    if (nsl < 1) nsl = 1;
    int slen = (Lk + nsl - 1) / nsl;
    nsl = (Lk + slen - 1) / slen;
    FS_TIME_BEGIN(ctx, FS_K_KV);
    kv_kernel<T><<<dim3((M + TM - 1) / TM, (N + TN - 1) / TN, BH * nsl), NTH, 0, ctx->stream>>>(
        phiK, (const T*)V, av, H, Lk, M, dv, slen, nsl, 0, KV);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
    FS_TIME_BEGIN(ctx, FS_K_OUT);
    out_kernel<T><<<gout, NTH, 0, ctx->stream>>>(phiQ, KV, nullptr, (const T*)V, av, (T*)Y, ay, H, Lq, M, dv, 0, 0,
                                                1, lsq, lsk, 0, ctx->d_status);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
  } else {
    const int C = chunk, nch = Lq / C;
    float* st = ws->take<float>((size_t)BH * nch * M * N);
    float* sc = ws->take<float>((size_t)BH * nch * C * C);
    __nv_bfloat16* st16 = tc_out ? ws->take<__nv_bfloat16>((size_t)BH * nch * M * N) : nullptr;
    __nv_bfloat16* sc16 = tc_out ? ws->take<__nv_bfloat16>((size_t)BH * nch * C * C) : nullptr;
    if (tc_kv) {
      FS_TRY(fs_tc_kv128(ctx, phiK16, V, av, B, H, Lk, M, C, st));
    } else {
      FS_TIME_BEGIN(ctx, FS_K_KV);
      kv_kernel<T><<<dim3((M + TM - 1) / TM, (N + TN - 1) / TN, BH * nch), NTH, 0, ctx->stream>>>(
          phiK, (const T*)V, av, H, Lk, M, dv, C, nch, 1, st);
      FS_TIME_END(ctx);
      FS_LAUNCH_CHECK(ctx);
    }
    int64_t elems = (int64_t)M * N;
    FS_TIME_BEGIN(ctx, FS_K_PREFIX);
    prefix_kernel<<<dim3((unsigned)((elems + NTH - 1) / NTH), BH), NTH, 0, ctx->stream>>>(st, nch, elems, st16);
    FS_TIME_END(ctx);
    FS_LAUNCH_CHECK(ctx);
    if (tc_scores) {
      FS_TRY(fs_tc_scores128(ctx, phiQ16, phiK16, BH, Lq, M, C, tc_out ? nullptr : sc, sc16));
    } else {
      FS_TIME_BEGIN(ctx, FS_K_SCORES);
      scores_kernel<<<dim3(C / TM, C / TN, BH * nch), NTH, 0, ctx->stream>>>(phiQ, phiK, Lq, M, C, nch, sc);
      FS_TIME_END(ctx);
      FS_LAUNCH_CHECK(ctx);
    }
    if (tc_out) {
      FS_TRY(fs_tc_out128(ctx, phiQ16, st16, sc16, V, av, Y, ay, B, H, Lq, M, C));
    } else {
      FS_TIME_BEGIN(ctx, FS_K_OUT);
      out_kernel<T><<<gout, NTH, 0, ctx->stream>>>(phiQ, st, sc, (const T*)V, av, (T*)Y, ay, H, Lq, M, dv, 1, C, nch,
                                                  nullptr, nullptr, tc_kv ? 1 : 0, ctx->d_status);
      FS_TIME_END(ctx);
      FS_LAUNCH_CHECK(ctx);
    }
  }
  return FSHARP_OK;
}

}  // namespace

int fs_simt_featurize(fsharp_ctx* ctx, const void* X, int dtype, TensorAddr ax, int B, int H, int L, int d,
                      int M, int pool, const float* prep, int side, float qk_scale, int stab,
                      float* rowc, unsigned* gmax, float* phi, float* logscale) {
  if (dtype == FSHARP_F32)
    return featurize_t<float>(ctx, X, ax, B, H, L, d, M, pool, prep, side, qk_scale, stab, rowc, gmax, phi,
                              logscale);
  return featurize_t<__nv_bfloat16>(ctx, X, ax, B, H, L, d, M, pool, prep, side, qk_scale, stab, rowc, gmax, phi,
                                    logscale);
}

size_t fs_simt_attend_scratch_bytes(const fsharp_dims* dm, int causal, int chunk) {
  const size_t BH = (size_t)dm->B * dm->H, N = dm->dv + 1;
  const size_t Lmax = dm->Lq > dm->Lk ? dm->Lq : dm->Lk;
  size_t b = ws_round(BH * dm->Lq * dm->M * 4) + ws_round(BH * dm->Lk * dm->M * 4) + ws_round(BH * Lmax * 4) +
             ws_round(BH * 4) + ws_round(BH * dm->Lq * 4) + ws_round(BH * 4);     // (the last two: the shifts of the unnormalised mode)
  if (!causal) {
    b += ws_round(BH * dm->M * N * 4);
  } else {
    size_t nch = chunk > 0 ? dm->Lq / chunk : 0;
    b += ws_round(BH * nch * dm->M * N * 4) + ws_round(BH * nch * (size_t)chunk * chunk * 4);
    b += ws_round(BH * dm->Lq * dm->M * 2) + ws_round(BH * dm->Lk * dm->M * 2);      // bf16 copies of the features
    b += ws_round(BH * nch * dm->M * N * 2) + ws_round(BH * nch * (size_t)chunk * chunk * 2);   // ... of the running sums and the scores
  }
  return b;
}

int fs_simt_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm,
                   int dtype, int causal, int chunk, float qk_scale, const float* prep, void* Y, WsAlloc* ws) {
  if (dtype == FSHARP_F32) return attend_t<float>(ctx, Q, K, V, dm, causal, chunk, qk_scale, prep, Y, ws, false);
  return attend_t<__nv_bfloat16>(ctx, Q, K, V, dm, causal, chunk, qk_scale, prep, Y, ws, false);
}

// The unnormalised operator Khat C (Section 2.1): the bidirectional pipeline with the shifts carried to the output.
int fs_simt_kernel_apply(fsharp_ctx* ctx, const void* X, const void* Yset, const void* Cmat, const fsharp_dims* dm,
                         int dtype, float qk_scale, const float* prep, void* out, WsAlloc* ws) {
  if (dtype == FSHARP_F32) return attend_t<float>(ctx, X, Yset, Cmat, dm, 0, 0, qk_scale, prep, out, ws, true);
  return attend_t<__nv_bfloat16>(ctx, X, Yset, Cmat, dm, 0, 0, qk_scale, prep, out, ws, true);
}

// params_out = params with alpha added to the diagonals of C1 and C2: exp(alpha |x|^2) f(w, x) is the DERF with
// C + alpha I (Section 2.3's reduction of K^(alpha) to K^(0)).
namespace {
__global__ void shift_c_kernel(const double* __restrict__ params, double* __restrict__ out, int d, double alpha, size_t total) {
  const size_t g = blockIdx.x;
  ParamsLayout pl{d};
  for (size_t e = threadIdx.x; e < total; e += blockDim.x) {
    double v = params[g * total + e];
    if (e >= pl.C(1) && e < pl.tail()) {
      const size_t r = (e - pl.C(1)) % pl.dd();
      if (r / d == r % d) v += alpha;
    }
    out[g * total + e] = v;
  }
}
}  // namespace
int fs_shift_c(fsharp_ctx* ctx, const double* params, double* out, int G, int d, double alpha) {
  if (G == 0) return FSHARP_OK;
  shift_c_kernel<<<G, 256, 0, ctx->stream>>>(params, out, d, alpha, ParamsLayout{d}.total());
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
