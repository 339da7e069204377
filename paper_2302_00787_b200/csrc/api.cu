// C-ABI entry points: argument checks, workspace sizing and dispatch to the kernel families.
#include <math.h>

#include "common.cuh"
#include "tc_layout.cuh"

// tensor-core path (tc_*.cu)
int fs_tc_supported(const fsharp_dims* dm, int dtype, int causal, int chunk, float qk_scale);
size_t fs_tc_attend_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm, int causal, int chunk);
int fs_tc_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, int causal,
                 int chunk, const uint8_t* images, const int* flags, void* Y, WsAlloc* ws);
int fs_tc_featurize_supported(const fsharp_dims* dm, int dtype, int stab);
int fs_tc_key_state_splits(const fsharp_ctx* ctx, const fsharp_dims* dm, int* tiles_per_split);
size_t fs_tc_key_state_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm);
int fs_tc_key_state(fsharp_ctx* ctx, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                    const int* flags, float* state, float* shifts, WsAlloc* ws);
int fs_tc_query_side(fsharp_ctx* ctx, const void* Q, const fsharp_dims* dm, const uint8_t* images, const float* partial,
                     const float* shifts, int nsplit, void* Y);
size_t fs_tc_causal_prefix_scratch_bytes(const fsharp_ctx* ctx, const fsharp_dims* dm, int nprefix);
int fs_tc_causal_prefix(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const fsharp_dims* dm, const uint8_t* images,
                        const int* flags, const float* pre_state, const float* pre_shifts, int nprefix, void* Y, WsAlloc* ws);
size_t fs_tc_featurize_scratch_bytes(const fsharp_dims* dm, int side);
int fs_tc_featurize(fsharp_ctx* ctx, const void* X, const fsharp_dims* dm, int side, int stab, const float* prep,
                    const uint8_t* images, const int* flags, float* phi, float* logscale, WsAlloc* ws);

namespace {

bool dim_ok(int d) { return d == 16 || d == 32 || d == 64 || d == 128; }

int check_dims(const fsharp_dims* dm, bool need_v) {
  if (!dm) return FSHARP_E_BADARG;
  if (dm->B < 0 || dm->H < 0 || dm->Lq < 0 || dm->Lk < 0) return FSHARP_E_SHAPE;
  if (!dim_ok(dm->d)) return FSHARP_E_SHAPE;
  if (need_v && !dim_ok(dm->dv)) return FSHARP_E_SHAPE;
  if (dm->M <= 0 || dm->M % 16 != 0 || dm->M > 1024) return FSHARP_E_SHAPE;
  if (dm->pool != FSHARP_POOL_PER_BH && dm->pool != FSHARP_POOL_PER_HEAD) return FSHARP_E_BADARG;
  if ((int64_t)dm->B * dm->H > 65535) return FSHARP_E_SHAPE;
  return FSHARP_OK;
}

int check_ptr(const void* p, int dtype, const int64_t s[3]) {
  if (!p) return FSHARP_E_BADARG;
  const size_t es = dtype == FSHARP_F32 ? 4 : 2;
  if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return FSHARP_E_ALIGN;
  for (int i = 0; i < 3; i++)
    if (s[i] < 0 || (s[i] * es) % 16 != 0) return FSHARP_E_ALIGN;
  return FSHARP_OK;
}

bool dtype_ok(int dtype) { return dtype == FSHARP_F32 || dtype == FSHARP_BF16; }

}  // namespace

extern "C" {

int fsharp_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dims, int dtype,
                 float qk_scale, double* stats) {
  FS_RANGE("fsharp_stats");
  if (!ctx) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, false));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (dims->B * dims->H == 0) return FSHARP_OK;
  if (!stats) return FSHARP_E_BADARG;
  FS_TRY(check_ptr(Q, dtype, dims->q_stride));
  FS_TRY(check_ptr(K, dtype, dims->k_stride));
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  return fs_run_stats(ctx, Q, K, dims, dtype, qk_scale, stats);
}

int fsharp_fit_params(fsharp_ctx* ctx, const double* stats, int G, int d, int variant, double ridge,
                      double* params) {
  FS_RANGE("fsharp_fit_params");
  if (!ctx || !stats || !params) return FSHARP_E_BADARG;
  if (G < 0 || !dim_ok(d)) return FSHARP_E_SHAPE;
  if (variant < FSHARP_POSRF || variant > FSHARP_SDERF) return FSHARP_E_BADARG;
  if (!(ridge >= 0.0)) return FSHARP_E_BADARG;
  if (G == 0) return FSHARP_OK;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  size_t need = ws_round(fs_fit_scratch_doubles(G, d) * sizeof(double));
  FS_TRY(fs_ws_reserve(ctx, need));
  return fs_run_fit(ctx, stats, G, d, variant, ridge, params, reinterpret_cast<double*>(ctx->ws));
}

int fsharp_featurize(fsharp_ctx* ctx, const void* X, const float* Omega, const double* params, int side,
                     const fsharp_dims* dims, int dtype, float qk_scale, int stab, float* phi, float* logscale) {
  FS_RANGE("fsharp_featurize");
  if (!ctx || !Omega || !params || !phi) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, false));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (side != 1 && side != 2) return FSHARP_E_BADARG;
  if (stab < FSHARP_STAB_NONE || stab > FSHARP_STAB_GROUP) return FSHARP_E_BADARG;
  if (stab != FSHARP_STAB_NONE && !logscale) return FSHARP_E_BADARG;
  const int L = side == 1 ? dims->Lq : dims->Lk;
  const int64_t* st = side == 1 ? dims->q_stride : dims->k_stride;
  if (dims->B * dims->H == 0 || L == 0) return FSHARP_OK;
  FS_TRY(check_ptr(X, dtype, st));
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  // tensor-core kernel (bf16, d = 64, M = 256, row shift or none, dense phi), unless the fp32 kernels are forced
  bool use_tc = false;
  if (ctx->impl != FSHARP_IMPL_SIMT) {
    use_tc = fs_tc_featurize_supported(dims, dtype, stab) != 0;
    if (!use_tc && ctx->impl == FSHARP_IMPL_TENSOR) return FSHARP_E_SHAPE;
  }
  if (use_tc) {
    FS_TRY(fs_ws_reserve(ctx, ws_round(prep_f * 4) + fs_tc_featurize_scratch_bytes(dims, side)));
    WsAlloc wst{ctx->ws, 0};
    float* prep_t = wst.take<float>(prep_f);
    uint8_t* images = wst.take<uint8_t>((size_t)G * 2 * tcl::IMG_BYTES);
    int* flags = wst.take<int>((size_t)G * 2 * tcl::FLAG_WORDS + 16);
    FS_TRY(fs_run_prep_images(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                              dims->H, dims->pool, dims->d, dims->M, prep_t, qk_scale, images, flags));
    return fs_tc_featurize(ctx, X, dims, side, stab, prep_t, images, flags, phi, logscale, &wst);
  }
  const size_t need = ws_round(prep_f * 4) + ws_round((size_t)dims->B * dims->H * L * 4) +
                      ws_round((size_t)dims->B * dims->H * 4);
  FS_TRY(fs_ws_reserve(ctx, need));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  float* rowc = ws.take<float>((size_t)dims->B * dims->H * L);
  unsigned* gmax = ws.take<unsigned>((size_t)dims->B * dims->H);
  FS_TRY(fs_run_prep(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                     dims->H, dims->pool, dims->d, dims->M, prep));
  return fs_simt_featurize(ctx, X, dtype, fs_addr(st, dims->H, L, dims->d), dims->B, dims->H, L, dims->d, dims->M,
                           dims->pool, prep, side, qk_scale, stab, rowc, gmax, phi, logscale);
}

int fsharp_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const float* Omega,
                  const double* params, const fsharp_dims* dims, int dtype, int causal, int chunk, float qk_scale,
                  void* Y) {
  FS_RANGE("fsharp_attend");
  if (!ctx || !Omega || !params) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (causal) {
    if (dims->Lq != dims->Lk) return FSHARP_E_SHAPE;
    if (chunk != 64 && chunk != 128 && chunk != 256) return FSHARP_E_SHAPE;
    if (dims->Lq % chunk != 0) return FSHARP_E_SHAPE;
  }
  if (dims->B * dims->H == 0 || dims->Lq == 0) return FSHARP_OK;
  if (dims->Lk == 0) return FSHARP_E_SHAPE;   // no key: the normaliser of Section 2.2 is zero
  FS_TRY(check_ptr(Q, dtype, dims->q_stride));
  FS_TRY(check_ptr(K, dtype, dims->k_stride));
  FS_TRY(check_ptr(V, dtype, dims->v_stride));
  FS_TRY(check_ptr(Y, dtype, dims->y_stride));
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  bool use_tc = false;
  if (ctx->impl != FSHARP_IMPL_SIMT) {
    use_tc = fs_tc_supported(dims, dtype, causal, chunk, qk_scale) != 0;
    if (!use_tc && ctx->impl == FSHARP_IMPL_TENSOR) return FSHARP_E_SHAPE;
  }
  // the fp32 path indexes (batch, head, chunk) through a grid z coordinate: refuse before anything is launched
  if (!use_tc && causal && (int64_t)dims->B * dims->H * (dims->Lq / chunk) > 65535) return FSHARP_E_SHAPE;
  const size_t need = ws_round(prep_f * 4) + (use_tc ? fs_tc_attend_scratch_bytes(ctx, dims, causal, chunk)
                                                     : fs_simt_attend_scratch_bytes(dims, causal, chunk));
  FS_TRY(fs_ws_reserve(ctx, need));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  if (use_tc) {
    // the prep kernel also writes the tensor-core path's operand images
    uint8_t* images = ws.take<uint8_t>((size_t)G * 2 * tcl::IMG_BYTES);
    int* flags = ws.take<int>((size_t)G * 2 * tcl::FLAG_WORDS + 16);
    FS_TRY(fs_run_prep_images(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                              dims->H, dims->pool, dims->d, dims->M, prep, qk_scale, images, flags));
    return fs_tc_attend(ctx, Q, K, V, dims, causal, chunk, images, flags, Y, &ws);
  }
  FS_TRY(fs_run_prep(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                     dims->H, dims->pool, dims->d, dims->M, prep));
  return fs_simt_attend(ctx, Q, K, V, dims, dtype, causal, chunk, qk_scale, prep, Y, &ws);
}

int fsharp_attend_backward(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const void* dY,
                           const float* Omega, const double* params, const fsharp_dims* dims, int dtype, int causal,
                           int chunk, float qk_scale, void* dQ, void* dK, void* dV) {
  FS_RANGE("fsharp_attend_backward");
  if (!ctx || !Omega || !params) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (causal) {
    if (dims->Lq != dims->Lk) return FSHARP_E_SHAPE;
    if (chunk != 64 && chunk != 128 && chunk != 256) return FSHARP_E_SHAPE;
    if (dims->Lq % chunk != 0) return FSHARP_E_SHAPE;
  }
  if (dims->B * dims->H == 0 || (dims->Lq == 0 && dims->Lk == 0)) return FSHARP_OK;
  if (dims->Lk == 0 || dims->Lq == 0) return FSHARP_E_SHAPE;   // no key: no normaliser; no query: nothing to differentiate
  FS_TRY(check_ptr(Q, dtype, dims->q_stride));
  FS_TRY(check_ptr(K, dtype, dims->k_stride));
  FS_TRY(check_ptr(V, dtype, dims->v_stride));
  FS_TRY(check_ptr(dY, dtype, dims->y_stride));
  FS_TRY(check_ptr(dQ, dtype, dims->q_stride));
  FS_TRY(check_ptr(dK, dtype, dims->k_stride));
  FS_TRY(check_ptr(dV, dtype, dims->v_stride));
  // (batch, head, chunk) is a grid z coordinate
  if (causal && (int64_t)dims->B * dims->H * (dims->Lq / chunk) > 65535) return FSHARP_E_SHAPE;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  FS_TRY(fs_ws_reserve(ctx, ws_round(prep_f * 4) + fs_backward_scratch_bytes(dims, causal, chunk)));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  FS_TRY(fs_run_prep(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                     dims->H, dims->pool, dims->d, dims->M, prep));
  return fs_backward(ctx, Q, K, V, dY, dims, dtype, causal, chunk, qk_scale, prep, dQ, dK, dV, &ws);
}

int fsharp_key_state_splits(fsharp_ctx* ctx, const fsharp_dims* dims) {
  if (!ctx) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (dims->B * dims->H == 0 || dims->Lk <= 0) return FSHARP_E_SHAPE;
  return fs_tc_key_state_splits(ctx, dims, nullptr);
}

int fsharp_attend_key_state(fsharp_ctx* ctx, const void* K, const void* V, const float* Omega, const double* params,
                            const fsharp_dims* dims, int dtype, float qk_scale, float* state, float* shifts) {
  FS_RANGE("fsharp_attend_key_state");
  if (!ctx || !Omega || !params || !state || !shifts) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (dims->B * dims->H == 0 || dims->Lk <= 0) return FSHARP_E_SHAPE;
  // the tensor-core kernels only (bf16, d = dv = 64, M = 256): the state is their key-side sum
  fsharp_dims kd = *dims;
  kd.Lq = kd.Lk;
  for (int i = 0; i < 3; i++) kd.q_stride[i] = kd.k_stride[i];
  if (!fs_tc_supported(&kd, dtype, 0, 0, qk_scale)) return FSHARP_E_SHAPE;
  FS_TRY(check_ptr(K, dtype, dims->k_stride));
  FS_TRY(check_ptr(V, dtype, dims->v_stride));
  if (reinterpret_cast<uintptr_t>(state) % 16 != 0 || reinterpret_cast<uintptr_t>(shifts) % 8 != 0) return FSHARP_E_ALIGN;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  FS_TRY(fs_ws_reserve(ctx, ws_round(prep_f * 4) + fs_tc_key_state_scratch_bytes(ctx, &kd)));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  uint8_t* images = ws.take<uint8_t>((size_t)G * 2 * tcl::IMG_BYTES);
  int* flags = ws.take<int>((size_t)G * 2 * tcl::FLAG_WORDS + 16);
  FS_TRY(fs_run_prep_images(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                            dims->H, dims->pool, dims->d, dims->M, prep, qk_scale, images, flags));
  return fs_tc_key_state(ctx, K, V, &kd, images, flags, state, shifts, &ws);
}

int fsharp_attend_with_state(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const float* Omega,
                             const double* params, const fsharp_dims* dims, int dtype, int causal, float qk_scale,
                             const float* states, const float* shifts, int n_states, void* Y) {
  FS_RANGE("fsharp_attend_with_state");
  if (!ctx || !Omega || !params) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (n_states < 0 || (n_states > 0 && (!states || !shifts))) return FSHARP_E_BADARG;
  if (causal ? dims->Lq != dims->Lk : n_states == 0) return FSHARP_E_SHAPE;   // bidirectional: every key is behind a state
  if (dims->B * dims->H == 0 || dims->Lq == 0) return FSHARP_OK;
  fsharp_dims qd = *dims;
  if (!causal) {                       // K and V are not read: the query tensor stands in for the shape checks
    qd.Lk = qd.Lq;
    for (int i = 0; i < 3; i++) qd.k_stride[i] = qd.v_stride[i] = qd.q_stride[i];
  }
  if (!fs_tc_supported(&qd, dtype, causal, 128, qk_scale)) return FSHARP_E_SHAPE;
  FS_TRY(check_ptr(Q, dtype, dims->q_stride));
  FS_TRY(check_ptr(Y, dtype, dims->y_stride));
  if (causal) {
    FS_TRY(check_ptr(K, dtype, dims->k_stride));
    FS_TRY(check_ptr(V, dtype, dims->v_stride));
  }
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  const size_t img_bytes = ws_round((size_t)G * 2 * tcl::IMG_BYTES) + ws_round((size_t)G * 2 * tcl::FLAG_WORDS * 4 + 64);
  FS_TRY(fs_ws_reserve(ctx, ws_round(prep_f * 4) + img_bytes + (causal ? fs_tc_causal_prefix_scratch_bytes(ctx, &qd, n_states) : 0)));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  uint8_t* images = ws.take<uint8_t>((size_t)G * 2 * tcl::IMG_BYTES);
  int* flags = ws.take<int>((size_t)G * 2 * tcl::FLAG_WORDS + 16);
  FS_TRY(fs_run_prep_images(ctx, Omega, dims->omega_head_stride, params, (int64_t)ParamsLayout{dims->d}.total(), G,
                            dims->H, dims->pool, dims->d, dims->M, prep, qk_scale, images, flags));
  if (causal) return fs_tc_causal_prefix(ctx, Q, K, V, &qd, images, flags, states, shifts, n_states, Y, &ws);
  return fs_tc_query_side(ctx, Q, &qd, images, states, shifts, n_states, Y);
}

int fsharp_kernel_apply(fsharp_ctx* ctx, const void* X, const void* Y, const void* Cmat, const float* Omega,
                        const double* params, double alpha, const fsharp_dims* dims, int dtype, float qk_scale, void* out) {
  FS_RANGE("fsharp_kernel_apply");
  if (!ctx || !Omega || !params) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (!isfinite(alpha)) return FSHARP_E_BADARG;
  if (dims->B * dims->H == 0 || dims->Lq == 0) return FSHARP_OK;
  if (dims->Lk == 0) return FSHARP_E_SHAPE;
  FS_TRY(check_ptr(X, dtype, dims->q_stride));
  FS_TRY(check_ptr(out, dtype, dims->y_stride));
  FS_TRY(check_ptr(Y, dtype, dims->k_stride));
  FS_TRY(check_ptr(Cmat, dtype, dims->v_stride));
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  const int G = fs_groups(dims);
  const size_t prep_f = (size_t)G * 2 * PrepLayout{dims->d, dims->M}.total();
  const size_t np = (size_t)G * ParamsLayout{dims->d}.total();
  FS_TRY(fs_ws_reserve(ctx, ws_round(prep_f * 4) + ws_round(np * 8) + fs_simt_attend_scratch_bytes(dims, 0, 0)));
  WsAlloc ws{ctx->ws, 0};
  float* prep = ws.take<float>(prep_f);
  double* shifted = ws.take<double>(np);
  FS_TRY(fs_shift_c(ctx, params, shifted, G, dims->d, alpha));
  FS_TRY(fs_run_prep(ctx, Omega, dims->omega_head_stride, shifted, (int64_t)ParamsLayout{dims->d}.total(), G, dims->H,
                     dims->pool, dims->d, dims->M, prep));
  return fs_simt_kernel_apply(ctx, X, Y, Cmat, dims, dtype, qk_scale, prep, out, &ws);
}

int fsharp_forward_host(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const float* Omega,
                        const fsharp_dims* dims, int dtype, int variant, int causal, int chunk, float qk_scale,
                        void* Y) {
  FS_RANGE("fsharp_forward_host");
  if (!ctx || !Q || !K || !V || !Omega || !Y) return FSHARP_E_BADARG;
  FS_TRY(check_dims(dims, true));
  if (!dtype_ok(dtype)) return FSHARP_E_DTYPE;
  if (variant < FSHARP_POSRF || variant > FSHARP_SDERF) return FSHARP_E_BADARG;
  if (dims->omega_head_stride != 0) return FSHARP_E_BADARG;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  fsharp_dims dd = *dims;
  for (int i = 0; i < 3; i++) dd.q_stride[i] = dd.k_stride[i] = dd.v_stride[i] = dd.y_stride[i] = 0;
  const size_t es = dtype == FSHARP_F32 ? 4 : 2;
  const size_t BH = (size_t)dd.B * dd.H;
  const size_t nq = BH * dd.Lq * dd.d * es, nk = BH * dd.Lk * dd.d * es, nv = BH * dd.Lk * dd.dv * es;
  const size_t ny = BH * dd.Lq * dd.dv * es, no = (size_t)dd.M * dd.d * 4;
  if (ny == 0) return FSHARP_OK;
  const int G = fs_groups(&dd);
  const size_t nstats = (size_t)G * StatsLayout{dd.d}.total() * 8, nparams = (size_t)G * ParamsLayout{dd.d}.total() * 8;
  // The staging buffers live at the END of the workspace so that the nested calls, which
  // carve their scratch from the start, do not overlap them.
  const size_t stage = ws_round(nq) + ws_round(nk) + ws_round(nv) + ws_round(ny) + ws_round(no) + ws_round(nstats) +
                       ws_round(nparams);
  const int G2 = G;
  size_t inner = ws_round((size_t)G2 * 2 * PrepLayout{dd.d, dd.M}.total() * 4);
  {
    size_t a = fs_simt_attend_scratch_bytes(&dd, causal, chunk);
    size_t b = fs_tc_supported(&dd, dtype, causal, chunk, qk_scale) ? fs_tc_attend_scratch_bytes(ctx, &dd, causal, chunk) : 0;
    size_t c = ws_round(fs_fit_scratch_doubles(G, dd.d) * 8);
    size_t use = ctx->impl == FSHARP_IMPL_SIMT ? a : (b ? b : a);
    inner += use > c ? use : c;
  }
  FS_TRY(fs_ws_reserve(ctx, inner + stage + 256));
  WsAlloc ws{ctx->ws, (ctx->ws_bytes - stage) & ~(size_t)255};
  char* dQ = ws.take<char>(nq);
  char* dK = ws.take<char>(nk);
  char* dV = ws.take<char>(nv);
  char* dY = ws.take<char>(ny);
  float* dO = ws.take<float>((size_t)dd.M * dd.d);
  double* dS = ws.take<double>(nstats / 8);
  double* dP = ws.take<double>(nparams / 8);
  if (!ctx->copy_stream) {
    FS_CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    FS_CUDA_OK(cudaStreamCreateWithFlags(&ctx->down_stream, cudaStreamNonBlocking));
    FS_CUDA_OK(cudaEventCreateWithFlags(&ctx->ev_inputs, cudaEventDisableTiming));
    FS_CUDA_OK(cudaEventCreateWithFlags(&ctx->ev_v, cudaEventDisableTiming));
  }
  // With one parameter group per (batch, head) the batch elements are independent all the way: element b's inputs go up
  // on the upload stream while element b - 1 runs on the context's stream and element b - 2's rows come down on the
  // download stream.  (An event may be recorded again while an earlier wait on it is pending: a wait refers to the
  // record that preceded it.)  Pooled groups (one per head over the whole batch) make one piece of the whole batch.
  const int pieces = dd.pool == FSHARP_POOL_PER_BH ? dd.B : 1;
  fsharp_dims dp = dd;
  dp.B = dd.B / pieces;
  const size_t f = (size_t)pieces;
  const int Gp = G / pieces;
  // the uploads start when the stream's earlier work (which may still read the staging buffers) has finished
  FS_CUDA_OK(cudaEventRecord(ctx->ev_inputs, ctx->stream));
  FS_CUDA_OK(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_inputs, 0));
  FS_CUDA_OK(cudaStreamWaitEvent(ctx->down_stream, ctx->ev_inputs, 0));
  FS_CUDA_OK(cudaMemcpyAsync(dO, Omega, no, cudaMemcpyHostToDevice, ctx->copy_stream));
  for (int p = 0; p < pieces; p++) {
    const char* hQ = static_cast<const char*>(Q) + p * (nq / f);
    const char* hK = static_cast<const char*>(K) + p * (nk / f);
    const char* hV = static_cast<const char*>(V) + p * (nv / f);
    char *pQ = dQ + p * (nq / f), *pK = dK + p * (nk / f), *pV = dV + p * (nv / f), *pY = dY + p * (ny / f);
    double* pS = dS + (size_t)p * Gp * StatsLayout{dd.d}.total();
    double* pP = dP + (size_t)p * Gp * ParamsLayout{dd.d}.total();
    FS_CUDA_OK(cudaMemcpyAsync(pQ, hQ, nq / f, cudaMemcpyHostToDevice, ctx->copy_stream));
    FS_CUDA_OK(cudaMemcpyAsync(pK, hK, nk / f, cudaMemcpyHostToDevice, ctx->copy_stream));
    FS_CUDA_OK(cudaEventRecord(ctx->ev_inputs, ctx->copy_stream));
    FS_CUDA_OK(cudaMemcpyAsync(pV, hV, nv / f, cudaMemcpyHostToDevice, ctx->copy_stream));
    FS_CUDA_OK(cudaEventRecord(ctx->ev_v, ctx->copy_stream));
    FS_CUDA_OK(cudaStreamWaitEvent(ctx->stream, ctx->ev_inputs, 0));
    FS_TRY(fsharp_stats(ctx, pQ, pK, &dp, dtype, qk_scale, pS));
    FS_TRY(fsharp_fit_params(ctx, pS, Gp, dd.d, variant, 0.0, pP));
    FS_CUDA_OK(cudaStreamWaitEvent(ctx->stream, ctx->ev_v, 0));
    FS_TRY(fsharp_attend(ctx, pQ, pK, pV, dO, pP, &dp, dtype, causal, chunk, qk_scale, pY));
    FS_CUDA_OK(cudaEventRecord(ctx->ev_v, ctx->stream));
    FS_CUDA_OK(cudaStreamWaitEvent(ctx->down_stream, ctx->ev_v, 0));
    FS_CUDA_OK(cudaMemcpyAsync(static_cast<char*>(Y) + p * (ny / f), pY, ny / f, cudaMemcpyDeviceToHost, ctx->down_stream));
  }
  FS_CUDA_OK(cudaStreamSynchronize(ctx->down_stream));
  FS_CUDA_OK(cudaStreamSynchronize(ctx->stream));
  return FSHARP_OK;
}

int fsharp_pair_estimate(fsharp_ctx* ctx, const float* X, const float* Y, const float* Omega, const double* params,
                         int64_t npairs, int d, int M, int R, float* est, double* var_cf, double* pooled) {
  FS_RANGE("fsharp_pair_estimate");
  if (!ctx || !Omega || !params) return FSHARP_E_BADARG;
  if (pooled && !var_cf) return FSHARP_E_BADARG;
  if (npairs < 0 || !dim_ok(d) || M <= 0 || M % 16 != 0 || M > 1024 || R <= 0 || R > 65535) return FSHARP_E_SHAPE;
  if (npairs > 0 && (!X || !Y || !est)) return FSHARP_E_BADARG;
  FS_CUDA_OK(cudaSetDevice(ctx->device));
  FS_TRY(fs_ws_reserve(ctx, fs_pairs_scratch_bytes(d, M, R)));
  WsAlloc ws{ctx->ws, 0};
  return fs_run_pairs(ctx, X, Y, Omega, params, npairs, d, M, R, est, var_cf, pooled, &ws);
}

}  // extern "C"
