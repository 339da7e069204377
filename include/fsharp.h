/*
 * fsharp.h -- C ABI of the FAVOR# hot path on one NVIDIA B200 (sm_100a).
 *
 * FAVOR# approximates softmax attention with dense exponential random
 * features (DERFs, Section 4 of the paper):
 *
 *   f^(k)(w, x) = D exp(w^T A w + w^T B^(k) x + x^T C^(k) x),  k = 1 (queries), 2 (keys)
 *   P_i = M^-1/2 (f^(1)(w_m, x_i))_m,   S_j = M^-1/2 (f^(2)(w_m, y_j))_m       (Section 2.1)
 *   Y   = diag(P S^T 1)^-1 P S^T V                                              (Section 2.2)
 *
 * The calls follow the paper's statement of the problem:
 *   fsharp_stats          set statistics M1, M2, mu4, mu5 of Theorems 4.2 / 4.3
 *   fsharp_fit_params     closed-form optimal A, B, C, D per parameter group
 *   fsharp_featurize      P or S for given parameters
 *   fsharp_attend         Y, bidirectional or causal (lower-triangular mask)
 *   fsharp_attend_backward  dQ, dK, dV for a cotangent dY of that Y
 *   fsharp_pair_estimate  Khat(x, y) for pairs, with Theorem 4.1's variance
 *   fsharp_kernel_apply   the unnormalised operator Khat^(alpha) C (softmax and Gaussian kernels)
 *   fsharp_attend_key_state, fsharp_attend_with_state   the same Y with the keys of a sequence spread over
 *                         several calls or devices (key-side sums of disjoint key ranges add)
 *
 * Conventions common to every call
 *   - All data pointers are DEVICE pointers owned by the caller unless the
 *     parameter is documented as host memory.  The library neither frees them
 *     nor keeps them after the call's work has finished on the stream.
 *   - Work is enqueued on the context's stream and the call returns without
 *     waiting, except where stated.
 *   - Tensors are addressed through element strides (batch, head, token); the
 *     innermost dimension (d, dv or M) is contiguous.  A stride triple of
 *     zeros means dense [B, H, L, inner].
 *   - Every function returns 0 on success or a negative FSHARP_E_* code.
 *     Nothing aborts, throws or traps.  Conditions found on the device
 *     (non-finite input, singular M1/M2, 8A not below I, a bounded wait that
 *     ran out) are latched in a device status word read by fsharp_status().
 *   - x = qk_scale * Q_i and y = qk_scale * K_j.  Section 2.2 uses
 *     qk_scale = d^-1/4; pass 1 if the tensors already hold x and y.
 *   - Supported shapes: d, dv in {16, 32, 64, 128}; M a multiple of 16, at
 *     most 1024; causal needs Lq == Lk and chunk in {64, 128, 256} dividing L.
 */
#ifndef FSHARP_H
#define FSHARP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fsharp_ctx fsharp_ctx;

enum {
  FSHARP_OK = 0,
  FSHARP_E_BADARG = -1,     /* null pointer, unknown enum value */
  FSHARP_E_SHAPE = -2,      /* unsupported or inconsistent sizes */
  FSHARP_E_ALIGN = -3,      /* base pointer or stride not 16-byte aligned */
  FSHARP_E_DTYPE = -4,
  FSHARP_E_NOMEM = -5,      /* workspace allocation failed */
  FSHARP_E_CONSTRAINT = -6, /* Theorem 4.1 / 4.2 preconditions violated (device-detected) */
  FSHARP_E_NONFINITE = -7,  /* NaN or Inf met on the device */
  FSHARP_E_TIMEOUT = -8,    /* a bounded device-side wait expired */
  FSHARP_E_CUDA = -9,       /* a CUDA runtime or driver call failed */
  FSHARP_E_LIMIT = -10,     /* problem needs more than the fixed scratch of fsharp_featurize_static, or more key
                             * states than one query-side launch merges */
  FSHARP_E_INTERNAL = -11   /* an index check of the debug build (-DFSHARP_DEBUG) failed on the device */
};

enum { FSHARP_F32 = 0, FSHARP_BF16 = 1 };
enum { FSHARP_POSRF = 0, FSHARP_GERF = 1, FSHARP_SADERF = 2, FSHARP_ADERF = 3, FSHARP_SDERF = 4 };
enum { FSHARP_POOL_PER_BH = 0, FSHARP_POOL_PER_HEAD = 1 };
enum { FSHARP_STAB_NONE = 0, FSHARP_STAB_ROW = 1, FSHARP_STAB_GROUP = 2 };
enum { FSHARP_IMPL_AUTO = 0, FSHARP_IMPL_SIMT = 1, FSHARP_IMPL_TENSOR = 2 };

/* Problem sizes and addressing.  G, the number of parameter groups, is B*H for
 * pool == FSHARP_POOL_PER_BH (one operator instance per group, as Theorems 4.2
 * and 4.3 define the statistics) and H for FSHARP_POOL_PER_HEAD (statistics
 * pooled over the batch).  Group of (b, h): b*H + h, respectively h. */
typedef struct {
  int32_t B, H, Lq, Lk, d, dv, M;
  int32_t pool;
  int64_t q_stride[3];        /* element strides of Q: batch, head, token */
  int64_t k_stride[3];
  int64_t v_stride[3];
  int64_t y_stride[3];
  int64_t omega_head_stride;  /* elements between the Omegas of two heads; 0 = one shared Omega */
} fsharp_dims;

/* ---- context ------------------------------------------------------------ */

/* Creates a context on CUDA device `device` that enqueues on `stream`
 * (a cudaStream_t passed as void*; NULL = the legacy default stream).
 * The context owns a scratch workspace in device memory that grows on demand
 * (growing synchronises the stream) and a device status word. */
int fsharp_create(fsharp_ctx** out, int device, void* stream);
int fsharp_destroy(fsharp_ctx* ctx);
int fsharp_set_stream(fsharp_ctx* ctx, void* stream);
/* Forces a kernel family for fsharp_attend and fsharp_featurize (FSHARP_IMPL_*).  AUTO picks the
 * tensor-core kernels when the shape allows it: bf16, d = dv = 64, M = 256 (attend, bidirectional or causal with
 * Lq == Lk; featurize with a row shift or none).  bf16 tensors with d = 128 have no fused kernel: under AUTO their
 * statistics, the exponents' product and, for causal attention with dv = 128, M a multiple of 128 and chunk 128 or 256,
 * the in-chunk scores, the per-chunk key-side sums and the query side run as separate tensor-core kernels, the rest
 * (shift and exponential, scan over chunks) on the fp32 kernels.  Everything else runs on the fp32 kernels.  TENSOR
 * refuses (FSHARP_E_SHAPE) what the fused tensor-core kernels do not cover; SIMT forces the fp32 kernels throughout. */
int fsharp_set_impl(fsharp_ctx* ctx, int impl);
/* Synchronises the stream, then returns the latched device status in *code
 * (0 or a negative FSHARP_E_*), and clears it. */
int fsharp_status(fsharp_ctx* ctx, int* code);
/* Number of kernels this context has launched since creation. */
int64_t fsharp_launch_count(const fsharp_ctx* ctx);
/* Per-kernel device times.  While timing is on, every launch of this context is
 * bracketed by a pair of CUDA events on the context's stream (up to 4096 launches
 * between two reads).  fsharp_read_timing synchronises the stream and returns, for
 * kernel ids 0..cap-1, the summed milliseconds and the launch count since the last
 * read (host arrays of `cap` entries); fsharp_kernel_name maps an id to the kernel's
 * name ("" for unused ids).  Ids are below 32. */
int fsharp_set_timing(fsharp_ctx* ctx, int on);
int fsharp_read_timing(fsharp_ctx* ctx, int cap, float* total_ms, int* launches);
const char* fsharp_kernel_name(int id);
/* Self-test of the bounded device-side waits (no counterpart in the paper): launches a one-warp kernel that waits, with
 * a limit of `limit_us` microseconds (1 .. 100000), on a barrier that nothing ever completes.  The wait gives up,
 * the kernel returns, and the next fsharp_status() reports FSHARP_E_TIMEOUT; the context stays usable. */
int fsharp_selftest_bounded_wait(fsharp_ctx* ctx, int limit_us);
/* Bytes of scratch the context currently holds. */
size_t fsharp_workspace_bytes(const fsharp_ctx* ctx);
const char* fsharp_strerror(int code);

/* ---- layouts of the two fp64 blobs ---------------------------------------- */

/* Doubles per group in the statistics blob:
 *   [M1 (d*d, row-major)] [M2 (d*d)] [mu4 (d)] [mu5 (d)]  = 2 d^2 + 2 d. */
size_t fsharp_stats_doubles(int d);
/* Doubles per group in the parameter blob:
 *   [A (d*d, symmetric)] [B1 (d*d)] [B2 (d*d)] [C1 (d*d)] [C2 (d*d)]
 *   [logD] [objective] [phi] [Jacobi sweeps spent by the fit] [4 reserved, zero]
 * = 5 d^2 + 8.  objective is the shifted log-variance of Section 3.1 at the
 * optimum (Theorems 4.2 / 4.3); phi is the argument of Lemma A.1 (ADERF, GERF,
 * SADERF; for SDERF the largest eigenvalue of N).  Only A, B, C and logD enter the
 * features; a caller may write a blob by hand (e.g. PosRF: A = 0, B = I, C = -I/2). */
size_t fsharp_params_doubles(int d);

/* ---- the path -------------------------------------------------------------- */

/* Statistics of Theorem 4.2 (M1 = L^-1 sum x x^T, M2 likewise for y) and Theorem
 * 4.3 (mu4 = mean x, mu5 = mean y) for every group, from Q [B,H,Lq,d] and
 * K [B,H,Lk,d] of type `dtype`.  stats: device, G * fsharp_stats_doubles(d). */
int fsharp_stats(fsharp_ctx* ctx, const void* Q, const void* K, const fsharp_dims* dims,
                 int dtype, float qk_scale, double* stats);

/* Closed-form minimisers of the shifted log-variance objective (Section 3.1):
 * PosRF and GERF (Section 2.3 / 3.1), SADERF (Section 4.3), ADERF (Theorem 4.2),
 * SDERF (Theorem 4.3), all through Lemma A.1's scalar map.  The symmetric
 * eigenproblems are solved on the device in fp64, one thread block per group
 * (d <= 64: tridiagonalisation, Sturm multisection and twisted-factorisation vectors,
 * confirmed by a cyclic Jacobi solver; d = 128: the Jacobi solver).  ADERF factors
 * M1 = L L^T (Cholesky) and solves one eigenproblem, of L^T M2 L: its eigenvectors
 * and eigenvalues are U and Sigma^2 of the theorem's SVD for the factor L^T of M1
 * (any factor F with F^T F = M1 gives the same B1, B2).  The literal B is "one of
 * the solutions" of the theorems (eigenvector signs and rotations inside equal
 * eigenvalues are free); there is no second, canonical form of the parameters.
 * ridge >= 0 adds ridge * tr(M)/d * I to M1 and M2 first (0 = the paper's formulas).
 * stats: device, G groups.  params: device, G * fsharp_params_doubles(d). */
int fsharp_fit_params(fsharp_ctx* ctx, const double* stats, int G, int d, int variant,
                      double ridge, double* params);

/* P (side = 1, parameters B1, C1) or S (side = 2, B2, C2) of Section 2.1 for the
 * DERF of Section 4: phi[b,h,i,m] * exp(logscale) = M^-1/2 D exp(w_m^T A w_m +
 * w_m^T B x_i + x_i^T C x_i).  X is addressed with (Lq, q_stride) for side 1 and
 * (Lk, k_stride) for side 2.  Omega: float32 [M, d] (or [H, M, d]).
 * phi: float32, dense [B,H,L,M].  logscale: float32, [B,H,L] for FSHARP_STAB_ROW,
 * [B,H] for FSHARP_STAB_GROUP, ignored (may be NULL) for FSHARP_STAB_NONE.
 * ROW shifts by the row's largest exponent, GROUP by the largest exponent of the whole
 * (batch, head), so phi <= 1 in both; any per-row factor on queries and any per-(batch,
 * head) factor on keys cancels in Section 2.2's normalisation. */
int fsharp_featurize(fsharp_ctx* ctx, const void* X, const float* Omega, const double* params,
                     int side, const fsharp_dims* dims, int dtype, float qk_scale, int stab,
                     float* phi, float* logscale);

/* (No counterpart in the paper: an integration aid.)  fsharp_featurize for callers that
 * cannot allocate device memory when they need features -- code running under a memory
 * pool that forbids foreign allocations, latency-critical loops that must not enter the
 * allocator (its locks, its implicit synchronisation), processes whose HBM is already fully
 * committed.  It takes no context and calls no cudaMalloc / cudaFree or any other allocating
 * routine: its scratch is a fixed array of fsharp_static_scratch_bytes() (8 MiB) inside the
 * loaded module, which every GPU that loads the library holds until the process exits.
 * Arguments as fsharp_featurize, plus the stream (cudaStream_t as void*) and an optional
 * device status word (device int*, may be NULL) that receives FSHARP_E_NONFINITE.
 * The scratch must hold G*2*(M*d + M + 8 + d*d) + B*H*L + B*H 4-byte words (each block
 * rounded up to 256 bytes); larger problems are refused with FSHARP_E_LIMIT and nothing runs.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress)
 * and, under lazy module loading, is also when the driver materialises the array; make
 * that first call before any stream capture begins.  All calls share the one array and
 * it keeps whatever the last call left in it; each call writes every word it later reads,
 * so stale contents are harmless, but two calls whose kernels may overlap on the GPU
 * (different streams, or different host threads) race on it: serialise them.
 * The work is launched on the CURRENT device: make the device that holds X current before the call.
 * With device_status == NULL a non-finite value met on the device is not reported anywhere. */
size_t fsharp_static_scratch_bytes(void);
int fsharp_featurize_static(void* stream, const void* X, const float* Omega, const double* params,
                            int side, const fsharp_dims* dims, int dtype, float qk_scale, int stab,
                            float* phi, float* logscale, int* device_status);

/* Y [B,H,Lq,dv] (type `dtype`) of Section 2.2 with Khat = P S^T in place of the
 * exact kernel matrix, evaluated as P (S^T [V | 1]) (Section 2.1's O(L M n) order).
 * causal != 0 restricts key j to j <= i and evaluates chunk by chunk with a running
 * prefix of S^T [V | 1]; chunk is ignored when causal == 0. */
int fsharp_attend(fsharp_ctx* ctx, const void* Q, const void* K, const void* V,
                  const float* Omega, const double* params, const fsharp_dims* dims,
                  int dtype, int causal, int chunk, float qk_scale, void* Y);

/* Backward pass of fsharp_attend (Section 5.3 trains Transformers through the attention of Section 2.2): with
 * Y = fsharp_attend(Q, K, V) and a cotangent dY [B,H,Lq,dv] (y_stride), writes the gradients of sum(dY * Y):
 * dQ [B,H,Lq,d] (q_stride), dK [B,H,Lk,d] (k_stride), dV [B,H,Lk,dv] (v_stride), all of type `dtype`.  Omega and the
 * fitted parameters are constants of the differentiation (no gradient flows through the statistics or the fit).
 * With [num | den]_i = P_i KV_i, G_i = [dY_i / den_i | -(dY_i . Y_i) / den_i] and R_j the sum of P_i G_i^T over the
 * queries i that see key j:  dlogP_i = (G_i KV_i^T) * P_i,  dlogS_j = ([V_j | 1] R_j^T) * S_j,  dV_j = S_j R_j[:, :dv],
 * and, the exponent of Section 4's feature being w^T B x + x^T C x + terms without x,
 * dx = dlog (Omega B) + rowsum(dlog) (C + C^T) x, dQ = qk_scale dx (likewise dK).  causal, chunk, qk_scale and the
 * argument checks are those of fsharp_attend; Q, K, V are read again (nothing is kept from the forward call).
 * fp32 kernels for every shape and both dtypes (bf16 tensors are widened on load, gradients rounded on store).
 * All pointers are device pointers, 16-byte aligned; asynchronous on the context's stream.  A normaliser that is
 * zero or not finite, or a gradient that is not finite, latches FSHARP_E_NONFINITE in the status word. */
int fsharp_attend_backward(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const void* dY,
                           const float* Omega, const double* params, const fsharp_dims* dims, int dtype, int causal,
                           int chunk, float qk_scale, void* dQ, void* dK, void* dV);

/* Sequence-parallel attention.  In Section 2.2's formula the numerator phi(Q) (phi(K)^T V) and the normaliser
 * phi(Q) (phi(K)^T 1) are sums over keys, so the key-side sums S^T [V | 1] of disjoint key ranges add: the keys of
 * one (batch, head) may be spread over several calls, contexts or devices, each of which reduces its range to a
 * "key state", and any holder of all the states of the keys a query may see can finish the query's row.
 * Tensor-core kernels only: dtype FSHARP_BF16, d = dv = 64, M = 256 (anything else: FSHARP_E_SHAPE); all calls that
 * take part must be given the same Omega and params.
 *
 * fsharp_key_state_splits   ns >= 1, the number of pieces a key-state call cuts its key range into (a function of
 *                           dims->B, H, Lk and the device's SM count), or a negative error code.
 * fsharp_attend_key_state   state  [B*H][ns][80][256] fp32 (device, 16-byte aligned): rows 0..64 of piece p are
 *                           sum_j phi(k_j) [v_j | 1]^T over the keys j of piece p, every feature half (128
 *                           features) scaled by 2^-shift; shifts [B*H][ns][2] fp32 (device): those shifts (log2).
 *                           K, V, strides and Lk as in fsharp_attend; Lq and the query strides are ignored.
 * fsharp_attend_with_state  states [B*H][n_states][80][256], shifts [B*H][n_states][2] (device): key states in the
 *                           layout above, concatenated along the piece index in any order.
 *                           causal = 0: Y = attention of Q over exactly the keys behind the states (n_states >= 1;
 *                           K and V are not read and may be null).
 *                           causal = 1: the keys behind the states precede every token of this call (n_states may
 *                           be 0); Y = causal attention of Q over those keys and, with the lower-triangular mask,
 *                           over K, V (Lq == Lk, any length).
 *                           n_states > 64 (causal = 0): FSHARP_E_LIMIT.
 * All pointers are device pointers; the calls are asynchronous on the context's stream like fsharp_attend. */
int fsharp_key_state_splits(fsharp_ctx* ctx, const fsharp_dims* dims);
int fsharp_attend_key_state(fsharp_ctx* ctx, const void* K, const void* V, const float* Omega, const double* params,
                            const fsharp_dims* dims, int dtype, float qk_scale, float* state, float* shifts);
int fsharp_attend_with_state(fsharp_ctx* ctx, const void* Q, const void* K, const void* V, const float* Omega,
                             const double* params, const fsharp_dims* dims, int dtype, int causal, float qk_scale,
                             const float* states, const float* shifts, int n_states, void* Y);

/* The unnormalised operator of Section 2.1: out = Khat^(alpha)(X, Y) C, the O(L M n) evaluation P (S^T C) of
 * K^(alpha)(x, y) = exp(alpha |x|^2 + x^T y + alpha |y|^2) applied to a matrix C, with the features
 * fhat = exp(alpha |x|^2) f of Section 2.3 (alpha = 0: softmax kernel; alpha = -1/2: Gaussian kernel).
 * X [B,H,Lq,d] (q_stride), Y [B,H,Lk,d] (k_stride), C [B,H,Lk,dv] (v_stride), out [B,H,Lq,dv] (y_stride), all of
 * type `dtype`; Omega and params as for fsharp_attend.  Nothing is normalised, so out carries the scale of the
 * kernel values (bf16 keeps the range, at 8 bits of precision).  Runs on the fp32 kernels for every shape.
 * Lk = 0 is refused (FSHARP_E_SHAPE). */
int fsharp_kernel_apply(fsharp_ctx* ctx, const void* X, const void* Y, const void* C, const float* Omega,
                        const double* params, double alpha, const fsharp_dims* dims, int dtype, float qk_scale,
                        void* out);

/* The whole path on HOST buffers: copies Q, K, V (dense [B,H,L,*], type `dtype`)
 * to the device, runs stats -> fit -> attend, copies Y back and waits for it.
 * Q, K, V, Y: host memory (pinned memory makes the copies asynchronous).
 * Omega: host float32 [M, d].  dims' strides are ignored (dense).
 * With one parameter group per (batch, head) the batch elements go through one after the other: the upload of one, the
 * path on the one before and the download of the one before that overlap (three streams owned by the context). */
int fsharp_forward_host(fsharp_ctx* ctx, const void* Q, const void* K, const void* V,
                        const float* Omega, const fsharp_dims* dims, int dtype, int variant,
                        int causal, int chunk, float qk_scale, void* Y);

/* Kernel estimates for npairs (x_p, y_p) pairs (Section 2.1: Khat = sum_m P_pm S_pm)
 * with R independent feature draws: X, Y float32 [npairs, d]; Omega float32
 * [R, M, d]; params: one group; est: float32 [R, npairs].  If var_cf is not NULL it
 * receives, per pair, Theorem 4.1's variance divided by M (needs a diagonal A).
 * If pooled is not NULL (device, 2 doubles; needs var_cf) it receives the two pooled numbers of
 * the variance study (Section 5.1) for this parameterisation: the mean over pairs of the unbiased
 * sample variance of the R estimates over K^2, and the mean over pairs of var_cf over K^2, with
 * K = exp(x^T y). */
int fsharp_pair_estimate(fsharp_ctx* ctx, const float* X, const float* Y, const float* Omega,
                         const double* params, int64_t npairs, int d, int M, int R,
                         float* est, double* var_cf, double* pooled);

#ifdef __cplusplus
}
#endif
#endif /* FSHARP_H */
