// Closed-form parameter fits (Section 3.1, Section 4.3, Theorems 4.2 and 4.3, Lemma A.1), fp64, one thread block
// per parameter group.  Symmetric eigenproblems, d <= 64: Householder tridiagonalisation, Sturm-count multisection,
// one vector per eigenvalue from the twisted factorisation, reflectors applied back, one symmetric orthogonalisation;
// a cyclic Jacobi solver then confirms convergence (or completes it).  d = 128: the Jacobi solver alone.
// ADERF factors M1 by Cholesky (M1 = L L^T) and solves ONE eigenproblem, of L^T M2 L (Theorem 4.2's U and Sigma^2
// for the factor L^T of M1).
#include "common.cuh"

namespace {

constexpr int FIT_THREADS = 512;
constexpr int JACOBI_MAX_SWEEPS = 40;

__device__ __forceinline__ double block_reduce(double v, double* red, int op /*0 sum, 1 max, 2 min*/) {
  const int tid = threadIdx.x;
  __syncthreads();
  red[tid] = v;
  __syncthreads();
  for (int s = FIT_THREADS / 2; s > 0; s >>= 1) {
    if (tid < s) {
      double a = red[tid], b = red[tid + s];
      red[tid] = op == 0 ? a + b : (op == 1 ? fmax(a, b) : fmin(a, b));
    }
    __syncthreads();
  }
  double r = red[0];
  __syncthreads();
  return r;
}

// Lemma A.1 in the cancellation-free form that follows from its proof:
// 1 - 8A = (2 phi + 1 + s)/2 with s = sqrt((2 phi + 1)^2 + 8 phi).
__device__ __forceinline__ double lemma_a1(double phi) {
  double s = sqrt((2.0 * phi + 1.0) * (2.0 * phi + 1.0) + 8.0 * phi);
  return -(2.0 * phi + (12.0 * phi + 4.0 * phi * phi) / (1.0 + s)) / 16.0;
}

// Two-sided cyclic Jacobi with the round-robin ("tournament") ordering: every round rotates
// d/2 disjoint index pairs at once.  On exit the diagonal of A holds the eigenvalues and ROW k
// of VT the k-th eigenvector.  A: d x d, leading dimension lda; VT likewise (ldvt).
// d is a power of two (log2d).  sched: the (d-1) x d/2 pairs of all rounds, filled once per
// block by jacobi_schedule.  cs: 2*d doubles, red: FIT_THREADS doubles (all shared memory).
//
// The rotation angle is computed in fp32 (fast divide and square root) and then (c, s) is made
// orthonormal in fp64: c = rsqrt(1 + t^2), s = t c.  An angle that is only accurate to 1e-7
// still annihilates a_pq to that relative level and keeps V exactly orthogonal; the sweeps
// repeat until the off-diagonal mass is below 1e-24 of the total.
__device__ void jacobi_schedule(ushort2* sched, int d) {
  const int half = d >> 1;
  for (int e = threadIdx.x; e < (d - 1) * half; e += FIT_THREADS) {
    int r = e / half, k = e % half, p, q;
    if (k == 0) { p = r; q = d - 1; }
    else { p = (r + k) % (d - 1); q = (r - k + (d - 1)) % (d - 1); }
    sched[e] = make_ushort2((unsigned short)p, (unsigned short)q);
  }
  __syncthreads();
}

__device__ __forceinline__ int jacobi_eig(double* __restrict__ A, int lda, double* __restrict__ VT, int ldvt, int d,
                                          int log2d, const ushort2* __restrict__ sched, double* __restrict__ cs_base,
                                          double* red) {
  const int tid = threadIdx.x;
  const int half = d >> 1, items = half << log2d, dm1 = d - 1;
  for (int e = tid; e < d * d; e += FIT_THREADS) VT[(e >> log2d) * ldvt + (e & dm1)] = ((e >> log2d) == (e & dm1)) ? 1.0 : 0.0;
  __syncthreads();
  int sweeps = 0;
  for (int sweep = 0; sweep < JACOBI_MAX_SWEEPS; sweep++) {
    double off = 0.0, tot = 0.0;
    for (int e = tid; e < d * d; e += FIT_THREADS) {
      int i = e >> log2d, j = e & dm1;
      double v = A[i * lda + j];
      tot += v * v;
      if (i != j) off += v * v;
    }
    off = block_reduce(off, red, 0);
    tot = block_reduce(tot, red, 0);
    if (off <= 1e-24 * tot || tot == 0.0) break;
    sweeps++;
    // Rotation parameters of round r live in cs[(r & 1) * d ...]; those of round r + 1 are
    // computed by the first d/2 threads while everybody applies round r to VT (VT does not feed
    // the parameters), so their latency is hidden.
    auto rotation_params = [&](int r) {
      const ushort2* sr = sched + r * half;
      double* csr = cs_base + (r & 1) * d;
      const int p = sr[tid].x, q = sr[tid].y;
      const double app = A[p * lda + p], aqq = A[q * lda + q], apq = A[p * lda + q];
      double c = 1.0, s = 0.0;
      const float num = (float)(aqq - app), den = (float)(2.0 * apq);
      if (den != 0.f) {
        const float zeta = __fdividef(num, den);
        const float tf = __fdividef(copysignf(1.f, zeta), fabsf(zeta) + sqrtf(fmaf(zeta, zeta, 1.f)));
        if (isfinite(tf)) {
          const double t = (double)tf;
          const double x = fma(t, t, 1.0);
          const double c0 = (double)rsqrtf(fmaf(tf, tf, 1.f));
          c = c0 * fma(-0.5 * x, c0 * c0, 1.5);       // one Newton step: |c^2 x - 1| ~ 1e-14
          s = t * c;
        }
      }
      csr[2 * tid] = c; csr[2 * tid + 1] = s;
    };
    if (tid < half) rotation_params(0);
    __syncthreads();
    for (int r = 0; r < d - 1; r++) {
      const ushort2* sr = sched + r * half;
      const double* cs = cs_base + (r & 1) * d;
      // A <- J^T A J, one 2 x 2 block per item: block (k, l) holds rows {p_k, q_k} and columns
      // {p_l, q_l}; it is rotated by J_k from the left and J_l from the right in registers, so A
      // is read and written once per round and no barrier separates the two sides.  Blocks of a
      // round are disjoint.  VT <- J^T VT (rows p, q) rides along as further disjoint items.
      const int log2h = log2d - 1;
      const int nblk = half << log2h;                 // (d/2)^2 blocks
      for (int e0 = tid; e0 < nblk; e0 += 2 * FIT_THREADS) {
        double a00[2], a01[2], a10[2], a11[2], ck[2], sk[2], cl[2], sl[2];
        int i00[2], i01[2], i10[2], i11[2];
#pragma unroll
        for (int u = 0; u < 2; u++) {
          const int e = e0 + u * FIT_THREADS;
          if (e < nblk) {
            const int k = e >> log2h, l = e & (half - 1);
            const int pk = sr[k].x, qk = sr[k].y, pl = sr[l].x, ql = sr[l].y;
            ck[u] = cs[2 * k]; sk[u] = cs[2 * k + 1]; cl[u] = cs[2 * l]; sl[u] = cs[2 * l + 1];
            i00[u] = pk * lda + pl; i01[u] = pk * lda + ql; i10[u] = qk * lda + pl; i11[u] = qk * lda + ql;
            a00[u] = A[i00[u]]; a01[u] = A[i01[u]]; a10[u] = A[i10[u]]; a11[u] = A[i11[u]];
          }
        }
#pragma unroll
        for (int u = 0; u < 2; u++) {
          const int e = e0 + u * FIT_THREADS;
          if (e < nblk) {
            // left: rows (p_k, q_k) <- (c x - s y, s x + c y)
            const double r00 = ck[u] * a00[u] - sk[u] * a10[u], r01 = ck[u] * a01[u] - sk[u] * a11[u];
            const double r10 = sk[u] * a00[u] + ck[u] * a10[u], r11 = sk[u] * a01[u] + ck[u] * a11[u];
            // right: columns (p_l, q_l) <- (c x - s y, s x + c y)
            A[i00[u]] = cl[u] * r00 - sl[u] * r01;
            A[i01[u]] = sl[u] * r00 + cl[u] * r01;
            A[i10[u]] = cl[u] * r10 - sl[u] * r11;
            A[i11[u]] = sl[u] * r10 + cl[u] * r11;
          }
        }
      }
      __syncthreads();
      if (tid < half && r + 1 < d - 1) rotation_params(r + 1);
      for (int e0 = tid; e0 < items; e0 += 4 * FIT_THREADS) {
        double xv[4], yv[4], cc[4], ss[4];
        int iv[4], jv[4];
#pragma unroll
        for (int u = 0; u < 4; u++) {
          const int e = e0 + u * FIT_THREADS;
          if (e < items) {
            const int k = e >> log2d, row = e & dm1;
            cc[u] = cs[2 * k]; ss[u] = cs[2 * k + 1];
            iv[u] = sr[k].x * ldvt + row; jv[u] = sr[k].y * ldvt + row;
            xv[u] = VT[iv[u]]; yv[u] = VT[jv[u]];
          }
        }
#pragma unroll
        for (int u = 0; u < 4; u++) {
          const int e = e0 + u * FIT_THREADS;
          if (e < items) {
            VT[iv[u]] = cc[u] * xv[u] - ss[u] * yv[u];
            VT[jv[u]] = ss[u] * xv[u] + cc[u] * yv[u];
          }
        }
      }
      __syncthreads();
    }
  }
  __syncthreads();
  return sweeps;
}

// The same iteration for matrices small enough that two copies of A fit in shared memory
// (d <= 64), with three kinds of warps working on a round at the same time, each in a loop of
// its own (jacobi_role) so that the register needs of one do not constrain the others:
//   JR_AHEAD  warp 0 looks ahead: it evaluates, straight from the old copy of A, the three
//             entries (a_pp, a_qq, a_pq after round r) of every pair of round r + 1 and turns
//             them into that round's rotations;
//   JR_VT     2 D threads keep V^T in registers, half a column each, stored in "seat" order
//             (seat 2k holds row p_k of the current round, seat 2k + 1 row q_k), so the rotations
//             touch fixed registers; between rounds the tournament moves every index one seat
//             along, which is a fixed register permutation plus one exchange between the two
//             halves of a column.  Afterwards they help with A;
//   JR_A      the other warps apply round r to A, reading one copy and writing the other, so
//             nothing is updated in place.  A is symmetric: only the blocks on and above the
//             block diagonal are computed, and element (i, j) lives at [min(i, j)][max(i, j)]
//             only; the block list pairs block row k with block row d/2 - k, which keeps the
//             shared-memory bank conflicts of a warp's accesses low.
// One block barrier per round remains; the three loops meet at the same barriers.
//   la  : [(d-1) x d/2] for round r and pair j of round r + 1, where that pair's two indices sit in
//         round r: x = rows (p, q) of both current pairs, y = the two pair numbers and two flags
//         (bit 16: the next p is its current pair's q; bit 17: the same for the next q)
//   tri : the (k, l), k <= l, block list
struct JacobiCtx {
  double* A0; double* A1; double* VT; double* cs_base; double* red;
  const ushort2* sched; const uint2* la; const uchar2* tri;
  int lda, ldvt;
};
enum { JR_AHEAD = 0, JR_VT = 1, JR_A = 2 };

// (c, s) that annihilates a_pq, from fp32 arithmetic with two special-function calls, then made
// orthonormal in fp64 (one Newton step on c^2 + s^2 = 1).  An angle accurate to 1e-7 still
// removes a_pq to that relative level and keeps V exactly orthogonal.  scale brings the entries
// to order one so that the fp32 squares neither overflow nor vanish.
__device__ __forceinline__ void jacobi_angle(double app, double aqq, double apq, double scale, double& c, double& s) {
  c = 1.0; s = 0.0;
  const float num = (float)((aqq - app) * scale), den = (float)((apq + apq) * scale);
  const float h2 = fmaf(num, num, den * den);
  const float u = fabsf(num) + h2 * rsqrtf(h2);            // |num| + hypot(num, den)
  const float rw = rsqrtf(fmaf(u, u, den * den));
  const float c0 = u * rw, s0 = copysignf(1.f, num) * den * rw;
  if (den != 0.f && isfinite(c0) && isfinite(s0)) {        // zero or non-finite: no rotation
    const double cd = (double)c0, sd = (double)s0;
    const double f = fma(-0.5, fma(cd, cd, sd * sd), 1.5);
    c = cd * f; s = sd * f;
  }
}

// where element (i, j) of the symmetric matrix is kept
__device__ __forceinline__ int jacobi_upper(int i, int j, int lda) { return i < j ? i * lda + j : j * lda + i; }

template <int D>
__device__ __forceinline__ void jacobi_a_items(const JacobiCtx& jc, const double* __restrict__ Ao, double* __restrict__ An,
                                               const ushort2* sr, const double* cs, int first, int last, int step) {
  const int lda = jc.lda;
  for (int e = first; e < last; e += step) {
    const uchar2 kl = jc.tri[e];
    const int k = kl.x, l = kl.y;
    const int pk = sr[k].x, qk = sr[k].y, pl = sr[l].x, ql = sr[l].y;
    const double2 rk = reinterpret_cast<const double2*>(cs)[k], rl = reinterpret_cast<const double2*>(cs)[l];
    const double ck = rk.x, sk = rk.y, cl = rl.x, sl = rl.y;
    const int i00 = jacobi_upper(pk, pl, lda), i01 = jacobi_upper(pk, ql, lda), i10 = jacobi_upper(qk, pl, lda), i11 = jacobi_upper(qk, ql, lda);
    const double a00 = Ao[i00], a01 = Ao[i01], a10 = Ao[i10], a11 = Ao[i11];
    // left: rows (p_k, q_k) <- (c x - s y, s x + c y); right: the same on columns (p_l, q_l)
    const double r00 = ck * a00 - sk * a10, r01 = ck * a01 - sk * a11;
    const double r10 = sk * a00 + ck * a10, r11 = sk * a01 + ck * a11;
    const double n00 = cl * r00 - sl * r01, n01 = sl * r00 + cl * r01;
    const double n10 = cl * r10 - sl * r11, n11 = sl * r10 + cl * r11;
    if (k == l) {
      An[i00] = n00; An[i11] = n11; An[i01] = 0.5 * (n01 + n10);       // i01 == i10
    } else {
      An[i00] = n00; An[i01] = n01; An[i10] = n10; An[i11] = n11;
    }
  }
}

// Returns the number of sweeps; *final_buf tells which copy (0: A0, 1: A1) holds the result.
template <int D, int ROLE>
__device__ __forceinline__ int jacobi_role(const JacobiCtx& jc_in, int* final_buf) {
  const JacobiCtx jc = jc_in;                            // by value: the fields stay in registers
  constexpr int d = D, half = D / 2, nrounds = D - 1, N2 = D / 2;
  constexpr int VT_THREADS = 2 * D;
  constexpr int ntri = half * (half + 1) / 2;            // blocks of A on and above the block diagonal
  constexpr int NA = FIT_THREADS - 32 - VT_THREADS;      // threads that only work on A
  // the V^T threads take the last VT_ITEMS blocks of A after their own work (measured best: three quarters
  // of a block per thread), the others share the rest
  constexpr int VT_ITEMS = (3 * VT_THREADS / 4) < ntri ? 3 * VT_THREADS / 4 : ntri;
  const int tid = threadIdx.x, lda = jc.lda;
  // JR_VT: column of V^T and which half of its seats.  The two halves of a column sit 16 lanes apart, so that
  // the eight lanes that share a shared-memory transaction read the same rotation (one broadcast, no bank conflict).
  const int vcol = ((tid - 32) >> 5) * 16 + (tid & 15), vh = (tid >> 4) & 1;
  const int a_first = ROLE == JR_A ? tid - 32 - VT_THREADS : ntri - VT_ITEMS + (tid - 32);
  const int a_last = ROLE == JR_A ? ntri - VT_ITEMS : ntri;
  constexpr int a_step = ROLE == JR_A ? NA : VT_THREADS;
  // index sitting at `seat` in round r
  auto seat_index = [](int r, int seat) {
    const int k = seat >> 1;
    if (k == 0) return (seat & 1) ? d - 1 : r;
    return (seat & 1) ? (r - k + nrounds) % nrounds : (r + k) % nrounds;
  };
  double x[ROLE == JR_VT ? N2 : 1];
  if (ROLE == JR_VT) {
#pragma unroll
    for (int j = 0; j < N2; j++) x[j] = seat_index(0, vh * N2 + j) == vcol ? 1.0 : 0.0;
  }
  int sweeps = 0, rr = 0;                           // rr: rounds done so far; A lives in copy rr & 1
  for (int sweep = 0; sweep < JACOBI_MAX_SWEEPS; sweep++) {
    const double* Ac = (rr & 1) ? jc.A1 : jc.A0;
    double off = 0.0, tot = 0.0;
    for (int e = tid; e < d * d; e += FIT_THREADS) {
      int i = e / d, j = e % d;
      if (i > j) continue;
      double v = Ac[i * lda + j];
      tot += i == j ? v * v : 2.0 * v * v;
      if (i != j) off += 2.0 * v * v;
    }
    off = block_reduce(off, jc.red, 0);
    tot = block_reduce(tot, jc.red, 0);
    if (off <= 1e-24 * tot || tot == 0.0) break;
    sweeps++;
    const double scale = ROLE == JR_AHEAD ? rsqrt(tot * (1.0 / d)) : 0.0;      // entries of A -> order one
    if (sweep == 0) {                               // later sweeps inherit round 0's rotations from the look-ahead
      if (ROLE == JR_AHEAD && tid < half) {
        const int p = jc.sched[tid].x, q = jc.sched[tid].y;
        double c, s;
        jacobi_angle(Ac[p * lda + p], Ac[q * lda + q], Ac[jacobi_upper(p, q, lda)], scale, c, s);
        jc.cs_base[2 * tid] = c; jc.cs_base[2 * tid + 1] = s;
      }
      __syncthreads();
    }
    for (int r = 0; r < nrounds; r++, rr++) {
      const double* __restrict__ Ao = (rr & 1) ? jc.A1 : jc.A0;
      double* __restrict__ An = (rr & 1) ? jc.A0 : jc.A1;
      const ushort2* sr = jc.sched + r * half;
      const double* cs = jc.cs_base + (rr & 1) * d;
      if (ROLE == JR_AHEAD) {
        // rotations of the next round from entries of J^T A J evaluated directly
        if (tid < half) {
          const uint2 t = jc.la[r * half + tid];
          const int pp = t.x & 255, pq_ = (t.x >> 8) & 255, qp = (t.x >> 16) & 255, qq_ = t.x >> 24;
          const double2 rx = reinterpret_cast<const double2*>(cs)[t.y & 255], ry = reinterpret_cast<const double2*>(cs)[(t.y >> 8) & 255];
          const double a_pp_pp = Ao[pp * lda + pp], a_pp_pq = Ao[jacobi_upper(pp, pq_, lda)], a_pq_pq = Ao[pq_ * lda + pq_];
          const double a_qp_qp = Ao[qp * lda + qp], a_qp_qq = Ao[jacobi_upper(qp, qq_, lda)], a_qq_qq = Ao[qq_ * lda + qq_];
          const double b00 = Ao[jacobi_upper(pp, qp, lda)], b01 = Ao[jacobi_upper(pp, qq_, lda)];
          const double b10 = Ao[jacobi_upper(pq_, qp, lda)], b11 = Ao[jacobi_upper(pq_, qq_, lda)];
          // new row/column x = f.p * old p + f.q * old q of x's current pair
          const bool xq = (t.y >> 16) & 1, yq = (t.y >> 17) & 1;
          const double fpp = xq ? rx.y : rx.x, fpq = xq ? rx.x : -rx.y;
          const double fqp = yq ? ry.y : ry.x, fqq = yq ? ry.x : -ry.y;
          const double napp = fpp * (fpp * a_pp_pp + fpq * a_pp_pq) + fpq * (fpp * a_pp_pq + fpq * a_pq_pq);
          const double naqq = fqp * (fqp * a_qp_qp + fqq * a_qp_qq) + fqq * (fqp * a_qp_qq + fqq * a_qq_qq);
          const double napq = fqp * (fpp * b00 + fpq * b10) + fqq * (fpp * b01 + fpq * b11);
          double c, s;
          jacobi_angle(napp, naqq, napq, scale, c, s);
          double* csn = jc.cs_base + ((rr + 1) & 1) * d;
          csn[2 * tid] = c; csn[2 * tid + 1] = s;
        }
      } else if (ROLE == JR_VT) {
        // V^T <- J^T V^T on this thread's half column, then every index moves one seat along
        const double2* cs2 = reinterpret_cast<const double2*>(cs) + vh * (N2 / 2);
#pragma unroll
        for (int jj = 0; jj < N2 / 2; jj++) {
          const double2 r2 = cs2[jj];
          const double a = x[2 * jj], b = x[2 * jj + 1];
          x[2 * jj] = r2.x * a - r2.y * b;
          x[2 * jj + 1] = r2.y * a + r2.x * b;
        }
        // Even seats move down by two, odd seats up by two; seat 1 is fixed, seat 0 goes to seat 3,
        // the last odd seat to the last even one.  Two values cross between the halves of a column.
        const double send = vh ? x[0] : x[N2 - 1];
        const double recv = __shfl_xor_sync(0xffffffffu, send, 16);
        const double t0 = x[0];
#pragma unroll
        for (int j = 0; j <= N2 - 4; j += 2) x[j] = x[j + 2];
        x[N2 - 2] = vh ? x[N2 - 1] : recv;
#pragma unroll
        for (int j = N2 - 1; j >= 5; j -= 2) x[j] = x[j - 2];
        x[3] = vh ? x[1] : t0;
        x[1] = vh ? recv : x[1];
        jacobi_a_items<D>(jc, Ao, An, sr, cs, a_first, a_last, a_step);
      } else {
        jacobi_a_items<D>(jc, Ao, An, sr, cs, a_first, a_last, a_step);
      }
      __syncthreads();
    }
  }
  // the seats now hold the order of round rr mod (d - 1): put the rows of V^T back
  if (ROLE == JR_VT) {
    const int rf = rr % nrounds;
#pragma unroll
    for (int j = 0; j < N2; j++) jc.VT[seat_index(rf, vh * N2 + j) * jc.ldvt + vcol] = x[j];
  }
  __syncthreads();
  *final_buf = rr & 1;
  return sweeps;
}

template <int D>
__device__ __forceinline__ int jacobi_eig_lookahead(const JacobiCtx& jc, int* final_buf) {
  const int tid = threadIdx.x;
  if (tid < 32) return jacobi_role<D, JR_AHEAD>(jc, final_buf);
  if (tid < 32 + 2 * D) return jacobi_role<D, JR_VT>(jc, final_buf);
  return jacobi_role<D, JR_A>(jc, final_buf);
}

// Tables of jacobi_eig_lookahead (pos is scratch: where every index sits in every round).
__device__ void jacobi_tables(const ushort2* sched, uchar2* pos, uint2* la, uchar2* tri, int d) {
  const int half = d >> 1;
  for (int e = threadIdx.x; e < (d - 1) * half; e += FIT_THREADS) {
    const int r = e / half, k = e % half;
    pos[r * d + sched[e].x] = make_uchar2((unsigned char)k, 0);
    pos[r * d + sched[e].y] = make_uchar2((unsigned char)k, 1);
  }
  for (int e = threadIdx.x; e < half * half; e += FIT_THREADS) {
    const int k = e / half, l = e % half;
    if (k > l) continue;
    // block row k <= half/2 is followed by block row half - k: together they fill `half` slots
    const int slot = k <= half / 2 ? half * k + (l - k) : half * (half - k) + k + (l - k);
    tri[slot] = make_uchar2((unsigned char)k, (unsigned char)l);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < (d - 1) * half; e += FIT_THREADS) {
    const int r = e / half, j = e % half;
    const int rn = (r + 1 == d - 1) ? 0 : r + 1;
    const ushort2 nx = sched[rn * half + j];
    const uchar2 px = pos[r * d + nx.x], py = pos[r * d + nx.y];
    const ushort2 cx = sched[r * half + px.x], cy = sched[r * half + py.x];
    la[e] = make_uint2((unsigned)cx.x | ((unsigned)cx.y << 8) | ((unsigned)cy.x << 16) | ((unsigned)cy.y << 24),
                       (unsigned)px.x | ((unsigned)py.x << 8) | ((unsigned)px.y << 16) | ((unsigned)py.y << 17));
  }
  __syncthreads();
}

// 1 / sqrt(t) and 1 / t to rounding: the 20-bit hardware estimate and two Newton steps (t normal and positive,
// resp. non-zero; no special cases).
__device__ __forceinline__ double rsqrt_fast(double t) {
  double q;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(q) : "d"(t));
  q = fma(q * 0.5, fma(-t * q, q, 1.0), q);
  return fma(q * 0.5, fma(-t * q, q, 1.0), q);
}
__device__ __forceinline__ double recip_fast(double t) {
  double q;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(q) : "d"(t));
  q = fma(q, fma(-t, q, 1.0), q);
  return fma(q, fma(-t, q, 1.0), q);
}

// Row handled by lane group `grp` when `parts` lanes share a row: with eight lanes per row the two rows of a
// half-warp are eight apart, so that their 8-byte accesses to a matrix with an odd leading dimension fall into
// different banks.
__device__ __forceinline__ int group_row(int grp, int parts) {
  return parts == 8 ? ((grp & ~15) | ((grp & 1) << 3) | ((grp >> 1) & 7)) : grp;
}

// D x D product with both operands in shared memory (leading dimension D + 1):
// out(r, c, sum_k a(r, k) b(k, c)) with a(r, k) = A[r][k] (TA: A[k][r]) and b(k, c) = B[k][c] (TB: B[c][k]).
// Thread t < (D/4)^2 owns the 4 x 4 outputs in rows t / (D/4) + u D/4 and columns t % (D/4) + v D/4: eight loads
// at fixed offsets from two running pointers feed sixteen fp64 multiply-adds, which keeps the fp64 pipe and not
// the shared-memory port or the issue slots the limit.
template <int D, bool TA, bool TB, class FO>
__device__ __forceinline__ void product_impl(const double* A, const double* B, FO out) {
  constexpr int q = D / 4, lda = D + 1;
  if ((int)threadIdx.x >= q * q) return;
  const int r0 = threadIdx.x / q, c0 = threadIdx.x % q;
  constexpr int sa_u = TA ? q : q * lda, sa_k = TA ? lda : 1;
  constexpr int sb_v = TB ? q * lda : q, sb_k = TB ? 1 : lda;
  const double* pa = A + (TA ? r0 : r0 * lda);
  const double* pb = B + (TB ? c0 * lda : c0);
  double acc[4][4];
#pragma unroll
  for (int u = 0; u < 4; u++)
#pragma unroll
    for (int v = 0; v < 4; v++) acc[u][v] = 0.0;
#pragma unroll 4
  for (int k = 0; k < D; k++) {
    double av[4], bv[4];
#pragma unroll
    for (int u = 0; u < 4; u++) av[u] = pa[u * sa_u + k * sa_k];
#pragma unroll
    for (int v = 0; v < 4; v++) bv[v] = pb[v * sb_v + k * sb_k];
#pragma unroll
    for (int u = 0; u < 4; u++)
#pragma unroll
      for (int v = 0; v < 4; v++) acc[u][v] = fma(av[u], bv[v], acc[u][v]);
  }
#pragma unroll
  for (int u = 0; u < 4; u++)
#pragma unroll
    for (int v = 0; v < 4; v++) out(r0 + u * q, c0 + v * q, acc[u][v]);
}
template <bool TA, bool TB, class FO>
__device__ __forceinline__ void smem_product(int d, const double* A, const double* B, FO out) {
  if (d == 64) product_impl<64, TA, TB>(A, B, out);
  else if (d == 32) product_impl<32, TA, TB>(A, B, out);
  else product_impl<16, TA, TB>(A, B, out);
}

// ---- direct eigensolver for d <= 64 --------------------------------------------------------------
// Householder tridiagonalisation, eigenvalues of the tridiagonal matrix by multisection on Sturm
// counts, one eigenvector per eigenvalue from the twisted factorisation of T - sigma I, the
// reflectors applied back, one first-order symmetric orthogonalisation, and A' = V^T A V.  The
// Jacobi solver then starts from A', which is diagonal to rounding whenever the eigenvalues are
// separated, and checks (or completes) the result with its own convergence test: the accuracy is
// that of the Jacobi solver, the cost that of a few matrix products.  Vectors that fail the
// orthogonality check (eigenvalues that agree to rounding, a matrix that splits) make the
// function return false with A restored; the caller then runs the Jacobi solver on A itself.
//
// Thread t = (row or vector r = t / P, part = t % P) with P = FIT_THREADS / D lanes of one warp
// sharing every reduction.
template <int D>
__device__ __forceinline__ bool direct_eig(double* __restrict__ As, double* __restrict__ A1, double* __restrict__ Vs,
                                           double* __restrict__ Ws, int lda, double* __restrict__ dd,
                                           double* __restrict__ ee, double* __restrict__ beta, double* red) {
  constexpr int P = FIT_THREADS / D, NU = (D + P - 1) / P;
  static_assert(P >= 8 && P <= 32, "lanes per vector");
  const int tid = threadIdx.x, part = tid % P;
  // row (or vector) of this group of lanes.  With eight lanes per row the two rows of a half-warp are eight
  // apart, so that their 8-byte accesses to a padded (odd leading dimension) matrix fall into different banks.
  const int grp = tid / P;
  const int r = group_row(grp, P);
  const int warp_row0 = P == 8 ? (((tid >> 5) * 4) & 48) | (((tid >> 5) * 2) & 6) : (tid & ~31) / P;   // smallest row of this warp
  auto gsum = [](double v) {
#pragma unroll
    for (int o = P >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
  };
  for (int e = tid; e < D * D; e += FIT_THREADS) Ws[(e / D) * lda + (e % D)] = As[(e / D) * lda + (e % D)];

  // 1. A -> Q^T A Q = T (tridiagonal).  Reflector k, I - beta_k v v^T with v = x - alpha e_1, acts on indices
  //    k+1..D-1 (x: column k below the diagonal); v is kept in column k of A.  Per step, with A22 the trailing
  //    block: y = A22 x and |x|^2 do not wait for alpha; p = beta A22 v = beta (y - alpha A22 e_1);
  //    w = p - (beta/2 v.p) v;  A22 -= v w^T + w v^T.  Warps whose rows all lie outside the block only keep the barriers.
  for (int k = 0; k < D - 2; k++) {
    const int n = D - k - 1;
    const bool active = warp_row0 < n;
    double* xc = As + (k + 1) * lda + k;              // x_i = xc[i * lda]
    double* A22 = As + (k + 1) * lda + (k + 1);
    double vj[NU], a22[NU], vr = 0.0, pr = 0.0, b = 0.0, alpha = 0.0, v0 = 0.0;
    if (active) {
      double s2a = 0.0, s2b = 0.0, ya = 0.0, yb = 0.0;
#pragma unroll
      for (int u = 0; u < NU; u++) {
        const int j = part + u * P;
        vj[u] = j < n ? xc[j * lda] : 0.0;
      }
      const double x0 = xc[0];
      const double ar0 = r < n ? A22[r * lda] : 0.0;   // A22[r][0]
      vr = r < n ? xc[r * lda] : 0.0;
#pragma unroll
      for (int u = 0; u < NU; u++) {
        const int j = part + u * P;
        a22[u] = (r < n && j < n) ? A22[r * lda + j] : 0.0;
        if (u & 1) { yb = fma(a22[u], vj[u], yb); if (j >= 1) s2b = fma(vj[u], vj[u], s2b); }
        else { ya = fma(a22[u], vj[u], ya); if (j >= 1) s2a = fma(vj[u], vj[u], s2a); }
      }
      double y = ya + yb, s2 = s2a + s2b;
#pragma unroll
      for (int o = P >> 1; o > 0; o >>= 1) {
        y += __shfl_xor_sync(0xffffffffu, y, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
      }
      alpha = x0; v0 = x0;
      if (s2 > 0.0) {
        const double nrm2 = fma(x0, x0, s2);
        const double anorm = nrm2 * rsqrt_fast(nrm2);                 // |x|
        alpha = -copysign(anorm, x0);
        v0 = x0 - alpha;
        b = recip_fast(fma(fabs(x0), anorm, nrm2));                   // 2 / |v|^2 = 1 / (|x|^2 + |x_0| |x|)
        if (part == 0) vj[0] = v0;
        if (r == 0) vr = v0;
      }
      pr = b * fma(-alpha, ar0, y);
      if (part == 0 && r < n) red[r] = pr;
    }
    __syncthreads();
    if (active) {
      if (tid == 0) { ee[k] = alpha; beta[k] = b; dd[k] = As[k * lda + k]; xc[0] = v0; }
      double pj[NU], ka = 0.0, kb = 0.0;
#pragma unroll
      for (int u = 0; u < NU; u++) {
        const int j = part + u * P;
        pj[u] = j < n ? red[j] : 0.0;
        if (u & 1) kb = fma(vj[u], pj[u], kb); else ka = fma(vj[u], pj[u], ka);
      }
      const double kk = gsum(ka + kb) * (0.5 * b);
      if (r < n && b != 0.0) {
        const double wr = fma(-kk, vr, pr);
#pragma unroll
        for (int u = 0; u < NU; u++) {
          const int j = part + u * P;
          if (j < n) {
            const double wj = fma(-kk, vj[u], pj[u]);
            A22[r * lda + j] = a22[u] - fma(vr, wj, wr * vj[u]);
          }
        }
      }
    }
    __syncthreads();
  }
  if (tid == 0) {
    dd[D - 2] = As[(D - 2) * lda + (D - 2)];
    dd[D - 1] = As[(D - 1) * lda + (D - 1)];
    ee[D - 2] = As[(D - 1) * lda + (D - 2)];
    ee[D - 1] = 0.0;
  }
  __syncthreads();

  // 2. Eigenvalues of T.  Gershgorin interval, T scaled by a power of two so that it is of order one (the
  //    vectors do not change; the final eigenvalues are read from A' later).
  double lo = 1e300, hi = -1e300;
#pragma unroll
  for (int u = 0; u < NU; u++) {
    const int i = part + u * P;
    if (i < D) {
      const double rad = fabs(ee[i]) + (i > 0 ? fabs(ee[i - 1]) : 0.0);
      lo = fmin(lo, dd[i] - rad);
      hi = fmax(hi, dd[i] + rad);
    }
  }
#pragma unroll
  for (int o = P >> 1; o > 0; o >>= 1) {
    lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  const double nrm = fmax(fabs(lo), fabs(hi));
  if (!(nrm > 1e-290) || !(nrm < 1e290)) {            // zero, non-finite or absurdly scaled: leave it to the caller
    __syncthreads();
    for (int e = tid; e < D * D; e += FIT_THREADS) As[(e / D) * lda + (e % D)] = Ws[(e / D) * lda + (e % D)];
    __syncthreads();
    return false;
  }
  const int nex = ((__double2hiint(nrm) >> 20) & 0x7ff) - 1023;
  const double sc = __hiloint2double((1023 - nex) << 20, 0);         // 2^-nex: nrm * sc in [1, 2)
  double2* de = reinterpret_cast<double2*>(red);      // de[i] = (d_i, e_{i-1}^2), scaled
  int* cnt = reinterpret_cast<int*>(red + 2 * D);     // counts at the FIT_THREADS points of the first grid
  __syncthreads();
  if (tid < D) {
    const double ep = tid > 0 ? ee[tid - 1] * sc : 0.0;
    de[tid] = make_double2(dd[tid] * sc, ep * ep);
  }
  __syncthreads();
  if (tid < D) { dd[tid] *= sc; ee[tid] *= sc; }
  __syncthreads();
  lo *= sc; hi *= sc;
  // Number of eigenvalues below x: sign changes along the leading principal minors p_i of T - x I,
  // p_i = (d_i - x) p_{i-1} - e_{i-1}^2 p_{i-2}, p_{-1} = 1.  The pair of minors is brought back to order one
  // every eight steps.
  auto below = [&](double x) {
    double pm2 = 1.0, pm1 = de[0].x - x;
    int c = (unsigned)__double2hiint(pm1) >> 31;
#pragma unroll 8
    for (int i = 1; i < D; i++) {
      const double2 t = de[i];
      const double p = fma(t.x - x, pm1, -(t.y * pm2));
      c += (unsigned)(__double2hiint(p) ^ __double2hiint(pm1)) >> 31;
      pm2 = pm1; pm1 = p;
      if ((i & 7) == 0) {
        const int ex = max((__double2hiint(pm1) >> 20) & 0x7ff, (__double2hiint(pm2) >> 20) & 0x7ff);
        if (ex > 0 && ex < 0x7fe) {
          const double s = __hiloint2double((2046 - ex) << 20, 0);
          pm1 *= s; pm2 *= s;
        }
      }
    }
    return c;
  };
  double sigma;
  {
    // first a grid of FIT_THREADS points over the whole interval, one count per thread ...
    double a = lo - 0.001 * (hi - lo) - 1e-3, bq = hi + 0.001 * (hi - lo) + 1e-3;
    {
      const double h = (bq - a) * (1.0 / (FIT_THREADS + 1));
      cnt[tid] = below(fma(h, (double)(tid + 1), a));
      __syncthreads();
      int lo_i = 0, hi_i = FIT_THREADS;               // first grid point with more than r eigenvalues below it
      while (lo_i < hi_i) {
        const int mid = (lo_i + hi_i) >> 1;
        if (cnt[mid] >= r + 1) hi_i = mid; else lo_i = mid + 1;
      }
      const double na = lo_i > 0 ? fma(h, (double)lo_i, a) : a;
      const double nb = lo_i < FIT_THREADS ? fma(h, (double)(lo_i + 1), a) : bq;
      a = na; bq = nb;
    }
    // ... then P points per step inside the bracket of this group's eigenvalue, to 2^-50 of the first interval
    constexpr int NIT = P == 8 ? 13 : (P == 16 ? 10 : 8);
    const unsigned gshift = (tid & 31) / P * P;
    for (int it = 0; it < NIT; it++) {
      const double h = (bq - a) * (1.0 / (P + 1));
      const double x = fma(h, (double)(part + 1), a);
      const bool above = below(x) >= r + 1;           // at least r + 1 eigenvalues lie below x
      unsigned mask = __ballot_sync(0xffffffffu, above) >> gshift;
      mask &= P < 32 ? (1u << (P & 31)) - 1u : 0xffffffffu;
      const int first = mask ? __ffs(mask) - 1 : P;   // first point with the r-th eigenvalue below it
      const double na = first > 0 ? fma(h, (double)first, a) : a;
      const double nb = first < P ? fma(h, (double)(first + 1), a) : bq;
      a = na; bq = nb;
    }
    sigma = 0.5 * (a + bq);
  }

  // 3. Eigenvector of T for sigma from the twisted factorisation.  With P+_i the leading and P-_i the trailing
  //    principal minors of T - sigma I (P+_{-1} = P-_D = 1), the pivots of the elimination from the top and from
  //    the bottom are D+_i = P+_i / P+_{i-1} and D-_i = P-_i / P-_{i+1}, and
  //    gamma_i = D+_i + D-_i - (d_i - sigma).  The vector starts with 1 at the index of the smallest |gamma| and
  //    runs outwards: z_i = -l+_i z_{i+1} with l+_i = e_i / D+_i, z_{i+1} = -l-_{i+1} z_i with l-_i = e_{i-1} / D-_i.
  //    Two lanes run the two minor recurrences (one multiply-add per step); all lanes then form the quotients.
  //    A minor that is exactly zero gives a non-finite vector, which the orthogonality check below rejects.
  double* Lp = A1 + r * lda;                          // P+, then l+, then the vector itself
  double* Lm = Vs + r * lda;                          // P-, then l-
  if (part < 2) {
    // lane 0 runs up from the top, lane 1 down from the bottom, in one instruction stream
    const bool fwd = part == 0;
    double* out = fwd ? Lp : Lm;
    const int i0 = fwd ? 0 : D - 1, di = fwd ? 1 : -1;
    double pm2 = 1.0, pm1 = de[i0].x - sigma;
    out[i0] = pm1;
    for (int s0 = 1; s0 < D; s0 += 8) {               // eight steps' operands are loaded ahead of the chain
      double dv[8], ev[8], pv[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int i = i0 + di * (s0 + q);
        const bool in = s0 + q < D;
        dv[q] = in ? de[i].x - sigma : 0.0;
        ev[q] = in ? de[fwd ? i : i + 1].y : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        pv[q] = fma(dv[q], pm1, -(ev[q] * pm2));
        pm2 = pm1; pm1 = pv[q];
      }
#pragma unroll
      for (int q = 0; q < 8; q++)
        if (s0 + q < D) out[i0 + di * (s0 + q)] = pv[q];
    }
  }
  __syncwarp();
  double gbest = 1e300;
  int ibest = 0;
  {
    double lp[NU], lm[NU];
#pragma unroll
    for (int u = 0; u < NU; u++) {
      const int i = part + u * P;
      lp[u] = lm[u] = 0.0;
      if (i < D) {
        const double pp = Lp[i], ppm = i > 0 ? Lp[i - 1] : 1.0;       // P+_i, P+_{i-1}
        const double pq = Lm[i], pqp = i < D - 1 ? Lm[i + 1] : 1.0;   // P-_i, P-_{i+1}
        const double rp = recip_fast(pp), rq = recip_fast(pq);
        lp[u] = ee[i] * ppm * rp;                                     // l+_i (unused for i = D - 1: e = 0)
        lm[u] = (i > 0 ? ee[i - 1] : 0.0) * pqp * rq;                 // l-_i
        const double g = fabs(fma(pp, recip_fast(ppm), fma(pq, recip_fast(pqp), -(dd[i] - sigma))));
        if (g < gbest) { gbest = g; ibest = i; }      // NaN never wins
      }
    }
    __syncwarp();
#pragma unroll
    for (int u = 0; u < NU; u++) {
      const int i = part + u * P;
      if (i < D) { Lp[i] = lp[u]; Lm[i] = lm[u]; }
    }
  }
#pragma unroll
  for (int o = P >> 1; o > 0; o >>= 1) {
    const double go = __shfl_xor_sync(0xffffffffu, gbest, o);
    const int io = __shfl_xor_sync(0xffffffffu, ibest, o);
    if (go < gbest || (go == gbest && io < ibest)) { gbest = go; ibest = io; }
  }
  __syncwarp();
  double zz = 0.0;
  if (part < 2) {
    const bool up = part == 0;
    const double* mul = up ? Lp : Lm;
    const int di = up ? -1 : 1;
    const int steps = up ? ibest : D - 1 - ibest;
    double z = 1.0;
    zz = up ? 1.0 : 0.0;
    for (int s0 = 1; s0 <= steps; s0 += 8) {
      double mv[8], zv[8];
#pragma unroll
      for (int q = 0; q < 8; q++) mv[q] = s0 + q <= steps ? mul[ibest + di * (s0 + q)] : 0.0;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        z = -mv[q] * z;
        zv[q] = z;
        zz = fma(z, z, zz);
      }
#pragma unroll
      for (int q = 0; q < 8; q++)
        if (s0 + q <= steps) Lp[ibest + di * (s0 + q)] = zv[q];
    }
  }
  __syncwarp();
  if (part == 0) Lp[ibest] = 1.0;
  zz = gsum(zz);
  __syncwarp();
  const double zn = rsqrt(zz);
  double z[NU];
#pragma unroll
  for (int u = 0; u < NU; u++) {
    const int i = part + u * P;
    z[u] = i < D ? Lp[i] * zn : 0.0;
  }
  __syncthreads();                                    // every vector is in registers: A1 and Vs are free

  // 4. Eigenvector of A = Q z: the reflectors in reverse order, each vector within its own lanes.
  for (int k = D - 3; k >= 0; k--) {
    const double b = beta[k];
    if (b == 0.0) continue;
    const double* vc = As + k;                        // v_i = vc[i * lda], i > k
    double vi[NU], dot = 0.0;
#pragma unroll
    for (int u = 0; u < NU; u++) {
      const int i = part + u * P;
      vi[u] = (i > k && i < D) ? vc[i * lda] : 0.0;
      dot = fma(vi[u], z[u], dot);
    }
    dot = gsum(dot) * b;
#pragma unroll
    for (int u = 0; u < NU; u++) z[u] = fma(-dot, vi[u], z[u]);
  }
#pragma unroll
  for (int u = 0; u < NU; u++) {
    const int i = part + u * P;
    if (i < D) Vs[r * lda + i] = z[u];                // row r of Vs: the r-th vector
  }
  __syncthreads();

  // 5. G = V V^T - I (rows are the vectors) -> A1; give up unless the vectors are orthonormal to 1e-6.
  double gmax = 0.0;
  product_impl<D, false, true>(Vs, Vs,
               [&](int i, int j, double v) {
                 v -= (i == j) ? 1.0 : 0.0;
                 A1[i * lda + j] = v;
                 gmax = fmax(gmax, isfinite(v) ? fabs(v) : 1e300);
               });
  gmax = block_reduce(gmax, red, 1);
  if (!(gmax <= 1e-6)) {
    for (int e = tid; e < D * D; e += FIT_THREADS) As[(e / D) * lda + (e % D)] = Ws[(e / D) * lda + (e % D)];
    __syncthreads();
    return false;
  }
  // V <- (I - G/2) V -> As: orthonormal to second order in G
  product_impl<D, false, false>(A1, Vs,
               [&](int j, int c, double v) { As[j * lda + c] = fma(-0.5, v, Vs[j * lda + c]); });
  __syncthreads();
  // V A -> A1, then A' = (V A) V^T -> Vs
  product_impl<D, false, false>(As, Ws,
               [&](int j, int m, double v) { A1[j * lda + m] = v; });
  __syncthreads();
  product_impl<D, false, true>(A1, As,
               [&](int i, int j, double v) { Vs[i * lda + j] = v; });
  __syncthreads();
  // A' -> As, V -> Ws
  for (int e = tid; e < D * D; e += FIT_THREADS) {
    const int o = (e / D) * lda + (e % D);
    Ws[o] = As[o];
    As[o] = Vs[o];
  }
  __syncthreads();
  return true;
}

// Cholesky M1 = L L^T (M1 in As, leading dimension D + 1) by elimination, one column per step, and L^-1 with
// it: the row operations that reduce M1 to L^T, applied to the identity, leave L^-1.  Step j subtracts
// f_i = a_ij / a_jj times row j from every row i > j, in the trailing block of M1 (kept symmetric, so that
// column j is read as row j) and in W, which carries the rows of L^-1 without their final scale 1/l_ii.
// The matrix lives in registers for the whole factorisation: lane group i holds row i, the slot of column c
// holding M1[i][c] while c > j and W[i][c] afterwards; only the pivot row of a step goes through shared memory
// (rowbuf, 2 D doubles), since it is the traffic through shared memory that bounds such a step.
// On exit As = L and W = L^-1 (both with zeros above the diagonal), rdiag[j] = 1 / l_jj.  Returns true when a
// pivot had to be raised to `floor_piv`.
template <int D>
__device__ __forceinline__ bool cholesky_inverse(double* __restrict__ As, double* __restrict__ W, double* __restrict__ rdiag,
                                                 double* __restrict__ ldiag, double* __restrict__ rowbuf, double floor_piv) {
  constexpr int P = FIT_THREADS / D, NU = (D + P - 1) / P, lda = D + 1;
  const int tid = threadIdx.x, part = tid % P, ri = group_row(tid / P, P);
  bool raised = false;
  double a[NU];
#pragma unroll
  for (int u = 0; u < NU; u++) {
    const int c = part + u * P;
    a[u] = c < D ? As[ri * lda + c] : 0.0;
    if (ri == 0 && c < D) rowbuf[c] = a[u];
  }
  __syncthreads();
  for (int j = 0; j < D; j++) {
    const double* rb = rowbuf + (j & 1) * D;
    double piv = rb[j];
    if (!(piv > floor_piv)) { raised = true; piv = floor_piv + 1e-300; }
    if (ri > j) {
      double rowj[NU];
#pragma unroll
      for (int u = 0; u < NU; u++) {
        const int c = part + u * P;
        rowj[u] = c < D ? rb[c] : 0.0;
      }
      const double arj = rb[ri];                      // M1[i][j] = M1[j][i]
      const double rs = rsqrt_fast(piv);
      const double lij = arj * rs, f = lij * rs;
#pragma unroll
      for (int u = 0; u < NU; u++) {
        const int c = part + u * P;
        a[u] = c == j ? -f : fma(-f, rowj[u], a[u]);  // W[j][j] = 1
      }
      if (part == j % P) As[ri * lda + j] = lij;
      if (ri == j + 1) {
        double* nb = rowbuf + ((j + 1) & 1) * D;
#pragma unroll
        for (int u = 0; u < NU; u++) {
          const int c = part + u * P;
          if (c < D) nb[c] = a[u];
        }
      }
    } else if (ri == j && part == 0) {
      const double rs = rsqrt_fast(piv);
      ldiag[j] = piv * rs;
      rdiag[j] = rs;
    }
    __syncthreads();
  }
  const double rd = rdiag[ri], ld = ldiag[ri];
#pragma unroll
  for (int u = 0; u < NU; u++) {
    const int c = part + u * P;
    if (c < D) {
      W[ri * lda + c] = c > ri ? 0.0 : (c == ri ? rd : a[u] * rd);
      if (c > ri) As[ri * lda + c] = 0.0;
      else if (c == ri) As[ri * lda + c] = ld;
    }
  }
  __syncthreads();
  return raised;
}

struct FitArgs {
  const double* stats;
  double* params;
  double* scratch;   // per group 5*d*d doubles
  int d, variant;
  double ridge;
  int v_in_smem;
  int* status;
};

template <bool V_IN_SMEM>
__global__ void __launch_bounds__(FIT_THREADS) fit_kernel(FitArgs a) {
  fs_grid_dependency_wait();
  extern __shared__ __align__(16) double sm[];
  const int d = a.d, tid = threadIdx.x, g = blockIdx.x;
  const int lda = d + 1;
  StatsLayout sl{d};
  ParamsLayout pl{d};
  const double* st = a.stats + (size_t)g * sl.total();
  double* out = a.params + (size_t)g * pl.total();
  double* gs = a.scratch + (size_t)g * 5 * d * d;

  double* As = sm;                                   // d*(d+1)
  double* A1 = As + d * lda;                         // second copy of A (look-ahead solver only)
  double* Vs = V_IN_SMEM ? A1 + d * lda : gs;        // eigenvectors, one per ROW
  const int ldv = V_IN_SMEM ? lda : d;
  double* Ws = Vs + d * lda;                         // fourth d x d buffer (ADERF products, d <= 64 only)
  double* vec = As + d * lda + (V_IN_SMEM ? 3 * d * lda : 0);
  double* lam = vec;             // [d]
  double* aux = vec + d;         // [d]
  double* cs = vec + 2 * d;      // [2d]
  double* red = vec + 4 * d;     // [FIT_THREADS]
  int* perm = reinterpret_cast<int*>(red + FIT_THREADS);          // [d]
  ushort2* sched = reinterpret_cast<ushort2*>(perm + d);          // [(d-1) * d/2]
  uint2* la = reinterpret_cast<uint2*>(sched + (d - 1) * (d / 2) + ((d - 1) * (d / 2) & 1));   // 8-byte aligned; look-ahead solver only
  uchar2* pos = reinterpret_cast<uchar2*>(la + (d - 1) * (d / 2));      // [(d-1) * d]
  uchar2* tri = pos + (d - 1) * d;                                      // [d/2 (d/2 + 1) / 2]
  int log2d = 0;
  while ((1 << log2d) < d) log2d++;
  if (!V_IN_SMEM && (a.variant == FSHARP_SDERF || a.variant == FSHARP_ADERF)) jacobi_schedule(sched, d);
  bool tables_built = false;            // the look-ahead solver's tables are built when it first has to sweep
  // eigen-decomposition of the matrix in As: eigenvalues on its diagonal, eigenvectors in the rows of Vs
  auto eig = [&]() -> int {
    if (!V_IN_SMEM) return jacobi_eig(As, lda, Vs, ldv, d, log2d, sched, cs, red);
    int buf = 0, n = 0;
    bool direct;
    if (d == 64) direct = direct_eig<64>(As, A1, Vs, Ws, lda, lam, aux, cs, red);
    else if (d == 32) direct = direct_eig<32>(As, A1, Vs, Ws, lda, lam, aux, cs, red);
    else direct = direct_eig<16>(As, A1, Vs, Ws, lda, lam, aux, cs, red);
    // As: A' = V A V^T with the rows of V (in Ws) the direct solver's eigenvectors, or A itself
    if (direct) {
      // the Jacobi solver's own convergence test on A': met, the direct solver's vectors stand
      double off = 0.0, tot = 0.0;
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        const int i = e / d, j = e % d;
        if (i > j) continue;
        const double v = As[i * lda + j];
        tot += i == j ? v * v : 2.0 * v * v;
        if (i != j) off += 2.0 * v * v;
      }
      off = block_reduce(off, red, 0);
      tot = block_reduce(tot, red, 0);
      if (off <= 1e-24 * tot || tot == 0.0) {
        for (int e = tid; e < d * d; e += FIT_THREADS) Vs[(e / d) * lda + (e % d)] = Ws[(e / d) * lda + (e % d)];
        __syncthreads();
        return 0;
      }
    }
    if (!tables_built) {
      jacobi_schedule(sched, d);
      jacobi_tables(sched, pos, la, tri, d);
      tables_built = true;
    }
    JacobiCtx jc{As, A1, Vs, cs, red, sched, la, tri, lda, ldv};
    if (d == 64) n = jacobi_eig_lookahead<64>(jc, &buf);
    else if (d == 32) n = jacobi_eig_lookahead<32>(jc, &buf);
    else n = jacobi_eig_lookahead<16>(jc, &buf);
    if (buf) {
      for (int e = tid; e < d * lda; e += FIT_THREADS) As[e] = A1[e];
      __syncthreads();
    }
    if (direct) {
      if (n == 0) {
        for (int e = tid; e < d * d; e += FIT_THREADS) Vs[(e / d) * lda + (e % d)] = Ws[(e / d) * lda + (e % d)];
      } else {
        // eigenvectors of A: (rows of the Jacobi solver's V^T) x (rows of V)
        smem_product<false, false>(d, Vs, Ws,
                     [&](int j, int c, double v) { A1[j * lda + c] = v; });
        __syncthreads();
        for (int e = tid; e < d * d; e += FIT_THREADS) Vs[(e / d) * lda + (e % d)] = A1[(e / d) * lda + (e % d)];
      }
      __syncthreads();
    }
    return n;
  };

  const double* M1 = st + sl.M(1);
  const double* M2 = st + sl.M(2);
  const double* mu4 = st + sl.mu(4);
  const double* mu5 = st + sl.mu(5);

  // traces, mu4.mu5, finiteness
  double t1 = 0.0, t2 = 0.0, mm = 0.0, badv = 0.0;
  for (int i = tid; i < d; i += FIT_THREADS) {
    t1 += M1[i * d + i];
    t2 += M2[i * d + i];
    mm += mu4[i] * mu5[i];
  }
  for (int e = tid; e < (int)sl.total(); e += FIT_THREADS)
    if (!isfinite(st[e])) badv = 1.0;
  t1 = block_reduce(t1, red, 0);
  t2 = block_reduce(t2, red, 0);
  mm = block_reduce(mm, red, 0);
  badv = block_reduce(badv, red, 1);
  if (badv > 0.0 && tid == 0) atomicExch(a.status, FSHARP_E_NONFINITE);
  const double rg1 = a.ridge * t1 / d, rg2 = a.ridge * t2 / d;
  t1 += d * rg1;
  t2 += d * rg2;

  double* oA = out + pl.A();
  double* oB1 = out + pl.B(1);
  double* oB2 = out + pl.B(2);
  double* oC1 = out + pl.C(1);
  double* oC2 = out + pl.C(2);
  double* tail = out + pl.tail();
  double logD = 0.0, obj = 0.0, phi = 0.0;
  bool violated = false;
  int nsweeps = 0;

  if (a.variant == FSHARP_POSRF || a.variant == FSHARP_GERF) {
    const double S = t1 + t2 + 2.0 * mm;
    double A = 0.0;
    if (a.variant == FSHARP_GERF) { phi = S / d; A = lemma_a1(phi); }
    const double b = sqrt(1.0 - 4.0 * A);
    for (int e = tid; e < d * d; e += FIT_THREADS) {
      double dg = (e / d == e % d) ? 1.0 : 0.0;
      oA[e] = A * dg; oB1[e] = b * dg; oB2[e] = b * dg; oC1[e] = -0.5 * dg; oC2[e] = -0.5 * dg;
    }
    logD = 0.25 * d * log(1.0 - 4.0 * A);
    obj = d * (log(1.0 - 4.0 * A) - 0.5 * log(1.0 - 8.0 * A)) + (2.0 - 8.0 * A) / (1.0 - 8.0 * A) * S - t1 - t2;
  } else if (a.variant == FSHARP_SADERF) {
    // Section 4.3: Psi_ll = (M2_ll / M1_ll)^(1/4), then the GERF fit on {Psi x}, {Psi^-1 y}.
    double sq = 0.0;
    for (int i = tid; i < d; i += FIT_THREADS) {
      double m1 = M1[i * d + i] + rg1, m2 = M2[i * d + i] + rg2;
      if (!(m1 > 0.0) || !(m2 > 0.0)) { violated = true; m1 = fmax(m1, 1e-300); m2 = fmax(m2, 1e-300); }
      double psi2 = sqrt(m2 / m1);
      lam[i] = sqrt(psi2);
      sq += sqrt(m1 * m2);
    }
    sq = block_reduce(sq, red, 0);
    const double S = 2.0 * sq + 2.0 * mm;
    phi = S / d;
    const double A = lemma_a1(phi);
    const double b = sqrt(1.0 - 4.0 * A);
    for (int e = tid; e < d * d; e += FIT_THREADS) {
      int i = e / d;
      double dg = (i == e % d) ? 1.0 : 0.0, psi = lam[i];
      oA[e] = A * dg; oB1[e] = b * psi * dg; oB2[e] = b / psi * dg;
      oC1[e] = -0.5 * psi * psi * dg; oC2[e] = -0.5 / (psi * psi) * dg;
    }
    logD = 0.25 * d * log(1.0 - 4.0 * A);
    obj = d * (log(1.0 - 4.0 * A) - 0.5 * log(1.0 - 8.0 * A)) + (2.0 - 8.0 * A) / (1.0 - 8.0 * A) * S - 2.0 * sq;
  } else if (a.variant == FSHARP_SDERF) {
    // Theorem 4.3: N = M1 + mu4 mu5^T + mu5 mu4^T + M2, eigenvalues non-ascending.
    for (int e0 = tid; e0 < d * d; e0 += 8 * FIT_THREADS) {          // global loads in batches ahead of the stores
      double m1[8], m2[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        m1[q] = e < d * d ? M1[e] : 0.0;
        m2[q] = e < d * d ? M2[e] : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        if (e < d * d) {
          const int i = e / d, j = e % d;
          As[i * lda + j] = m1[q] + m2[q] + mu4[i] * mu5[j] + mu5[i] * mu4[j] + (i == j ? rg1 + rg2 : 0.0);
        }
      }
    }
    __syncthreads();
    nsweeps += eig();
    for (int i = tid; i < d; i += FIT_THREADS) {
      double li = As[i * lda + i];
      int rank = 0;
      for (int j = 0; j < d; j++) {
        double lj = As[j * lda + j];
        rank += (lj > li) || (lj == li && j < i);
      }
      perm[rank] = i;
    }
    __syncthreads();
    double sl_log = 0.0, so = 0.0;
    for (int l = tid; l < d; l += FIT_THREADS) {
      double lv = fmax(As[perm[l] * lda + perm[l]], 0.0);   // N is PSD; rounding may give -1e-17
      double al = lemma_a1(lv);
      lam[l] = lv;
      aux[l] = al;
      sl_log += log(1.0 - 4.0 * al);
      so += log(1.0 - 4.0 * al) - 0.5 * log(1.0 - 8.0 * al) + (1.0 + 1.0 / (1.0 - 8.0 * al)) * lv;
    }
    sl_log = block_reduce(sl_log, red, 0);
    so = block_reduce(so, red, 0);
    for (int e = tid; e < d * d; e += FIT_THREADS) {
      int l = e / d, j = e % d;
      double dg = (l == j) ? 1.0 : 0.0;
      double b = sqrt(1.0 - 4.0 * aux[l]) * Vs[perm[l] * ldv + j];     // B = (I-4A)^1/2 Q3^T
      oA[e] = aux[l] * dg; oB1[e] = b; oB2[e] = b; oC1[e] = -0.5 * dg; oC2[e] = -0.5 * dg;
    }
    logD = 0.25 * sl_log;
    obj = so - t1 - t2;
    phi = lam[0];
  } else {  // FSHARP_ADERF, Theorem 4.2
    // The theorem writes M1 = Q1 L1 Q1^T and uses F = L1^1/2 Q1^T only as a factor with F^T F = M1:
    // with any other such factor F' = O F (O orthogonal), F' M2 F'^T = O (F M2 F^T) O^T has the
    // eigenvectors U' = O U and the same Sigma^2, so B1 = r Sigma^1/2 U'^T F'^-T and
    // B2 = r Sigma^-1/2 U'^T F' come out the same.  The Cholesky factor F' = L^T (M1 = L L^T) is
    // taken: one eigen-solve is left instead of two.
    double* Lg = gs + (size_t)d * d;        // L     [i][j], lower triangular (upper part zero)
    double* T1g = gs + (size_t)2 * d * d;
    double* Ug = gs + (size_t)3 * d * d;
    double* Lig = gs + (size_t)4 * d * d;   // L^-1  [i][j], lower triangular
    for (int e0 = tid; e0 < d * d; e0 += 8 * FIT_THREADS) {          // global loads in batches ahead of the stores
      double m1[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        m1[q] = e < d * d ? M1[e] : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        if (e < d * d) As[(e / d) * lda + (e % d)] = m1[q] + (e / d == e % d ? rg1 : 0.0);
      }
    }
    __syncthreads();
    const int parts = FIT_THREADS / d, part = tid % parts;
    const double floor_piv = 1e-12 * t1 / d;
    double* Li = V_IN_SMEM ? A1 : Lig;
    const int ldi = V_IN_SMEM ? lda : d;
    if (V_IN_SMEM) {
      // Cholesky M1 = L L^T by elimination, one column per step, and L^-1 with it: the row operations that reduce
      // M1 to L^T, applied to the identity, leave L^-1.  Step j scales by 1/l_jj and subtracts multiples of row j
      // from the rows below; W (in A1) carries the rows of L^-1 without their final scale 1/l_ii.  The trailing
      // block of M1 is updated in both triangles, so that column j can be read as row j.
      if (d == 64) violated |= cholesky_inverse<64>(As, A1, lam, aux, red, floor_piv);
      else if (d == 32) violated |= cholesky_inverse<32>(As, A1, lam, aux, red, floor_piv);
      else violated |= cholesky_inverse<16>(As, A1, lam, aux, red, floor_piv);
    } else {
      // Cholesky, column by column: `parts` threads share the dot product of a row.
      const int ri = tid / parts;
      for (int j = 0; j < d; j++) {
        double t = 0.0;
        if (ri >= j) {
          for (int k = part; k < j; k += parts) t = fma(As[ri * lda + k], As[j * lda + k], t);
        }
        for (int o = parts >> 1; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (ri >= j && part == 0) aux[ri] = As[ri * lda + j] - t;
        __syncthreads();
        double piv = aux[j];
        if (!(piv > floor_piv)) { violated = true; piv = floor_piv + 1e-300; }
        double rs = rsqrt(piv);
        rs = rs * fma(-0.5 * piv * rs, rs, 1.5);       // one Newton step on 1 / sqrt(piv)
        if (part == 0) {
          if (ri == j) { As[j * lda + j] = piv * rs; lam[j] = rs; }     // lam: 1 / l_jj
          else if (ri > j) As[ri * lda + j] = aux[ri] * rs;
          else As[ri * lda + j] = 0.0;                 // upper triangle
        }
        __syncthreads();
      }
      // L^-1 by forward substitution, one column per thread group (columns are independent; the
      // threads of a group sit in one warp).  It is built in shared memory when there is room.
      {
        const int c = ri;
        for (int i = 0; i < d; i++) {
          double t = 0.0;
          if (i > c)
            for (int k = c + part; k < i; k += parts) t = fma(As[i * lda + k], Li[k * ldi + c], t);
          for (int o = parts >> 1; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
          if (part == 0) Li[i * ldi + c] = i < c ? 0.0 : (i == c ? lam[c] : -t * lam[i]);
          __syncwarp();
        }
      }
      __syncthreads();
    }
    for (int e0 = tid; e0 < d * d; e0 += 8 * FIT_THREADS) {
      double m2[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        m2[q] = (V_IN_SMEM && e < d * d) ? M2[e] : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int e = e0 + q * FIT_THREADS;
        if (e >= d * d) continue;
        Lg[e] = As[(e / d) * lda + (e % d)];
        if (V_IN_SMEM) {
          Lig[e] = Li[(e / d) * ldi + (e % d)];
          Vs[(e / d) * lda + (e % d)] = m2[q] + ((e / d) == (e % d) ? rg2 : 0.0);    // M2 into shared memory
        }
      }
    }
    __syncthreads();
    if (V_IN_SMEM) {
      // T1 = M2 L (M2 in Vs, L in As) -> Ws
      smem_product<false, false>(d, Vs, As,
                   [&](int r, int c, double v) { Ws[r * lda + c] = v; });
      __syncthreads();
      // L^T T1 -> A1 (its L^-1 is already in global memory), then Z Z^T = its symmetric part -> Vs
      smem_product<true, false>(d, As, Ws,
                   [&](int r, int c, double v) { A1[r * lda + c] = v; });
      __syncthreads();
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        int r = e / d, c = e % d;
        Vs[r * lda + c] = 0.5 * (A1[r * lda + c] + A1[c * lda + r]);
      }
      __syncthreads();
      for (int e = tid; e < d * lda; e += FIT_THREADS) As[e] = Vs[e];
      __syncthreads();
    } else {
      // T1 = M2 L
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        int i = e / d, l = e % d;
        double s = 0.0;
        for (int j = l; j < d; j++) s = fma(M2[i * d + j] + (i == j ? rg2 : 0.0), Lg[j * d + l], s);
        T1g[e] = s;
      }
      __syncthreads();
      // Z Z^T = L^T M2 L  (symmetric; both triangles written from the same sum)
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        int r = e / d, c = e % d;
        if (r > c) continue;
        double s = 0.0;
        for (int i = r; i < d; i++) s = fma(Lg[i * d + r], T1g[i * d + c], s);
        double s2 = 0.0;
        for (int i = c; i < d; i++) s2 = fma(Lg[i * d + c], T1g[i * d + r], s2);
        double v = 0.5 * (s + s2);
        As[r * lda + c] = v;
        As[c * lda + r] = v;
      }
      __syncthreads();
    }
    nsweeps += eig();     // eigenvalues Sigma^2, eigenvectors U (rows of Vs)
    double smin = 1e300, smax = 0.0, ssum = 0.0;
    for (int l = tid; l < d; l += FIT_THREADS) {
      double sg = sqrt(fmax(As[l * lda + l], 0.0));
      aux[l] = sg;
      smin = fmin(smin, sg); smax = fmax(smax, sg); ssum += sg;
    }
    smin = block_reduce(smin, red, 2);
    smax = block_reduce(smax, red, 1);
    ssum = block_reduce(ssum, red, 0);
    if (!(smin > 1e-12 * smax)) violated = true;
    for (int l = tid; l < d; l += FIT_THREADS) aux[l] = fmax(aux[l], 1e-300 + 1e-12 * smax);
    const double mu3 = mm / d;
    phi = 2.0 * ssum / d + 2.0 * mu3;
    const double A = lemma_a1(phi);
    const double r = sqrt(1.0 - 4.0 * A);
    if (V_IN_SMEM) {
      // L^-1 -> A1, L -> Ws (shared memory again; the eigen-solve used both buffers)
      for (int e0 = tid; e0 < d * d; e0 += 8 * FIT_THREADS) {
        double li[8], lg[8];
#pragma unroll
        for (int q = 0; q < 8; q++) {
          const int e = e0 + q * FIT_THREADS;
          li[q] = e < d * d ? Lig[e] : 0.0;
          lg[q] = e < d * d ? Lg[e] : 0.0;
        }
#pragma unroll
        for (int q = 0; q < 8; q++) {
          const int e = e0 + q * FIT_THREADS;
          if (e < d * d) { A1[(e / d) * lda + (e % d)] = li[q]; Ws[(e / d) * lda + (e % d)] = lg[q]; }
        }
      }
      __syncthreads();
      // B1 = r Sigma^1/2 U^T L^-1 -> As,  B2 = r Sigma^-1/2 U^T L^T -> global, then A1 once L^-1 is no longer read
      smem_product<false, false>(d, Vs, A1,
                   [&](int l, int j, double v) {
                     const double b1 = r * sqrt(aux[l]) * v;
                     As[l * lda + j] = b1;
                     oB1[l * d + j] = b1;
                     oA[l * d + j] = (l == j) ? A : 0.0;
                   });
      __syncthreads();
      smem_product<false, true>(d, Vs, Ws,
                   [&](int l, int j, double v) {
                     const double b2 = r / sqrt(aux[l]) * v;
                     A1[l * lda + j] = b2;
                     oB2[l * d + j] = b2;
                   });
      __syncthreads();
      // C = -B^T B / (2 (1 - 4A))
      const double cf = -1.0 / (2.0 * (1.0 - 4.0 * A));
      smem_product<true, false>(d, As, As,
                   [&](int i, int j, double v) { oC1[i * d + j] = cf * v; });
      smem_product<true, false>(d, A1, A1,
                   [&](int i, int j, double v) { oC2[i * d + j] = cf * v; });
    } else {
      for (int e = tid; e < d * d; e += FIT_THREADS) Ug[e] = Vs[(e % d) * ldv + (e / d)];     // U[i][l]
      __syncthreads();
      // B1 = r Sigma^1/2 U^T L^-1,  B2 = r Sigma^-1/2 U^T L^T
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        int l = e / d, j = e % d;
        double s1 = 0.0, s2 = 0.0;
        for (int i = j; i < d; i++) s1 = fma(Ug[i * d + l], Lig[i * d + j], s1);
        for (int i = 0; i <= j; i++) s2 = fma(Ug[i * d + l], Lg[j * d + i], s2);
        double sg = sqrt(aux[l]);
        oB1[e] = r * sg * s1;
        oB2[e] = r / sg * s2;
        oA[e] = (l == j) ? A : 0.0;
      }
      __syncthreads();
      for (int e = tid; e < d * d; e += FIT_THREADS) {
        int i = e / d, j = e % d;
        double s1 = 0.0, s2 = 0.0;
        for (int l = 0; l < d; l++) {
          s1 = fma(oB1[l * d + i], oB1[l * d + j], s1);
          s2 = fma(oB2[l * d + i], oB2[l * d + j], s2);
        }
        oC1[e] = -s1 / (2.0 * (1.0 - 4.0 * A));
        oC2[e] = -s2 / (2.0 * (1.0 - 4.0 * A));
      }
    }
    logD = 0.25 * d * log(1.0 - 4.0 * A);
    obj = d * (log(1.0 - 4.0 * A) - 0.5 * log(1.0 - 8.0 * A) + 2.0 / (1.0 - 8.0 * A) * (ssum / d + mu3) + 2.0 * mu3);
  }
  if (tid == 0) {
    tail[PT_LOGD] = logD;
    tail[PT_OBJ] = obj;
    tail[PT_PHI] = phi;
    tail[3] = (double)nsweeps;     // Jacobi sweeps spent (diagnostic)
    for (int i = 4; i < 8; i++) tail[i] = 0.0;
  }
  if (violated) atomicExch(a.status, FSHARP_E_CONSTRAINT);
}

size_t fit_smem_bytes(int d, int v_in_smem) {
  size_t dbl = (size_t)d * (d + 1) * (v_in_smem ? 4 : 1) + 4 * (size_t)d + FIT_THREADS;
  size_t tables = v_in_smem ? ((size_t)(d - 1) * d + (size_t)(d / 2) * (d / 2 + 1) / 2) * sizeof(uchar2) +
                                  ((size_t)(d - 1) * (d / 2) + 1) * sizeof(uint2) : 0;
  return dbl * sizeof(double) + (size_t)d * sizeof(int) + (size_t)(d - 1) * (d / 2) * sizeof(ushort2) + tables;
}

}  // namespace

size_t fs_fit_scratch_doubles(int G, int d) { return (size_t)G * 5 * d * d; }

int fs_run_fit(fsharp_ctx* ctx, const double* stats, int G, int d, int variant, double ridge,
               double* params, double* scratch) {
  if (G == 0) return FSHARP_OK;
  FitArgs a;
  a.stats = stats; a.params = params; a.scratch = scratch; a.d = d; a.variant = variant; a.ridge = ridge;
  a.v_in_smem = d <= 64 ? 1 : 0;
  a.status = ctx->d_status;
  size_t smem = fit_smem_bytes(d, a.v_in_smem);
  if (a.v_in_smem) FS_CUDA_OK(cudaFuncSetAttribute(fit_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  else FS_CUDA_OK(cudaFuncSetAttribute(fit_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  FS_TIME_BEGIN(ctx, FS_K_FIT);
  if (a.v_in_smem) (void)fs_launch_chained(fit_kernel<true>, dim3(G), dim3(FIT_THREADS), smem, ctx->stream, a);
  else (void)fs_launch_chained(fit_kernel<false>, dim3(G), dim3(FIT_THREADS), smem, ctx->stream, a);
  FS_TIME_END(ctx);
  FS_LAUNCH_CHECK(ctx);
  return FSHARP_OK;
}
