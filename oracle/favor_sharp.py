"""fp64 CPU oracle for FAVOR# (dense exponential random features + linear attention).

THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct
restatement of the paper's definitions in numpy float64.  Only the test-suite,
the smoke check and the benchmark's CPU-baseline leg may import it; the product
(the CUDA library and its Python binding) never does, and this file imports
nothing from the product.  It contains no blocking, fusion or stabilisation:
every function follows the passage it cites, in the paper's notation.

Notation (Section 2): L sequence length, d head dimension, M number of random
features, Omega the (M, d) matrix whose rows are the omegas, X (L, d) the set
{x^(i)}, Y (L, d) the set {y^(j)}, P and S the (L, M) feature matrices.

Parity status: every function here is pinned by tests that do not go through
the function itself (quadrature, Monte Carlo, closed forms, brute force); the
one exception is the literal entries of B^(1), B^(2), B returned by fit_aderf /
fit_sderf -- "parity unpinned" elementwise, because the theorems say "one of the
solutions" and eigenvector signs / rotations inside equal eigenvalues are free.
Those matrices are pinned through the rotation-invariant quantities
B^T B, B1^T B2, C and the objective value.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Lemma A.1: the scalar map phi -> A
# --------------------------------------------------------------------------
def lemma_a1_A(phi):
    """Minimiser of log(1-4A) - 1/2 log(1-8A) + phi/(1-8A) on (-inf, 1/8).

    Lemma A.1: A* = (1 - 2 phi - sqrt((2 phi + 1)^2 + 8 phi)) / 16, phi >= 0.
    """
    phi = np.asarray(phi, dtype=F64)
    return (1.0 - 2.0 * phi - np.sqrt((2.0 * phi + 1.0) ** 2 + 8.0 * phi)) / 16.0


def lemma_a1_objective(A, phi):
    """The function f(A) of Lemma A.1."""
    A = np.asarray(A, dtype=F64)
    return np.log(1.0 - 4.0 * A) - 0.5 * np.log(1.0 - 8.0 * A) + phi / (1.0 - 8.0 * A)


# --------------------------------------------------------------------------
# Set statistics (Theorems 4.2 and 4.3)
# --------------------------------------------------------------------------
def set_statistics(X, Y):
    """M1 = L^-1 sum x x^T, M2 = L^-1 sum y y^T (Thm 4.2); mu4 = mean x,
    mu5 = mean y (Thm 4.3); mu3 = d^-1 L^-2 (sum x)^T (sum y) (Thm 4.2)."""
    X = np.asarray(X, dtype=F64)
    Y = np.asarray(Y, dtype=F64)
    Lx, d = X.shape
    Ly = Y.shape[0]
    M1 = X.T @ X / Lx
    M2 = Y.T @ Y / Ly
    mu4 = X.sum(axis=0) / Lx
    mu5 = Y.sum(axis=0) / Ly
    mu3 = float(mu4 @ mu5) / d
    return {"M1": M1, "M2": M2, "mu4": mu4, "mu5": mu5, "mu3": mu3, "d": d}


# --------------------------------------------------------------------------
# Theorem 4.1: variance of one DERF product, and the objective built on it
# --------------------------------------------------------------------------
def derf_second_moment_log(x, y, p):
    """log E[f1(w,x)^2 f2(w,y)^2] for DERF parameters p (first term of the
    variance expression of Theorem 4.1)."""
    x = np.asarray(x, dtype=F64)
    y = np.asarray(y, dtype=F64)
    d = x.shape[0]
    I = np.eye(d)
    R8 = np.linalg.inv(I - 8.0 * p["A"])
    _, logdet8 = np.linalg.slogdet(I - 8.0 * p["A"])
    B1, B2, C1, C2 = p["B1"], p["B2"], p["C1"], p["C2"]
    e = (2.0 * x @ (C1 + B1.T @ R8 @ B1) @ x
         + 2.0 * y @ (C2 + B2.T @ R8 @ B2) @ y
         + 4.0 * x @ B1.T @ R8 @ B2 @ y)
    return 4.0 * p["logD"] - 0.5 * logdet8 + e


def derf_variance(x, y, p):
    """Var_w f1(w,x) f2(w,y) of Theorem 4.1 (one omega, i.e. M = 1)."""
    return np.exp(derf_second_moment_log(x, y, p)) - np.exp(2.0 * float(np.dot(x, y)))


def gerf_variance(A, x, y):
    """Scalar-parameter variance of Section 2.3: exp(L_GE) - K^2 with
    L_GE = d log((1-4A)/sqrt(1-8A)) + 2(1-4A)/(1-8A) |x+y|^2 - |x|^2 - |y|^2."""
    x = np.asarray(x, dtype=F64)
    y = np.asarray(y, dtype=F64)
    d = x.shape[0]
    L_ge = (d * np.log((1.0 - 4.0 * A) / np.sqrt(1.0 - 8.0 * A))
            + 2.0 * (1.0 - 4.0 * A) / (1.0 - 8.0 * A) * np.sum((x + y) ** 2)
            - np.sum(x * x) - np.sum(y * y))
    return np.exp(L_ge) - np.exp(2.0 * float(np.dot(x, y)))


def shifted_log_variance_bruteforce(X, Y, p):
    """The shifted log-variance objective of Section 3.1 written out:
    L^-2 sum_{i,j} log(Var[f1(w,x_i) f2(w,y_j)] + K(x_i,y_j)^2).
    Var + K^2 is the second moment, so the log is taken of that directly."""
    X = np.asarray(X, dtype=F64)
    Y = np.asarray(Y, dtype=F64)
    tot = 0.0
    for i in range(X.shape[0]):
        for j in range(Y.shape[0]):
            tot += derf_second_moment_log(X[i], Y[j], p)
    return tot / (X.shape[0] * Y.shape[0])


# --------------------------------------------------------------------------
# Parameter fits.  Every fit returns the DERF form
#   {A (d,d) symmetric, B1, B2, C1, C2 (d,d), logD, objective, phi, variant}
# --------------------------------------------------------------------------
def _pack(variant, A, B1, B2, C1, C2, logD, objective, phi):
    return {"variant": variant, "A": np.asarray(A, F64), "B1": np.asarray(B1, F64),
            "B2": np.asarray(B2, F64), "C1": np.asarray(C1, F64), "C2": np.asarray(C2, F64),
            "logD": float(logD), "objective": float(objective), "phi": phi}


def fit_posrf(st):
    """Positive random features (Section 2.3): exp(w^T x - |x|^2/2), i.e. the
    DERF with A = 0, B = I, C = -I/2, D = 1.  Objective from Section 3.1 at A=0."""
    d = st["d"]
    I = np.eye(d)
    S = np.trace(st["M1"]) + np.trace(st["M2"]) + 2.0 * float(st["mu4"] @ st["mu5"])
    obj = 2.0 * S - np.trace(st["M1"]) - np.trace(st["M2"])
    return _pack("posrf", 0.0 * I, I, I, -0.5 * I, -0.5 * I, 0.0, obj, 0.0)


def fit_gerf(st):
    """GERF (Section 2.3) with A minimising the objective of Section 3.1:
    d[log(1-4A) - 1/2 log(1-8A)] + (2-8A)/(1-8A) S - tr M1 - tr M2,
    S = L^-2 sum |x_i + y_j|^2.  Since (2-8A)/(1-8A) = 1 + 1/(1-8A) this is
    d * f(A) of Lemma A.1 with phi = S/d, plus a constant."""
    d = st["d"]
    I = np.eye(d)
    t1, t2 = np.trace(st["M1"]), np.trace(st["M2"])
    S = t1 + t2 + 2.0 * float(st["mu4"] @ st["mu5"])
    phi = S / d
    A = float(lemma_a1_A(phi))
    B = np.sqrt(1.0 - 4.0 * A)
    logD = 0.25 * d * np.log(1.0 - 4.0 * A)
    obj = (d * np.log((1.0 - 4.0 * A) / np.sqrt(1.0 - 8.0 * A))
           + (2.0 - 8.0 * A) / (1.0 - 8.0 * A) * S - t1 - t2)
    return _pack("gerf", A * I, B * I, B * I, -0.5 * I, -0.5 * I, logD, obj, phi)


def fit_saderf(st):
    """Simplified ADERF (Section 4.3): f1(w,x) = f_GE(w, Psi x),
    f2(w,y) = f_GE(w, Psi^-1 y), Psi_ll = (sum_j y_l^2 / sum_i x_l^2)^(1/4),
    then the GERF fit on the rescaled sets."""
    d = st["d"]
    m1 = np.diag(st["M1"]).copy()
    m2 = np.diag(st["M2"]).copy()
    psi = (m2 / m1) ** 0.25
    t1 = float(np.sum(psi ** 2 * m1))
    t2 = float(np.sum(m2 / psi ** 2))
    S = t1 + t2 + 2.0 * float(st["mu4"] @ st["mu5"])
    phi = S / d
    A = float(lemma_a1_A(phi))
    b = np.sqrt(1.0 - 4.0 * A)
    logD = 0.25 * d * np.log(1.0 - 4.0 * A)
    obj = (d * np.log((1.0 - 4.0 * A) / np.sqrt(1.0 - 8.0 * A))
           + (2.0 - 8.0 * A) / (1.0 - 8.0 * A) * S - t1 - t2)
    I = np.eye(d)
    return _pack("saderf", A * I, b * np.diag(psi), b * np.diag(1.0 / psi),
                 -0.5 * np.diag(psi ** 2), -0.5 * np.diag(psi ** -2.0), logD, obj, phi)


def fit_aderf(st):
    """Asymmetric DERF, Theorem 4.2, literal: eigendecompose M1, M2, take the
    SVD of Lambda1^(1/2) Q1^T Q2 Lambda2^(1/2), phi = 2/d sum Sigma_ll + 2 mu3."""
    d = st["d"]
    lam1, Q1 = np.linalg.eigh(st["M1"])
    lam2, Q2 = np.linalg.eigh(st["M2"])
    if lam1.min() <= 0.0 or lam2.min() <= 0.0:
        raise ValueError("Theorem 4.2 needs nonsingular M1, M2")
    Z = (np.sqrt(lam1)[:, None] * Q1.T) @ (Q2 * np.sqrt(lam2)[None, :])
    U, sig, _Vt = np.linalg.svd(Z)
    mu3 = st["mu3"]
    phi = 2.0 * float(sig.sum()) / d + 2.0 * mu3
    A = float(lemma_a1_A(phi))
    r = np.sqrt(1.0 - 4.0 * A)
    B1 = r * (np.sqrt(sig)[:, None] * U.T) @ ((1.0 / np.sqrt(lam1))[:, None] * Q1.T)
    B2 = r * ((1.0 / np.sqrt(sig))[:, None] * U.T) @ (np.sqrt(lam1)[:, None] * Q1.T)
    C1 = -(B1.T @ B1) / (2.0 * (1.0 - 4.0 * A))
    C2 = -(B2.T @ B2) / (2.0 * (1.0 - 4.0 * A))
    logD = 0.25 * d * np.log(1.0 - 4.0 * A)
    obj = d * (np.log(1.0 - 4.0 * A) - 0.5 * np.log(1.0 - 8.0 * A)
               + 2.0 / (1.0 - 8.0 * A) * (float(sig.sum()) / d + mu3) + 2.0 * mu3)
    return _pack("aderf", A * np.eye(d), B1, B2, C1, C2, logD, obj, phi)


def fit_sderf(st):
    """Symmetric DERF, Theorem 4.3: eigendecompose
    N = M1 + mu4 mu5^T + mu5 mu4^T + M2 with eigenvalues non-ascending,
    A_ll from Lemma A.1 per eigenvalue, B = (I-4A)^(1/2) Q3^T, C = -I/2."""
    d = st["d"]
    N = st["M1"] + np.outer(st["mu4"], st["mu5"]) + np.outer(st["mu5"], st["mu4"]) + st["M2"]
    lam, Q3 = np.linalg.eigh(N)
    order = np.argsort(-lam, kind="stable")
    lam, Q3 = lam[order], Q3[:, order]
    lam = np.maximum(lam, 0.0)          # N is PSD; rounding may give -1e-17
    a = lemma_a1_A(lam)
    B = np.sqrt(1.0 - 4.0 * a)[:, None] * Q3.T
    logD = 0.25 * float(np.sum(np.log(1.0 - 4.0 * a)))
    obj = float(np.sum(np.log(1.0 - 4.0 * a) - 0.5 * np.log(1.0 - 8.0 * a)
                       + (1.0 + 1.0 / (1.0 - 8.0 * a)) * lam)
                - np.trace(st["M1"]) - np.trace(st["M2"]))
    I = np.eye(d)
    return _pack("sderf", np.diag(a), B, B, -0.5 * I, -0.5 * I, logD, obj, lam)


FITS = {"posrf": fit_posrf, "gerf": fit_gerf, "saderf": fit_saderf,
        "aderf": fit_aderf, "sderf": fit_sderf}


def fit_params(X, Y, variant):
    return FITS[variant](set_statistics(X, Y))


# --------------------------------------------------------------------------
# Features (Section 4 definition, with the M^-1/2 of Section 2.1)
# --------------------------------------------------------------------------
def derf_log_features(X, Omega, A, B, C, logD):
    """log of P (or S): row i, column m =
    -1/2 log M + log D + w_m^T A w_m + w_m^T B x_i + x_i^T C x_i."""
    X = np.asarray(X, dtype=F64)
    Om = np.asarray(Omega, dtype=F64)
    M = Om.shape[0]
    a = np.einsum("md,de,me->m", Om, np.asarray(A, F64), Om)
    lin = X @ (Om @ np.asarray(B, F64)).T
    c = np.einsum("ld,de,le->l", X, np.asarray(C, F64), X)
    return -0.5 * np.log(M) + logD + a[None, :] + lin + c[:, None]


def derf_features(X, Omega, A, B, C, logD):
    """P (or S) of Section 2.1 for the DERF f of Section 4, no stabilisation."""
    return np.exp(derf_log_features(X, Omega, A, B, C, logD))


def features_pair(X, Y, Omega, p):
    """P = phi^(1)(X) and S = phi^(2)(Y)."""
    P = derf_features(X, Omega, p["A"], p["B1"], p["C1"], p["logD"])
    S = derf_features(Y, Omega, p["A"], p["B2"], p["C2"], p["logD"])
    return P, S


def posrf_features_direct(X, Omega):
    """Positive random features written straight from Section 2.3:
    M^-1/2 exp(w^T x - |x|^2 / 2).  Independent of derf_features."""
    X = np.asarray(X, dtype=F64)
    Om = np.asarray(Omega, dtype=F64)
    out = np.empty((X.shape[0], Om.shape[0]), dtype=F64)
    for i in range(X.shape[0]):
        for m in range(Om.shape[0]):
            out[i, m] = np.exp(np.dot(Om[m], X[i]) - 0.5 * np.dot(X[i], X[i]))
    return out / np.sqrt(Om.shape[0])


# --------------------------------------------------------------------------
# Attention (Section 2.2) on given feature matrices
# --------------------------------------------------------------------------
def attend_bidirectional(P, S, V):
    """Y = diag(Khat 1)^-1 Khat V with Khat = P S^T, evaluated in the
    O(L M n) order of Section 2.1: S^T [V | 1] first."""
    V = np.asarray(V, dtype=F64)
    V1 = np.concatenate([V, np.ones((V.shape[0], 1))], axis=1)
    KV = S.T @ V1
    out = P @ KV
    return out[:, :-1] / out[:, -1:]


def attend_bidirectional_explicit(P, S, V):
    """Same, with the L x L matrix Khat formed explicitly."""
    Khat = P @ S.T
    return (Khat @ np.asarray(V, F64)) / Khat.sum(axis=1, keepdims=True)


def attend_causal_explicit(P, S, V):
    """Lower-triangular (diagonal included) masked form:
    Y_i = sum_{j<=i} Khat_ij V_j / sum_{j<=i} Khat_ij."""
    Khat = np.tril(P @ S.T)
    return (Khat @ np.asarray(V, F64)) / Khat.sum(axis=1, keepdims=True)


def attend_causal_recurrent(P, S, V):
    """The same quantity token by token: T += S_j [V_j | 1]^T, then
    [num | den] = P_i^T T (update before read, so j = i is included)."""
    V = np.asarray(V, dtype=F64)
    L, M = P.shape
    n = V.shape[1]
    T = np.zeros((M, n + 1))
    out = np.empty((L, n))
    v1 = np.ones(n + 1)
    for i in range(L):
        v1[:n] = V[i]
        T += np.outer(S[i], v1)
        r = P[i] @ T
        out[i] = r[:n] / r[n]
    return out


def attend_causal_rows(P_rows, rows, S, V):
    """Selected rows of attend_causal_explicit: P_rows[k] is the feature row of
    query rows[k]; only keys j <= rows[k] enter."""
    V = np.asarray(V, dtype=F64)
    out = np.empty((len(rows), V.shape[1]))
    for k, i in enumerate(rows):
        w = S[: i + 1] @ P_rows[k]
        out[k] = (w @ V[: i + 1]) / w.sum()
    return out


def softmax_attention_exact(X, Y, V, causal=False):
    """Exact attention of Section 2.2 with kernel K(x,y) = exp(x^T y)."""
    X = np.asarray(X, F64)
    Y = np.asarray(Y, F64)
    Z = X @ Y.T
    if causal:
        Z = np.where(np.tril(np.ones_like(Z)) > 0, Z, -np.inf)
    Z = Z - Z.max(axis=1, keepdims=True)
    W = np.exp(Z)
    return (W @ np.asarray(V, F64)) / W.sum(axis=1, keepdims=True)


def favor_sharp_attention(Q, K, V, Omega, p, causal=False, qk_scale=1.0, rows=None):
    """End to end for one (batch, head): x = qk_scale Q_i, y = qk_scale K_j
    (Section 2.2 puts qk_scale = d^-1/4), features with parameters p, then
    attention.  rows selects query rows (all keys still enter)."""
    X = qk_scale * np.asarray(Q, F64)
    Y = qk_scale * np.asarray(K, F64)
    S = derf_features(Y, Omega, p["A"], p["B2"], p["C2"], p["logD"])
    if rows is None:
        P = derf_features(X, Omega, p["A"], p["B1"], p["C1"], p["logD"])
        return attend_causal_explicit(P, S, V) if causal else attend_bidirectional(P, S, V)
    rows = np.asarray(rows)
    P = derf_features(X[rows], Omega, p["A"], p["B1"], p["C1"], p["logD"])
    if causal:
        return attend_causal_rows(P, rows, S, V)
    return attend_bidirectional(P, S, V)


# --------------------------------------------------------------------------
# Backward pass (Section 5.3 trains Transformers through this attention): the
# vector-Jacobian product of favor_sharp_attention with the parameters held fixed
# --------------------------------------------------------------------------
def favor_sharp_attention_vjp(Q, K, V, dY, Omega, p, causal=False, qk_scale=1.0):
    """(dQ, dK, dV) = gradient of sum(dY * favor_sharp_attention(Q, K, V, ...)) for one
    (batch, head), Omega and the parameters p being constants.  The chain rule on the
    explicit L x L form of Section 2.2, step by step:

      Khat = P S^T (lower triangle when causal), den = Khat 1, Y = Khat V / den
      dNum = dY / den,  dden_i = -sum_c dY_ic Y_ic / den_i
      dKhat_ij = dNum_i . V_j + dden_i   (same mask),   dV = Khat^T dNum
      dP = dKhat S,  dS = dKhat^T P;  through the exponential: dlogP = dP * P, dlogS = dS * S
      log feature (Section 4): w^T B x + x^T C x + terms without x, so
      dx_i = sum_m dlog_im B^T w_m + (C + C^T) x_i sum_m dlog_im,  dQ = qk_scale dx.
    """
    X = qk_scale * np.asarray(Q, F64)
    Yk = qk_scale * np.asarray(K, F64)
    V = np.asarray(V, F64)
    dY = np.asarray(dY, F64)
    Om = np.asarray(Omega, F64)
    P = derf_features(X, Om, p["A"], p["B1"], p["C1"], p["logD"])
    S = derf_features(Yk, Om, p["A"], p["B2"], p["C2"], p["logD"])
    Khat = P @ S.T
    if causal:
        Khat = np.tril(Khat)
    den = Khat.sum(axis=1, keepdims=True)
    Yout = (Khat @ V) / den
    dNum = dY / den
    dden = -np.sum(dY * Yout, axis=1, keepdims=True) / den
    dKhat = dNum @ V.T + dden
    if causal:
        dKhat = np.tril(dKhat)
    dV = Khat.T @ dNum
    dlogP = (dKhat @ S) * P
    dlogS = (dKhat.T @ P) * S
    C1 = np.asarray(p["C1"], F64)
    C2 = np.asarray(p["C2"], F64)
    dX = dlogP @ (Om @ np.asarray(p["B1"], F64)) + dlogP.sum(axis=1, keepdims=True) * (X @ (C1 + C1.T))
    dYk = dlogS @ (Om @ np.asarray(p["B2"], F64)) + dlogS.sum(axis=1, keepdims=True) * (Yk @ (C2 + C2.T))
    return qk_scale * dX, qk_scale * dYk, dV


# --------------------------------------------------------------------------
# Kernel estimation for pairs (Section 2.1 estimator, Section 5.1 setting)
# --------------------------------------------------------------------------
def pair_estimate(X, Y, Omega, p):
    """Khat(x_p, y_p) = sum_m P_pm S_pm for each pair p (row p of X with row p of Y)."""
    P, S = features_pair(X, Y, Omega, p)
    return np.sum(P * S, axis=1)


def pair_closed_form_variance(X, Y, p, M):
    """Per-pair Var Khat = Var_w[f1 f2] / M (Section 2.1) with Theorem 4.1's variance."""
    X = np.asarray(X, F64)
    Y = np.asarray(Y, F64)
    return np.array([derf_variance(X[i], Y[i], p) for i in range(X.shape[0])]) / M


def pair_pooled_relative_variance(est, X, Y, var_cf):
    """The two pooled numbers of the variance study (Section 5.1), for one parameterisation:
    mean over pairs of (sample variance of Khat over the R feature draws) / K^2, and
    mean over pairs of (Theorem 4.1's variance / M) / K^2, with K = exp(x^T y) (Section 2.1, alpha = 0).
    est: (R, npairs) estimates, one row per draw; var_cf: (npairs,) from pair_closed_form_variance.
    The sample variance is the unbiased one (divisor R - 1)."""
    est = np.asarray(est, F64)
    X = np.asarray(X, F64)
    Y = np.asarray(Y, F64)
    K2 = np.exp(2.0 * np.sum(X * Y, axis=1))
    emp = est.var(axis=0, ddof=1) / K2
    return float(emp.mean()), float((np.asarray(var_cf, F64) / K2).mean())


# --------------------------------------------------------------------------
# The unnormalised operator (Section 2.1), scaled softmax kernel K^(alpha)
# --------------------------------------------------------------------------
def kernel_matrix_exact(X, Y, alpha):
    """K^(alpha)(x, y) = exp(alpha |x|^2 + x^T y + alpha |y|^2) (Section 2.1) for all pairs: (Lx, Ly)."""
    X = np.asarray(X, F64)
    Y = np.asarray(Y, F64)
    return np.exp(alpha * np.sum(X * X, axis=1)[:, None] + X @ Y.T + alpha * np.sum(Y * Y, axis=1)[None, :])


def kernel_apply(X, Y, Cmat, Omega, p, alpha):
    """Khat^(alpha)(X, Y) C with Khat = P S^T (Section 2.1), P and S built from fhat = exp(alpha |x|^2) f
    (Section 2.3), evaluated in the O(L M n) order P (S^T C)."""
    X = np.asarray(X, F64)
    Y = np.asarray(Y, F64)
    P, S = features_pair(X, Y, Omega, p)
    P = P * np.exp(alpha * np.sum(X * X, axis=1))[:, None]
    S = S * np.exp(alpha * np.sum(Y * Y, axis=1))[:, None]
    return P @ (S.T @ np.asarray(Cmat, F64))
