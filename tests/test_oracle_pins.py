"""Pins for the fp64 checker: each test ties a function of oracle/favor_sharp.py to
something other than itself -- quadrature, Monte Carlo, a hand-worked closed form,
a brute-force double sum, or a special case that reduces to a textbook routine."""
import os

import numpy as np
import pytest

from oracle import favor_sharp as fs

HERE = os.path.dirname(os.path.abspath(__file__))


# ------------------------------------------------------------------ helpers
def random_valid_derf(rng, d, a_lo=-0.4, a_hi=0.07, dense_A=True):
    """Random parameters satisfying the conditions of Theorem 4.1."""
    if dense_A:
        Qr, _ = np.linalg.qr(rng.standard_normal((d, d)))
        A = Qr @ np.diag(rng.uniform(a_lo, a_hi, d)) @ Qr.T
    else:
        A = np.diag(rng.uniform(a_lo, a_hi, d))
    I = np.eye(d)
    B1 = rng.standard_normal((d, d)) + 1.5 * I
    B2 = (I - 4 * A) @ np.linalg.inv(B1).T          # B1^T (I-4A)^-1 B2 = I
    Sinv = np.linalg.inv(I - 4 * A)
    C1 = -0.5 * B1.T @ Sinv @ B1
    C2 = -0.5 * B2.T @ Sinv @ B2
    logD = 0.25 * np.linalg.slogdet(I - 4 * A)[1]
    return {"A": A, "B1": B1, "B2": B2, "C1": C1, "C2": C2, "logD": logD}


def gauss_hermite_nodes(d, n):
    """Tensor-product nodes/weights for E_{w ~ N(0, I_d)}[g(w)]."""
    x, w = np.polynomial.hermite_e.hermegauss(n)
    w = w / np.sqrt(2 * np.pi)
    grids = np.meshgrid(*([x] * d), indexing="ij")
    nodes = np.stack([g.ravel() for g in grids], axis=1)
    wg = np.meshgrid(*([w] * d), indexing="ij")
    weights = np.prod(np.stack([g.ravel() for g in wg], axis=1), axis=1)
    return nodes, weights


def toy_sets(rng, L, d, shift=0.3, scale=0.5):
    X = scale * rng.standard_normal((L, d)) * rng.uniform(0.5, 1.5, d)
    Y = scale * rng.standard_normal((L, d)) * rng.uniform(0.5, 1.5, d) + shift
    return X, Y


# ------------------------------------------------------------------ Lemma A.1
def test_lemma_a1_golden_surds():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "lemma_a1_values.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for phi, p, q, r in rows:
        expect = (float(p) + float(q) * np.sqrt(float(r))) / 16.0
        assert abs(fs.lemma_a1_A(float(phi)) - expect) < 1e-15


def test_lemma_a1_is_the_minimiser():
    for phi in [0.0, 1e-6, 0.01, 0.3, 1.0, 7.0, 50.0]:
        A = float(fs.lemma_a1_A(phi))
        assert A <= 0.0 and 1 - 8 * A >= 1.0
        # stationarity, central difference on f
        h = 1e-5 * max(1.0, abs(A))
        g = (fs.lemma_a1_objective(A + h, phi) - fs.lemma_a1_objective(A - h, phi)) / (2 * h)
        assert abs(g) < 1e-7
        # beats a fine grid over (-inf, 1/8)
        grid = np.concatenate([-np.logspace(-6, 3, 4000), np.linspace(0, 0.1249, 500)])
        assert fs.lemma_a1_objective(A, phi) <= fs.lemma_a1_objective(grid, phi).min() + 1e-12
    assert fs.lemma_a1_A(0.0) == 0.0


# ------------------------------------------------------------------ Theorem 4.1
@pytest.mark.parametrize("d,n", [(1, 160), (2, 90)])
def test_unbiasedness_and_variance_by_quadrature(d, n):
    """E[f1 f2] = exp(x^T y) and the variance formula, by Gauss-Hermite quadrature.
    The features come from derf_features, so a wrong sign, a transposed B or a
    dropped C term fails here."""
    rng = np.random.default_rng(10 + d)
    nodes, wts = gauss_hermite_nodes(d, n)
    Mq = nodes.shape[0]
    for _ in range(4):
        p = random_valid_derf(rng, d, a_lo=-0.3, a_hi=0.03)
        x = 0.6 * rng.standard_normal(d)
        y = 0.6 * rng.standard_normal(d)
        P = fs.derf_features(x[None], nodes, p["A"], p["B1"], p["C1"], p["logD"])[0]
        S = fs.derf_features(y[None], nodes, p["A"], p["B2"], p["C2"], p["logD"])[0]
        prod = P * S * Mq                       # undo the two M^-1/2 factors
        mean = np.sum(wts * prod)
        assert abs(mean / np.exp(x @ y) - 1) < 1e-9
        second = np.sum(wts * prod ** 2)
        var = second - np.exp(2 * x @ y)
        ref = fs.derf_variance(x, y, p)
        assert abs(var - ref) < 1e-7 * max(1.0, second)


def test_unbiasedness_monte_carlo_small_d():
    """Brute-force Monte Carlo, iid omegas, d = 3 and 4: the sample mean of the
    estimator is within 4 standard errors of exp(x^T y), the standard error taken
    from Theorem 4.1's variance; the sample variance agrees with that formula."""
    rng = np.random.default_rng(5)
    nsamp = 1_500_000
    for d in (3, 4):
        p = random_valid_derf(rng, d, a_lo=-0.3, a_hi=0.0)
        x = 0.35 * rng.standard_normal(d)
        y = 0.35 * rng.standard_normal(d)
        Om = rng.standard_normal((nsamp, d))
        P = fs.derf_features(x[None], Om, p["A"], p["B1"], p["C1"], p["logD"])[0]
        S = fs.derf_features(y[None], Om, p["A"], p["B2"], p["C2"], p["logD"])[0]
        z = P * S * nsamp
        var = fs.derf_variance(x, y, p)
        se = np.sqrt(var / nsamp)
        assert abs(z.mean() - np.exp(x @ y)) < 4 * se
        assert abs(z.var() / var - 1) < 0.1
        # estimator form: Khat = sum_m P_m S_m equals the sample mean
        assert abs(fs.pair_estimate(x[None], y[None], Om, p)[0] - z.mean()) < 1e-12


def test_posrf_special_case_reproduces_direct_formula():
    rng = np.random.default_rng(3)
    d, L, M = 5, 7, 11
    X = rng.standard_normal((L, d))
    Om = rng.standard_normal((M, d))
    p = fs.fit_posrf(fs.set_statistics(X, X))
    assert np.all(p["A"] == 0) and p["logD"] == 0.0
    got = fs.derf_features(X, Om, p["A"], p["B1"], p["C1"], p["logD"])
    ref = fs.posrf_features_direct(X, Om)
    assert np.max(np.abs(got / ref - 1)) < 1e-14


def test_scalar_variance_formula_agrees_with_dense_one():
    rng = np.random.default_rng(4)
    d = 6
    for A in (-0.7, -0.05, 0.0, 0.06):
        I = np.eye(d)
        B = np.sqrt(1 - 4 * A)
        p = {"A": A * I, "B1": B * I, "B2": B * I, "C1": -0.5 * I, "C2": -0.5 * I,
             "logD": 0.25 * d * np.log(1 - 4 * A)}
        x = 0.5 * rng.standard_normal(d)
        y = 0.5 * rng.standard_normal(d)
        assert abs(fs.derf_variance(x, y, p) / fs.gerf_variance(A, x, y) - 1) < 1e-12


def test_empirical_variance_matches_closed_form():
    """Variance of Khat over independent draws of M iid omegas = Var/M."""
    rng = np.random.default_rng(8)
    d, M, R = 4, 16, 60000
    X, Y = toy_sets(rng, 32, d, shift=0.1, scale=0.3)
    for variant in ("posrf", "gerf", "aderf", "sderf"):
        p = fs.fit_params(X, Y, variant)
        x, y = X[:1], Y[:1]
        Om = rng.standard_normal((R * M, d))
        P, S = fs.features_pair(x, y, Om, p)
        est = (P * S * (R * M)).reshape(R, M).mean(axis=1)
        cf = fs.pair_closed_form_variance(x, y, p, M)[0]
        assert abs(est.var() / cf - 1) < 0.08, variant
        assert abs(est.mean() / np.exp(x[0] @ y[0]) - 1) < 4 * np.sqrt(cf / R) / np.exp(x[0] @ y[0])


def test_pooled_relative_variances_agree_on_small_norm_iid_draws():
    """Pooled over pairs, the empirical relative variance over R draws of M iid omegas agrees with the pooled
    closed form (Theorem 4.1 / M) -- small norms and small d, where the summands have light tails -- and the
    pooled numbers equal their definitions written out pair by pair."""
    rng = np.random.default_rng(44)
    d, M, R, npairs = 4, 8, 100000, 16
    X, Y = toy_sets(rng, npairs, d, shift=0.1, scale=0.3)
    Om = rng.standard_normal((R * M, d))            # R independent draws of M iid omegas, side by side
    for variant in ("posrf", "gerf", "aderf", "sderf"):
        p = fs.fit_params(X, Y, variant)
        P, S = fs.features_pair(X, Y, Om, p)         # scaled by (R M)^-1/2: undo, then average each draw's M features
        est = (P * S * (R * M)).reshape(npairs, R, M).mean(axis=2).T
        cf = fs.pair_closed_form_variance(X, Y, p, M)
        emp_pooled, cf_pooled = fs.pair_pooled_relative_variance(est, X, Y, cf)
        assert abs(emp_pooled / cf_pooled - 1) < 0.05, variant
        # definitions, one pair at a time
        e2 = c2 = 0.0
        for i in range(npairs):
            K = np.exp(X[i] @ Y[i])
            m = est[:, i].sum() / R
            e2 += ((est[:, i] - m) ** 2).sum() / (R - 1) / K ** 2
            c2 += cf[i] / K ** 2
        assert abs(emp_pooled - e2 / npairs) < 1e-12 * abs(emp_pooled)
        assert abs(cf_pooled - c2 / npairs) < 1e-12 * abs(cf_pooled)


def test_unnormalised_operator_converges_to_the_exact_kernel_matrix():
    """Khat^(alpha) C approaches K^(alpha) C as M grows, at rate M^-1/2, for the softmax (alpha = 0) and the
    Gaussian kernel (alpha = -1/2); the exact Gaussian kernel matrix is exp(-|x - y|^2 / 2); and the result equals
    the explicit L x L form."""
    rng = np.random.default_rng(90)
    d, L, n = 4, 24, 3
    X, Y = toy_sets(rng, L, d, shift=0.1, scale=0.4)
    Cm = rng.standard_normal((L, n))
    D2 = ((X[:, None, :] - Y[None, :, :]) ** 2).sum(axis=2)
    assert np.abs(fs.kernel_matrix_exact(X, Y, -0.5) - np.exp(-0.5 * D2)).max() < 1e-14
    assert np.abs(fs.kernel_matrix_exact(X, Y, 0.0) - np.exp(X @ Y.T)).max() < 1e-14
    for variant in ("posrf", "sderf", "aderf"):
        p = fs.fit_params(X, Y, variant)
        for alpha in (0.0, -0.5):
            exact = fs.kernel_matrix_exact(X, Y, alpha) @ Cm
            errs = []
            for M in (64, 4096, 262144):
                Om = rng.standard_normal((M, d))
                got = fs.kernel_apply(X, Y, Cm, Om, p, alpha)
                errs.append(np.abs(got - exact).max() / np.abs(exact).max())
                if M == 64:                                   # explicit form: every entry of Khat, then the product
                    P, S = fs.features_pair(X, Y, Om, p)
                    Kh = (P @ S.T) * fs.kernel_matrix_exact(X, Y, alpha) / np.exp(X @ Y.T)
                    assert np.abs(got - Kh @ Cm).max() < 1e-12 * np.abs(got).max()
            assert errs[2] < 0.02 and errs[2] < errs[0] / 8, (variant, alpha, errs)


# ------------------------------------------------------------------ fits
def thm41_residuals(p):
    d = p["A"].shape[0]
    I = np.eye(d)
    Sinv = np.linalg.inv(I - 4 * p["A"])
    r = [np.abs(p["B1"].T @ Sinv @ p["B2"] - I).max(),
         np.abs(p["C1"] + 0.5 * p["B1"].T @ Sinv @ p["B1"]).max(),
         np.abs(p["C2"] + 0.5 * p["B2"].T @ Sinv @ p["B2"]).max(),
         abs(p["logD"] - 0.25 * np.linalg.slogdet(I - 4 * p["A"])[1])]
    assert np.linalg.eigvalsh(p["A"]).max() < 1 / 8
    return max(r)


@pytest.mark.parametrize("variant", ["posrf", "gerf", "saderf", "aderf", "sderf"])
def test_fits_are_valid_and_objective_matches_brute_force(variant):
    rng = np.random.default_rng(21)
    X, Y = toy_sets(rng, 24, 5)
    p = fs.fit_params(X, Y, variant)
    assert thm41_residuals(p) < 1e-12
    brute = fs.shifted_log_variance_bruteforce(X, Y, p)
    assert abs(p["objective"] - brute) < 1e-10 * max(1.0, abs(brute))


def test_objective_ordering_of_the_families():
    rng = np.random.default_rng(22)
    for trial in range(5):
        X, Y = toy_sets(rng, 40, 6, shift=0.4 * trial)
        o = {v: fs.fit_params(X, Y, v)["objective"] for v in fs.FITS}
        eps = 1e-12
        assert o["sderf"] <= o["gerf"] + eps <= o["posrf"] + 2 * eps
        assert o["aderf"] <= o["saderf"] + eps <= o["gerf"] + 2 * eps


def _sym_expm(S):
    lam, Q = np.linalg.eigh(S)
    return Q @ np.diag(np.exp(lam)) @ Q.T


def test_aderf_is_a_minimum_within_its_family():
    """Random feasible perturbations (A scalar < 1/8, E = B1^T B1 SPD, B2 from the
    constraint) never lower the brute-force objective."""
    rng = np.random.default_rng(23)
    d = 4
    X, Y = toy_sets(rng, 16, d)
    p = fs.fit_params(X, Y, "aderf")
    base = fs.shifted_log_variance_bruteforce(X, Y, p)
    A0 = p["A"][0, 0]
    I = np.eye(d)
    for t in (1e-3, 1e-2, 0.1, 0.5):
        for _ in range(6):
            Dl = rng.standard_normal((d, d))
            Dl = 0.5 * (Dl + Dl.T)
            A = min(A0 + t * rng.standard_normal() * 0.3, 0.12)
            B1 = p["B1"] @ _sym_expm(t * Dl) * np.sqrt((1 - 4 * A) / (1 - 4 * A0))
            B2 = (1 - 4 * A) * np.linalg.inv(B1).T
            q = {"A": A * I, "B1": B1, "B2": B2,
                 "C1": -B1.T @ B1 / (2 * (1 - 4 * A)), "C2": -B2.T @ B2 / (2 * (1 - 4 * A)),
                 "logD": 0.25 * d * np.log(1 - 4 * A)}
            assert thm41_residuals(q) < 1e-10
            assert fs.shifted_log_variance_bruteforce(X, Y, q) >= base - 1e-11


def test_aderf_phi_carries_the_factor_two():
    """With E fixed at its optimum the objective is a function of the scalar A alone;
    the fitted A must minimise it over a fine grid.  Dropping the factor 2 in
    phi = 2/d sum Sigma + 2 mu3 moves A away from the grid minimum."""
    rng = np.random.default_rng(24)
    d = 4
    X, Y = toy_sets(rng, 16, d)
    st = fs.set_statistics(X, Y)
    p = fs.fit_aderf(st)
    A0 = p["A"][0, 0]
    F = p["B1"].T @ p["B1"] / (1 - 4 * A0)
    assert np.abs(F @ st["M1"] @ F - st["M2"]).max() < 1e-10        # proof of Thm 4.2
    sig_sum = (p["phi"] - 2 * st["mu3"]) * d / 2
    assert abs(np.trace(F @ st["M1"]) - sig_sum) < 1e-10
    I = np.eye(d)
    lamF, QF = np.linalg.eigh(F)
    Fh = QF @ np.diag(np.sqrt(lamF)) @ QF.T

    def obj(A):
        B1 = np.sqrt(1 - 4 * A) * Fh
        B2 = np.sqrt(1 - 4 * A) * np.linalg.inv(Fh)
        q = {"A": A * I, "B1": B1, "B2": B2, "C1": -0.5 * F, "C2": -0.5 * np.linalg.inv(F),
             "logD": 0.25 * d * np.log(1 - 4 * A)}
        return fs.shifted_log_variance_bruteforce(X[:8], Y[:8], q)

    # the same 8x8 subsample for grid and optimum: refit on it so the optimum applies
    p8 = fs.fit_params(X[:8], Y[:8], "aderf")
    A8 = p8["A"][0, 0]
    F8 = p8["B1"].T @ p8["B1"] / (1 - 4 * A8)
    lamF, QF = np.linalg.eigh(F8)
    Fh = QF @ np.diag(np.sqrt(lamF)) @ QF.T
    F = F8
    grid = A8 + np.linspace(-0.2, 0.2, 81) * abs(A8)
    vals = np.array([obj(a) for a in grid])
    assert abs(grid[vals.argmin()] - A8) <= 0.0026 * abs(A8)
    assert abs(obj(A8) - p8["objective"]) < 1e-10


def test_sderf_is_a_minimum_within_its_family():
    rng = np.random.default_rng(25)
    d = 4
    X, Y = toy_sets(rng, 16, d, shift=0.5)
    p = fs.fit_params(X, Y, "sderf")
    base = fs.shifted_log_variance_bruteforce(X, Y, p)
    a0 = np.diag(p["A"])
    Q0 = p["B1"] / np.sqrt(1 - 4 * a0)[:, None]
    assert np.abs(Q0 @ Q0.T - np.eye(d)).max() < 1e-12
    assert np.all(np.diff(a0) >= -1e-15)      # eigenvalues non-ascending => A non-descending
    I = np.eye(d)
    for t in (1e-3, 1e-2, 0.1, 0.6):
        for _ in range(6):
            K = rng.standard_normal((d, d))
            K = t * (K - K.T)
            # Cayley transform: an orthogonal matrix near I
            R = np.linalg.solve(I - 0.5 * K, I + 0.5 * K)
            a = np.minimum(a0 + t * 0.2 * rng.standard_normal(d), 0.12)
            B = np.sqrt(1 - 4 * a)[:, None] * (Q0 @ R)
            q = {"A": np.diag(a), "B1": B, "B2": B, "C1": -0.5 * I, "C2": -0.5 * I,
                 "logD": 0.25 * np.sum(np.log(1 - 4 * a))}
            assert thm41_residuals(q) < 1e-10
            assert fs.shifted_log_variance_bruteforce(X, Y, q) >= base - 1e-11


def test_containments_on_isotropic_sets():
    """Sets with M1 = M2 = m I and zero means: ADERF, SADERF and SDERF all reduce to
    GERF (same scalar A, same objective)."""
    d, a = 5, 0.7
    X = np.concatenate([a * np.eye(d), -a * np.eye(d)])
    Y = X.copy()
    st = fs.set_statistics(X, Y)
    assert np.abs(st["M1"] - a * a / d * np.eye(d)).max() < 1e-15
    g = fs.fit_gerf(st)
    for v in ("saderf", "aderf", "sderf"):
        p = fs.FITS[v](st)
        assert abs(p["objective"] - g["objective"]) < 1e-12, v
        assert np.abs(np.diag(p["A"]) - g["A"][0, 0]).max() < 1e-14, v
        assert abs(p["logD"] - g["logD"]) < 1e-13, v
    s = fs.fit_saderf(st)
    assert np.abs(s["B1"] - g["B1"]).max() < 1e-14


def test_saderf_psi_is_the_stated_ratio():
    rng = np.random.default_rng(26)
    X, Y = toy_sets(rng, 30, 4)
    p = fs.fit_params(X, Y, "saderf")
    psi = (np.sum(Y ** 2, axis=0) / np.sum(X ** 2, axis=0)) ** 0.25
    b = np.sqrt(1 - 4 * p["A"][0, 0])
    assert np.abs(np.diag(p["B1"]) - b * psi).max() < 1e-13
    assert np.abs(np.diag(p["B2"]) - b / psi).max() < 1e-13


# ------------------------------------------------------------------ attention
def _features_for_attention(rng, L, d, M, variant="sderf"):
    X, Y = toy_sets(rng, L, d)
    V = rng.standard_normal((L, d))
    Om = rng.standard_normal((M, d))
    p = fs.fit_params(X, Y, variant)
    P, S = fs.features_pair(X, Y, Om, p)
    return X, Y, V, Om, p, P, S


def test_bidirectional_forms_agree_and_are_right_stochastic():
    rng = np.random.default_rng(31)
    X, Y, V, Om, p, P, S = _features_for_attention(rng, 40, 6, 24, "aderf")
    a = fs.attend_bidirectional(P, S, V)
    b = fs.attend_bidirectional_explicit(P, S, V)
    assert np.abs(a - b).max() < 1e-12
    assert np.all(P > 0) and np.all(S > 0)
    ones = fs.attend_bidirectional(P, S, np.ones_like(V))
    assert np.abs(ones - 1).max() < 1e-13
    perm = rng.permutation(40)
    c = fs.attend_bidirectional(P, S[perm], V[perm])
    assert np.abs(a - c).max() < 1e-12
    # Y is a convex combination of rows of V
    assert a.max() <= V.max() + 1e-12 and a.min() >= V.min() - 1e-12


def test_causal_forms_agree():
    rng = np.random.default_rng(32)
    X, Y, V, Om, p, P, S = _features_for_attention(rng, 33, 5, 16)
    a = fs.attend_causal_explicit(P, S, V)
    b = fs.attend_causal_recurrent(P, S, V)
    rows = [0, 1, 7, 32]
    c = fs.attend_causal_rows(P[rows], rows, S, V)
    assert np.abs(a - b).max() < 1e-12
    assert np.abs(a[rows] - c).max() < 1e-12
    assert np.abs(a[0] - V[0]).max() < 1e-13          # first token sees only itself
    # brute force on the definition, row by row
    for i in (3, 20):
        w = np.array([P[i] @ S[j] for j in range(i + 1)])
        assert np.abs(a[i] - (w[:, None] * V[: i + 1]).sum(0) / w.sum()).max() < 1e-12
    # future tokens do not matter
    S2, V2 = S.copy(), V.copy()
    S2[20:] *= 3.0
    V2[20:] += 1.0
    a2 = fs.attend_causal_explicit(P, S2, V2)
    assert np.abs(a2[:20] - a[:20]).max() < 1e-13


def test_end_to_end_wrapper_matches_pieces():
    rng = np.random.default_rng(33)
    X, Y, V, Om, p, P, S = _features_for_attention(rng, 20, 4, 8, "aderf")
    full = fs.favor_sharp_attention(X, Y, V, Om, p, causal=True)
    assert np.abs(full - fs.attend_causal_explicit(P, S, V)).max() < 1e-13
    rows = [2, 11]
    assert np.abs(fs.favor_sharp_attention(X, Y, V, Om, p, causal=True, rows=rows) - full[rows]).max() < 1e-12
    fb = fs.favor_sharp_attention(X, Y, V, Om, p, causal=False)
    assert np.abs(fs.favor_sharp_attention(X, Y, V, Om, p, causal=False, rows=rows) - fb[rows]).max() < 1e-12
    # qk_scale is applied to Q and K before everything else
    fq = fs.favor_sharp_attention(2 * X, 2 * Y, V, Om, p, causal=False, qk_scale=0.5)
    assert np.abs(fq - fb).max() < 1e-13


def test_linear_attention_approaches_softmax_attention_as_M_grows():
    rng = np.random.default_rng(34)
    d, L = 8, 48
    X, Y = toy_sets(rng, L, d, shift=0.1, scale=0.45)
    V = rng.standard_normal((L, d))
    exact = fs.softmax_attention_exact(X, Y, V)
    # exact attention itself: softmax of the Gram matrix, checked on one row by hand
    w = np.exp(X[5] @ Y.T)
    assert np.abs(exact[5] - w @ V / w.sum()).max() < 1e-13
    p = fs.fit_params(X, Y, "sderf")
    errs = []
    for M in (32, 512, 8192):
        e = []
        for s in range(6):
            Om = np.random.default_rng(100 * M + s).standard_normal((M, d))
            e.append(np.sqrt(np.mean((fs.favor_sharp_attention(X, Y, V, Om, p) - exact) ** 2)))
        errs.append(np.mean(e))
    assert errs[0] > 2.5 * errs[1] > 2.5 * 2.5 * errs[2] * 0.999
    # rate close to M^-1/2: a 256x larger M gives roughly a 16x smaller error
    assert 8 < errs[0] / errs[2] < 32
    # causal variant converges to causal softmax attention too
    ec = fs.softmax_attention_exact(X, Y, V, causal=True)
    Om = np.random.default_rng(7).standard_normal((8192, d))
    assert np.sqrt(np.mean((fs.favor_sharp_attention(X, Y, V, Om, p, causal=True) - ec) ** 2)) < 2.5 * errs[2]


def test_sderf_variance_gain_on_heterogeneous_sets():
    """Soft sanity on magnitudes: on shifted ('heterogen'-like) sets SDERF's mean log
    second moment sits well below GERF's."""
    rng = np.random.default_rng(35)
    d, L, sigma = 16, 64, 0.5
    X = sigma * rng.standard_normal((L, d))
    Y = sigma * rng.standard_normal((L, d)) + sigma
    g = fs.fit_params(X, Y, "gerf")["objective"]
    s = fs.fit_params(X, Y, "sderf")["objective"]
    assert s < g - 0.5


# ------------------------------------------------------------------ backward pass
def _vjp_case(seed, causal, L=11, d=4, M=8, dv=3):
    rng = np.random.default_rng(seed)
    p = random_valid_derf(rng, d)
    # a C that is not symmetric, so that (C + C^T) is told apart from 2 C
    p["C1"] = p["C1"] + 0.05 * rng.standard_normal((d, d))
    p["C2"] = p["C2"] + 0.05 * rng.standard_normal((d, d))
    Om = rng.standard_normal((M, d))
    Q = 0.6 * rng.standard_normal((L, d))
    K = 0.6 * rng.standard_normal((L, d))
    V = rng.standard_normal((L, dv))
    dY = rng.standard_normal((L, dv))
    return Q, K, V, dY, Om, p


@pytest.mark.parametrize("causal", [False, True])
def test_attention_vjp_matches_central_differences(causal):
    """The gradient formulas against the numerical derivative of the (pinned) forward function."""
    Q, K, V, dY, Om, p = _vjp_case(31, causal)
    qk = 0.8
    dQ, dK, dV = fs.favor_sharp_attention_vjp(Q, K, V, dY, Om, p, causal=causal, qk_scale=qk)

    def loss(q, k, v):
        return float(np.sum(dY * fs.favor_sharp_attention(q, k, v, Om, p, causal=causal, qk_scale=qk)))

    h = 1e-5
    for arr, grad, which in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            a_p = arr.copy(); a_p[idx] += h
            a_m = arr.copy(); a_m[idx] -= h
            args_p = [Q, K, V]; args_p[which] = a_p
            args_m = [Q, K, V]; args_m[which] = a_m
            num[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        assert np.max(np.abs(num - grad)) <= 2e-7 * max(1.0, np.max(np.abs(grad)))


@pytest.mark.parametrize("causal", [False, True])
def test_attention_vjp_closed_form_properties(causal):
    """Y(V + 1 c^T) = Y + 1 c^T, so the column sums of dV equal those of dY; Y does not move when all
    queries (or all keys) are featurised with a common extra factor, which the x^T C x term of the
    queries is per row: dQ is the same with C1 replaced by any other matrix."""
    Q, K, V, dY, Om, p = _vjp_case(32, causal)
    dQ, dK, dV = fs.favor_sharp_attention_vjp(Q, K, V, dY, Om, p, causal=causal)
    assert np.allclose(dV.sum(axis=0), dY.sum(axis=0), rtol=1e-10, atol=1e-12)
    p2 = dict(p); p2["C1"] = np.zeros_like(p["C1"])
    dQ2, dK2, dV2 = fs.favor_sharp_attention_vjp(Q, K, V, dY, Om, p2, causal=causal)
    assert np.allclose(dQ, dQ2, rtol=1e-9, atol=1e-12)
    assert np.allclose(dK, dK2, rtol=1e-9, atol=1e-12) and np.allclose(dV, dV2, rtol=1e-9, atol=1e-12)


def test_causal_attention_vjp_sees_no_future():
    """A cotangent on row i alone: no gradient reaches keys or values after i, nor any other query."""
    Q, K, V, dY, Om, p = _vjp_case(33, True)
    i = 6
    dY1 = np.zeros_like(dY); dY1[i] = dY[i]
    dQ, dK, dV = fs.favor_sharp_attention_vjp(Q, K, V, dY1, Om, p, causal=True)
    assert np.all(dK[i + 1:] == 0) and np.all(dV[i + 1:] == 0)
    assert np.all(np.delete(dQ, i, axis=0) == 0)
    assert np.any(dK[: i + 1] != 0) and np.any(dV[: i + 1] != 0) and np.any(dQ[i] != 0)
