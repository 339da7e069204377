"""Derives the coefficients of exp2_poly (tc_common.cuh): the cubic p with p(0) = 1 that minimises the
largest relative error of p(f) against 2^f on [0, 1), by a Remez exchange on the three free coefficients.

    python exp2_poly_fit.py        prints c1, c2, c3 (as float32) and the error bound

2^x for any x is then 2^floor(x) * p(x - floor(x)); the factor 2^floor(x) is an integer added to the
exponent field.  A relative error near 1e-4 is far below the 2^-9 rounding of the bf16 features.
"""
import numpy as np


def fit(deg=3, iters=50):
    # p(f) = 1 + c1 f + ... ; error e(f) = p(f) 2^-f - 1, equioscillating at deg + 1 points
    x = np.linspace(0.0, 1.0, deg + 3)[1:-1] if deg + 1 <= 2 else 0.5 - 0.5 * np.cos(np.pi * (np.arange(deg + 1) + 0.5) / (deg + 1))
    grid = np.linspace(0.0, 1.0, 200001)
    for _ in range(iters):
        # solve sum_k c_k x^k 2^-x - (1 - 2^-x) = (-1)^i E   (i = 0..deg)  for c_1..c_deg and E
        A = np.zeros((deg + 1, deg + 1))
        for k in range(1, deg + 1):
            A[:, k - 1] = x ** k * 2.0 ** -x
        A[:, deg] = -((-1.0) ** np.arange(deg + 1))
        rhs = 1.0 - 2.0 ** -x
        sol = np.linalg.solve(A, rhs)
        c = sol[:deg]
        err = (1.0 + sum(c[k - 1] * grid ** k for k in range(1, deg + 1))) * 2.0 ** -grid - 1.0
        # new reference: the extremum of each sign-constant stretch
        sgn = np.sign(err)
        idx = np.flatnonzero(np.diff(sgn) != 0)
        bounds = np.concatenate([[0], idx + 1, [len(grid)]])
        ext = [lo + np.argmax(np.abs(err[lo:hi])) for lo, hi in zip(bounds[:-1], bounds[1:]) if hi > lo]
        if len(ext) < deg + 1:
            break
        # keep the deg + 1 largest consecutive extrema
        ext = np.array(ext)
        if len(ext) > deg + 1:
            best = max(range(len(ext) - deg), key=lambda s: np.min(np.abs(err[ext[s:s + deg + 1]])))
            ext = ext[best:best + deg + 1]
        xn = grid[ext]
        if np.allclose(xn, x, atol=1e-9):
            break
        x = xn
    return c, np.abs(err).max()


if __name__ == "__main__":
    c, e = fit(3)
    c32 = c.astype(np.float32)
    g = np.linspace(0, 1, 100001).astype(np.float32)
    p = np.float32(1) + g * (c32[0] + g * (c32[1] + g * c32[2]))
    e32 = np.abs(p.astype(np.float64) * 2.0 ** -g.astype(np.float64) - 1).max()
    print("c1, c2, c3 =", ", ".join(repr(float(v)) for v in c32))
    print("max relative error: exact coefficients %.3e, float32 evaluation %.3e" % (e, e32))
