"""Prints the coefficients used by theory_math.cuh: a degree-7 polynomial P with
acos(x) ~= sqrt(1 - x) * P(x) on [0, 1] (the form of Abramowitz & Stegun 4.4.46), fitted here by
interpolation at Chebyshev nodes followed by a few Remez-style exchange steps, in float64.

    python paper_2602_02199_b200/csrc/acos_poly.py
"""
import numpy as np


def target(x):
    x = np.asarray(x, dtype=np.float64)
    out = np.empty_like(x)
    near = x > 1 - 1e-9
    out[~near] = np.arccos(x[~near]) / np.sqrt(1 - x[~near])
    out[near] = np.sqrt(2.0) * (1 + (1 - x[near]) / 12)      # series of acos at 1
    return out


def fit(deg=7, iters=12):
    n = deg + 2
    k = np.arange(n)
    nodes = 0.5 - 0.5 * np.cos(np.pi * k / (n - 1))          # Chebyshev extrema on [0, 1]
    grid = np.linspace(0.0, 1.0, 200001)
    for _ in range(iters):
        # solve P(x_i) + (-1)^i E = f(x_i)
        A = np.hstack([np.vander(nodes, deg + 1, increasing=True), ((-1.0) ** k)[:, None]])
        sol = np.linalg.solve(A, target(nodes))
        coef = sol[:-1]
        err = np.polyval(coef[::-1], grid) - target(grid)
        # exchange: new nodes at the extrema of the error between sign changes
        sign = np.sign(err)
        edges = np.flatnonzero(sign[1:] != sign[:-1]) + 1
        segs = np.split(np.arange(grid.size), edges)
        ext = np.array([s[np.argmax(np.abs(err[s]))] for s in segs])
        if ext.size != n:
            break
        nodes = grid[ext]
    return coef, np.abs(err).max()


if __name__ == "__main__":
    coef, e = fit()
    for i, c in enumerate(coef):
        print(f"a{i} = {c:.10e}    a{i} / pi = {c / np.pi:.10e}")
    x = np.linspace(0, 1, 100001)
    approx = np.sqrt(1 - x) * np.polyval(coef[::-1].astype(np.float32).astype(np.float64), x)
    print(f"max |P - f| = {e:.3e}; max |acos error| with float32 coefficients = {np.abs(approx - np.arccos(x)).max():.3e}")
