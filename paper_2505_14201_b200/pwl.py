"""Piece-wise linear tables for the accuracy study of Sec. IV-B.

The paper approximates the sigmoid (input range [-6, 11]) and the natural
logarithm on (0, 1) with 8 line segments each, fitted with a least-squares PWL
library, and does not print the coefficients.  This module refits them: a
continuous PWL function with free interior breakpoints, least squares on a dense
grid, breakpoints optimised from a fixed start (deterministic).  It holds none
of the attention arithmetic: the tables it returns are *inputs* of the CUDA
entry point and of the oracle's PWL variant, like the seeded tensors.
"""
import math

import numpy as np

SIGMOID_RANGE = (-6.0, 11.0)           # Sec. IV-B: the sigmoid argument is confined to this range


def sigmoid(x):
    x = np.asarray(x, dtype=np.float64)
    return np.where(x >= 0, 1.0 / (1.0 + np.exp(-np.abs(x))), np.exp(-np.abs(x)) / (1.0 + np.exp(-np.abs(x))))


def ln_range(lo=SIGMOID_RANGE[0]):
    """Domain of ln w: w is a sigmoid output of an argument >= lo, and at most 1."""
    return (float(sigmoid(lo)), 1.0)


def _hat_matrix(nodes, grid):
    """Columns = hat functions of the nodes evaluated on the grid (linear interpolation basis)."""
    A = np.zeros((grid.size, nodes.size))
    idx = np.clip(np.searchsorted(nodes, grid, side="right") - 1, 0, nodes.size - 2)
    t = (grid - nodes[idx]) / (nodes[idx + 1] - nodes[idx])
    A[np.arange(grid.size), idx] = 1.0 - t
    A[np.arange(grid.size), idx + 1] = t
    return A


def _fit_values(fn_vals, nodes, grid):
    A = _hat_matrix(nodes, grid)
    y, *_ = np.linalg.lstsq(A, fn_vals, rcond=None)
    r = A @ y - fn_vals
    return y, float(r @ r)


def fit_pwl(fn, lo, hi, n_seg=8, grid_points=4001, start="uniform"):
    """Continuous least-squares PWL fit of ``fn`` on [lo, hi] with ``n_seg`` segments.
    Returns (xs, ys) as float32 arrays of n_seg + 1 nodes."""
    from scipy.optimize import minimize
    grid = np.linspace(lo, hi, grid_points)
    vals = fn(grid)
    if start == "geometric":       # breakpoints crowd towards lo (for ln near 0)
        inner0 = lo + (hi - lo) * (np.geomspace(1.0, 2.0 ** n_seg, n_seg + 1)[1:-1] - 1.0) / (2.0 ** n_seg - 1.0)
    else:
        inner0 = np.linspace(lo, hi, n_seg + 1)[1:-1]

    def nodes_of(z):
        # unconstrained z -> strictly increasing interior breakpoints in (lo, hi)
        w = np.exp(z - z.max())
        c = np.cumsum(w) / (w.sum())
        return np.concatenate(([lo], lo + (hi - lo) * c[:-1], [hi]))

    gaps0 = np.diff(np.concatenate(([lo], inner0, [hi])))
    z0 = np.log(gaps0 / gaps0.sum())

    def cost(z):
        nodes = nodes_of(z)
        if np.min(np.diff(nodes)) < 1e-9 * (hi - lo):
            return 1e30
        return _fit_values(vals, nodes, grid)[1]

    res = minimize(cost, z0, method="Nelder-Mead", options={"maxiter": 4000, "xatol": 1e-6, "fatol": 1e-14})
    nodes = nodes_of(res.x)
    y, _ = _fit_values(vals, nodes, grid)
    return nodes.astype(np.float32), y.astype(np.float32)


def sampled_pwl(fn, lo, hi, n_seg):
    """Interpolating table: ``n_seg`` uniform segments through the exact function values."""
    xs = np.linspace(lo, hi, n_seg + 1)
    return xs.astype(np.float64), np.asarray(fn(xs), dtype=np.float64)


def paper_tables(n_seg=8, lo=SIGMOID_RANGE[0], hi=SIGMOID_RANGE[1]):
    """The two tables of Sec. IV-B: sigmoid on [lo, hi] and ln on [sigmoid(lo), 1]."""
    sig = fit_pwl(sigmoid, lo, hi, n_seg)
    wl, wh = ln_range(lo)
    ln = fit_pwl(np.log, wl, wh, n_seg, start="geometric")
    return sig, ln


def max_error(table, fn, lo, hi, points=20001):
    xs, ys = np.asarray(table[0], dtype=np.float64), np.asarray(table[1], dtype=np.float64)
    g = np.linspace(lo, hi, points)
    return float(np.max(np.abs(np.interp(g, xs, ys) - fn(g))))


if __name__ == "__main__":
    sig, ln = paper_tables()
    print("sigmoid nodes", sig[0], sig[1], "max err", max_error(sig, sigmoid, *SIGMOID_RANGE))
    print("ln nodes", ln[0], ln[1], "max err", max_error(ln, np.log, *ln_range()))
