"""ORACLE (test infrastructure, CPU only): error against simulated wall clock on a common time grid,
the picture behind the paper's error-runtime trade-off (Section 2.3's two metrics combined): at
grid time g the error of a replica is the error recorded at its last update completed by g; the
curve is the mean over the replicas that have completed at least one update by then."""
import numpy as np


def error_curve(t, err, grid):
    """t, err: [R, J] (clock and error at each update); grid: [G].  Returns (mean [G], count [G])."""
    t, err, grid = np.asarray(t, np.float64), np.asarray(err, np.float64), np.asarray(grid, np.float64)
    mean = np.zeros(grid.size)
    count = np.zeros(grid.size, np.int32)
    for i, g in enumerate(grid):
        total = 0.0
        for r in range(t.shape[0]):
            j = int(np.searchsorted(t[r], g, side="right")) - 1      # last update with t <= g
            if j >= 0:
                total += err[r, j]
                count[i] += 1
        mean[i] = total / count[i] if count[i] else 0.0
    return mean, count


def envelope(curves, counts):
    """Lower envelope of several error curves on one grid: curves, counts [n, G].  At each grid point the smallest
    value among the curves that have data there (count > 0) and the index of that curve (the lowest index on
    ties); where no curve has data the value is 0 and the index -1."""
    curves, counts = np.asarray(curves, np.float64), np.asarray(counts)
    n, G = curves.shape
    env, best = np.zeros(G), np.full(G, -1, np.int32)
    for g in range(G):
        for c in range(n):
            if counts[c, g] > 0 and (best[g] < 0 or curves[c, g] < env[g]):
                env[g], best[g] = curves[c, g], c
    return env, best
