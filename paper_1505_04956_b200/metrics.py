"""Evaluation helpers that are not on the timed path."""
import numpy as np


def generator_centre_error(generator_centres, centres):
    """Mean distance between generator centres and the found centres under a greedy pairing (Section 5.4).

    Pairing rule: repeatedly take the closest pair among the generator centres and found centres that
    are still free (ties: the lowest generator index, then the lowest centre index) until the smaller
    set is used up.  Returns (mean distance, list of (generator index, centre index)).
    """
    g = np.asarray(generator_centres, dtype=np.float64)
    c = np.asarray(centres, dtype=np.float64)
    g2 = (g * g).sum(1)[:, None]
    c2 = (c * c).sum(1)[None, :]
    d2 = np.maximum(g2 + c2 - 2.0 * (g @ c.T), 0.0)
    # exact distances for the pairs taken; the expanded form only ranks them
    n = min(g.shape[0], c.shape[0])
    free = d2.copy()
    pairs, total = [], 0.0
    for _ in range(n):
        flat = int(np.argmin(free))                      # first minimum in row-major order
        i, j = divmod(flat, c.shape[0])
        pairs.append((i, j))
        total += float(np.sqrt(((g[i] - c[j]) ** 2).sum()))
        free[i, :] = np.inf
        free[:, j] = np.inf
    return total / n, pairs
