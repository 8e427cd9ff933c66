"""TEST INFRASTRUCTURE -- not part of the product.

Error against the generator's centres (Section 5.4 of Keuper & Pfreundt, arXiv 1505.04956: for synthetic
data the result is judged by the distance of the found prototypes to the centres the data were drawn
around).  The paper does not say how prototypes are paired with generator centres; the reading taken
here is a greedy pairing: all (generator centre, prototype) pairs are sorted by Euclidean distance and
taken in that order, skipping pairs whose centre or prototype is already paired; the error is the mean
distance over the min(C, k) pairs.  Plain numpy, fp64; pinned in tests/test_centre_error.py.
"""
import numpy as np


def centre_error(generator_centres, prototypes):
    mu = np.asarray(generator_centres, dtype=np.float64)
    w = np.asarray(prototypes, dtype=np.float64)
    C, k = mu.shape[0], w.shape[0]
    dist = np.sqrt(((mu[:, None, :] - w[None, :, :]) ** 2).sum(axis=2))
    order = np.argsort(dist, axis=None, kind="stable")          # ties: lowest (centre, prototype) first
    used_c, used_w = np.zeros(C, bool), np.zeros(k, bool)
    pairs, total = [], 0.0
    for flat in order:
        c, a = divmod(int(flat), k)
        if used_c[c] or used_w[a]:
            continue
        used_c[c] = used_w[a] = True
        pairs.append((c, a))
        total += dist[c, a]
        if len(pairs) == min(C, k):
            break
    return total / len(pairs), pairs
