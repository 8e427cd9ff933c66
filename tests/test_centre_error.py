"""Error against the generator's centres (Section 5.4): pins of the oracle's greedy pairing, and the
library's helper against it."""
import itertools

import numpy as np

from oracle.centre_error import centre_error
from paper_1505_04956_b200.metrics import generator_centre_error


def test_hand_cases_in_one_dimension():
    # closest pair (0, 1) first, then (10, 2): (1 + 8) / 2
    err, pairs = centre_error([[0.0], [10.0]], [[1.0], [2.0]])
    assert pairs == [(0, 0), (1, 1)] and abs(err - 4.5) < 1e-12
    # greedy is not the optimal assignment: (3, 2) = 1 goes first, leaving (0, 4) = 4 -> 2.5 (optimal would be 1.5)
    err, pairs = centre_error([[0.0], [3.0]], [[2.0], [4.0]])
    assert pairs == [(1, 0), (0, 1)] and abs(err - 2.5) < 1e-12
    # more prototypes than generator centres: the spare prototype stays unpaired
    err, pairs = centre_error([[0.0], [10.0]], [[9.0], [100.0], [0.5]])
    assert sorted(pairs) == [(0, 2), (1, 0)] and abs(err - 0.75) < 1e-12


def test_permuted_centres_give_zero_and_the_permutation():
    rng = np.random.default_rng(0)
    mu = rng.normal(size=(12, 5)) * 10
    perm = rng.permutation(12)
    err, pairs = centre_error(mu, mu[perm])
    assert err == 0.0
    assert all(perm[a] == c for c, a in pairs)


def test_first_pair_is_the_global_minimum_and_every_later_pair_is_minimal_among_the_free():
    rng = np.random.default_rng(1)
    mu, w = rng.normal(size=(6, 3)), rng.normal(size=(8, 3))
    err, pairs = centre_error(mu, w)
    dist = np.sqrt(((mu[:, None] - w[None]) ** 2).sum(2))
    free_c, free_w = set(range(6)), set(range(8))
    for c, a in pairs:
        best = min(dist[i, j] for i, j in itertools.product(free_c, free_w))
        assert dist[c, a] == best
        free_c.remove(c)
        free_w.remove(a)
    assert abs(err - np.mean([dist[c, a] for c, a in pairs])) < 1e-12


def test_library_helper_agrees_with_the_oracle():
    rng = np.random.default_rng(2)
    for C, k, d in ((10, 10, 10), (7, 12, 4), (20, 9, 3), (64, 64, 32)):
        mu = rng.normal(size=(C, d)) * 5
        w = mu[rng.permutation(C)[: min(C, k)]] + rng.normal(size=(min(C, k), d)) * 0.3
        if k > C:
            w = np.vstack([w, rng.normal(size=(k - C, d)) * 5])
        e1, p1 = centre_error(mu, w)
        e2, p2 = generator_centre_error(mu.astype(np.float32), w.astype(np.float32))
        assert sorted(p1) == sorted(p2)
        assert abs(e1 - e2) < 1e-5 * max(1.0, e1)
