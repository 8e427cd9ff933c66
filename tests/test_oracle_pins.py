"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's code.

Every test names the passage of the paper it takes its expectation from.
"""
import os

import numpy as np
import pytest
from scipy.cluster.vq import vq

from oracle import asgd_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1
GOLDEN_GAMMA = 0x9E3779B97F4A7C15


# ----------------------------------------------------------------------------------------------
# schedule random numbers
# ----------------------------------------------------------------------------------------------
def test_splitmix64_published_vectors():
    for line in open(os.path.join(GOLD, "splitmix64_vectors.txt")):
        if line.startswith("#") or not line.strip():
            continue
        seed, idx, out = (int(x, 0) for x in line.split())
        assert orc.sm64((seed + idx * GOLDEN_GAMMA) & M64) == out


def test_draw_is_chain_of_generator_outputs():
    # h(seed, tag, a, b, c) is defined as a chain of SplitMix64 first outputs
    seed, tag, a, b, c = 42, 2, 5, 77, 1
    h = orc.sm64(seed ^ tag)
    for x in (a, b, c):
        h = orc.sm64((h + x) & M64)
    assert orc.draw(seed, tag, a, b, c) == h


def _lattice_problem(k=4, d=3, per=25, W=1, spread=0.05, seed=0, gap=10.0):
    """Well separated clusters: the label of every row is known by construction."""
    rng = np.random.default_rng(seed)
    centres = (rng.permutation(k)[:, None] * gap + np.arange(d)[None, :]).astype(np.float32)
    labels = rng.integers(0, k, size=per * k * W)
    X = centres[labels] + rng.uniform(-spread, spread, size=(labels.size, d)).astype(np.float32)
    return X.astype(np.float32), labels.astype(np.int32), centres


def test_permutation_and_recipients():
    X, _, c = _lattice_problem(W=16, per=32)
    o = orc.Oracle(X, c, W=16, b=4, eps=0.1, comm_interval=1, fanout=3, slots=2, seed=9)
    for i in range(16):
        p = o.perm(i)
        assert sorted(p.tolist()) == list(range(o.B))
    assert any((o.perm(i) != np.arange(o.B)).any() for i in range(16))
    hist = np.zeros(16)
    for i in range(16):
        for t in range(200):
            peers, slots = o.recipients(i, t)
            assert i not in peers and len(set(peers.tolist())) == 3
            assert ((0 <= peers) & (peers < 16)).all() and ((0 <= slots) & (slots < 2)).all()
            hist[peers[0]] += 1
    # first recipient is uniform over the other 15 workers: chi-square smoke test (very loose)
    exp = hist.sum() / 16
    assert ((hist - exp) ** 2 / exp).sum() < 60.0
    o2 = orc.Oracle(X, c, W=16, b=4, eps=0.1, shuffle=0, seed=9)
    assert (o2.perm(3) == np.arange(o2.B)).all()


# ----------------------------------------------------------------------------------------------
# assignment and E(w)   (Eq. 8)
# ----------------------------------------------------------------------------------------------
def test_assignment_known_by_construction_and_label_permutation():
    X, labels, c = _lattice_problem(k=5, d=3, per=12)
    a, d1, d2 = orc.assign(X, c)
    assert (a == labels).all()
    perm = np.array([3, 0, 4, 1, 2])
    a2, _, _ = orc.assign(X, c[perm])
    assert (perm[a2] == labels).all()
    assert (d1 <= d2).all() and (d1 >= 0).all()


def test_assignment_exact_ties_go_to_lowest_index():
    w = np.array([[0.0, 0.0], [2.0, 0.0], [0.0, 2.0], [2.0, 2.0]], np.float32)
    X = np.array([[1.0, 0.0], [1.0, 1.0], [2.0, 1.0], [0.0, 1.0], [1.0, 2.0]], np.float32)
    a, d1, d2 = orc.assign(X, w)
    assert a.tolist() == [0, 0, 1, 0, 2]
    assert np.allclose(d1, d2)
    # duplicate prototypes: the first one wins
    a, _, _ = orc.assign(X, np.vstack([w[3:], w[3:], w]))
    assert (a != 1).all()


def test_assignment_and_error_against_scipy_vq():
    rng = np.random.default_rng(3)
    X = rng.normal(size=(64, 3)).astype(np.float32)
    w = rng.normal(size=(5, 3)).astype(np.float32)
    code, dist = vq(X.astype(np.float64), w.astype(np.float64))
    a, d1, _ = orc.assign(X, w)
    assert (a == code).all()
    assert np.allclose(np.sqrt(d1), dist, rtol=1e-12, atol=0)
    E = orc.quantization_error(X, w)
    assert abs(E - 0.5 * (dist ** 2).sum()) <= 1e-12 * E


def test_error_expanded_form_and_sanity_range():
    # E computed through ||x||^2 - 2 x.w + ||w||^2 in fp64 agrees with the oracle's direct form
    rng = np.random.default_rng(4)
    k, d, n, sigma = 10, 10, 20000, 1.0
    mu = rng.uniform(-10, 10, size=(k, d))
    lab = rng.integers(0, k, n)
    X = (mu[lab] + sigma * rng.normal(size=(n, d))).astype(np.float32)
    w = mu.astype(np.float32)
    Xd, wd = X.astype(np.float64), w.astype(np.float64)
    sc = (Xd ** 2).sum(1)[:, None] - 2 * Xd @ wd.T + (wd ** 2).sum(1)[None, :]
    E = orc.quantization_error(X, w)
    assert abs(E - 0.5 * sc.min(1).sum()) <= 1e-10 * E
    # at the generator's centres of a well separated isotropic mixture E/N is about d*sigma^2/2
    assert 0.9 * 0.5 * d < E / n < 1.1 * 0.5 * d
    assert abs(orc.quantization_error(X, w, threads=2) - E) <= 1e-12 * E


# ----------------------------------------------------------------------------------------------
# mini-batch step   (Eq. 9, Algorithm 4)
# ----------------------------------------------------------------------------------------------
def test_step_closed_form_counts_and_sums():
    # labels known by construction => n_k and mean_k known without any distance computation
    k, d, b, eps = 4, 3, 40, 0.25
    X, labels, c = _lattice_problem(k=k, d=d, per=b // k)
    w0 = (c + 0.3).astype(np.float32)
    w0[3] = c[3] + 100.0          # pushed far away: it attracts nothing, so n_3 = 0
    o = orc.Oracle(X[:b], w0, W=1, b=b, eps=eps, shuffle=0)
    o.rounds(1)
    tr = o.last_step(0)
    lab = labels[:b].copy()
    # rows of cluster 3 now fall to the nearest remaining centre; recompute only those by hand
    near3 = int(np.argmin([np.sum((c[3].astype(np.float64) - w0[j].astype(np.float64)) ** 2) for j in range(k)]))
    lab[lab == 3] = near3
    n = np.bincount(lab, minlength=k)
    assert tr["counts"].tolist() == n.tolist() and n.sum() == b
    assert (tr["assign"] == lab).all()
    w1 = o.state(0).astype(np.float64)
    for j in range(k):
        if n[j] == 0:
            assert (w1[j] == w0[j]).all()              # a centre with no samples does not move
        else:
            mean = X[:b][lab == j].astype(np.float64).mean(0)
            f = eps * n[j] / b
            assert np.allclose(w1[j], (1 - f) * w0[j] + f * mean, rtol=2e-7, atol=1e-6)
    # conservation: sum_k S_k = sum of the batch, seen through the update
    lhs = ((w1 - w0.astype(np.float64)) * b / eps + n[:, None] * w0).sum(0)
    assert np.allclose(lhs, X[:b].astype(np.float64).sum(0), rtol=1e-5, atol=1e-3)


def test_single_centre_is_exponential_moving_average():
    # k = 1 on constant data x0: w_t = x0 + (1-eps)^t (w_0 - x0)
    x0 = np.array([1.5, -2.0, 0.25], np.float32)
    X = np.tile(x0, (64, 1))
    w0 = np.array([[4.0, 4.0, 4.0]], np.float32)
    eps, T = 0.125, 9
    o = orc.Oracle(X, w0, W=1, b=8, eps=eps)
    o.rounds(T)
    want = x0 + (1 - eps) ** T * (w0[0].astype(np.float64) - x0)
    assert np.allclose(o.state(0)[0], want, rtol=1e-6)
    # k = 1, general data: w' = (1-eps) w + eps * mean(M)
    rng = np.random.default_rng(0)
    X = rng.normal(size=(32, 3)).astype(np.float32)
    o = orc.Oracle(X, w0, W=1, b=32, eps=eps, shuffle=0)
    o.rounds(1)
    assert np.allclose(o.state(0)[0], (1 - eps) * w0[0] + eps * X.astype(np.float64).mean(0), rtol=1e-6, atol=1e-7)


def test_full_step_to_the_mean_is_one_lloyd_step():
    # eps = 1 and the whole mini-batch in one cluster => that centre lands on the batch mean
    rng = np.random.default_rng(1)
    X = (rng.normal(size=(16, 2)) * 0.1 + np.array([5.0, 5.0])).astype(np.float32)
    w0 = np.array([[4.0, 4.5], [-50.0, -50.0]], np.float32)
    o = orc.Oracle(X, w0, W=1, b=16, eps=1.0, shuffle=0)
    o.rounds(1)
    w1 = o.state(0)
    assert np.allclose(w1[0], X.astype(np.float64).mean(0), rtol=1e-6)
    assert (w1[1] == w0[1]).all()


def _sequential_minibatch_sgd(X, w0, b, eps, order, steps):
    """Algorithm 4 for K-Means written on its own: plain Python, fp64, state stored as fp32."""
    w = w0.astype(np.float32).copy()
    k, d = w.shape
    for t in range(steps):
        rows = X[order[t % len(order)] * b:(order[t % len(order)] + 1) * b]
        grad = np.zeros((k, d))
        for x in rows:
            best, bd = 0, float("inf")
            for j in range(k):
                dist = 0.0
                for q in range(d):
                    dist += (float(x[q]) - float(w[j, q])) ** 2
                if dist < bd:
                    best, bd = j, dist
            for q in range(d):
                grad[best, q] += float(w[best, q]) - float(x[q])
        # the oracle forms (n w - S)/b; here the gradient is summed sample by sample, so compare
        # to within fp64 rounding of that reordering, after the fp32 store
        w = (w.astype(np.float64) - eps * grad / b).astype(np.float32)
    return w


@pytest.mark.parametrize("mode", ["W1", "silent", "fanout0"])
def test_no_communication_reduces_to_sequential_minibatch_sgd(mode):
    # Section 4: with the communication interval at infinity ASGD is SimuParallelSGD, i.e. every
    # worker runs Algorithm 4 on its own shard
    rng = np.random.default_rng(5)
    k, d, b, eps, T = 3, 2, 8, np.float32(0.2), 7
    mu = np.array([[0, 0], [4, 0], [0, 4]], np.float64)
    W = 1 if mode == "W1" else 3
    n = 40 * W
    X = (mu[rng.integers(0, k, n)] + rng.normal(size=(n, d))).astype(np.float32)
    w0 = X[:k].copy()
    kw = dict(W=W, b=b, eps=float(eps), seed=11)
    if mode == "silent":
        kw.update(comm_interval=0, fanout=1)
    elif mode == "fanout0":
        kw.update(comm_interval=1, fanout=0)
    else:
        kw.update(comm_interval=1, fanout=0)
    o = orc.Oracle(X, w0, **kw)
    o.rounds(T)
    for i in range(W):
        shard = X[i * o.H:(i + 1) * o.H]
        want = _sequential_minibatch_sgd(shard, w0, b, float(eps), o.perm(i), T)
        got = o.state(i)
        assert np.allclose(got, want, rtol=0, atol=2e-7 * np.abs(want).max())
        assert o.stats(i)["received"] == 0 and o.stats(i)["sent"] == 0


# ----------------------------------------------------------------------------------------------
# external states   (Eq. 2-7, Fig. 4)
# ----------------------------------------------------------------------------------------------
def test_parzen_1d_hand_cases():
    for line in open(os.path.join(GOLD, "parzen_1d_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w, x, eps, v, parzen, delta, w_new = (float(s) for s in line.split())
        X = np.full((8, 1), x, np.float32)
        o = orc.Oracle(X, np.array([[w]], np.float32), W=2, b=4, eps=eps, comm_interval=0, fanout=1,
                       parzen=int(parzen))
        o.put(0, 0, np.array([[v]], np.float32))
        o.rounds(1)
        tr = o.last_step(0)
        assert tr["accept"][0] == int(delta), line
        assert abs(float(o.state(0)[0, 0]) - w_new) < 1e-6, line
        # the other worker got nothing: plain local step (Eq. 3 with every buffer empty)
        assert abs(float(o.state(1)[0, 0]) - (w - eps * (w - x))) < 1e-6
        st = o.stats(0)
        assert st["received"] == 1 and st["accepted"] == int(delta)


def _known_gradient_problem(seed=0, k=3, d=4, b=30):
    X, labels, c = _lattice_problem(k=k, d=d, per=b // k, seed=seed)
    rng = np.random.default_rng(seed + 100)
    w = (c + rng.uniform(-0.4, 0.4, size=c.shape)).astype(np.float32)
    n = np.bincount(labels[:b], minlength=k).astype(np.float64)
    S = np.zeros((k, d))
    for r in range(b):
        S[labels[r]] += X[r].astype(np.float64)
    D = (n[:, None] * w.astype(np.float64) - S) / b          # Eq. 9, true-gradient sign
    return X[:b], w, D


def test_parzen_delta_equivalent_inner_product_form_and_special_states():
    # Eq. 4  <=>  2 <D, w - v> > eps ||D||^2   (expand the left square)
    eps = 0.3
    rng = np.random.default_rng(7)
    agree = 0
    for trial in range(40):
        X, w, D = _known_gradient_problem(seed=trial)
        v = (w + rng.normal(size=w.shape) * eps * np.abs(D).max()).astype(np.float32)
        Xd = np.vstack([X, X])
        o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1)
        o.put(0, 0, v)
        o.rounds(1)
        tr = o.last_step(0)
        wd, vd = w.astype(np.float64), v.astype(np.float64)
        e = float(np.float32(eps))
        margin = 2 * (D * (wd - vd)).sum() - e * (D ** 2).sum()
        if abs(margin) > 1e-9:
            assert tr["accept"][0] == int(margin > 0)
            agree += 1
        assert np.isclose(tr["rhs"][0], ((wd - vd) ** 2).sum(), rtol=1e-12)
        assert np.isclose(tr["lhs"][0], ((wd - e * D - vd) ** 2).sum(), rtol=1e-9)
    assert agree >= 35
    # special external states
    X, w, D = _known_gradient_problem(seed=99)
    Xd = np.vstack([X, X])
    e = float(np.float32(eps))
    for v, want in ((w, 0), ((w - e * D).astype(np.float32), 1), ((w + e * D).astype(np.float32), 0)):
        o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1)
        o.put(0, 0, v)
        o.rounds(1)
        assert o.last_step(0)["accept"][0] == want


def test_merge_of_several_buffers_eq6():
    # S = 3 buffers: one accepted, one rejected, one empty.  Eq. 6 by hand in numpy.
    eps = 0.2
    X, w, D = _known_gradient_problem(seed=3)
    e = float(np.float32(eps))
    wd = w.astype(np.float64)
    good = (wd - 2 * e * D).astype(np.float32)        # beyond the projected step, same direction
    bad = (wd + 3 * e * D).astype(np.float32)         # behind
    Xd = np.vstack([X, X])
    o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1, slots=3)
    o.put(0, 0, bad)
    o.put(0, 2, good)
    o.rounds(1)
    tr = o.last_step(0)
    assert tr["accept"].tolist() == [0, -1, 1]
    want = wd - e * (wd - (wd + good.astype(np.float64)) / 2 + D)
    assert np.allclose(o.state(0), want, rtol=1e-6, atol=1e-6)
    # window off (Eq. 3): both received states enter the mean, the empty buffer does not
    o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1, slots=3, parzen=0)
    o.put(0, 0, bad)
    o.put(0, 2, good)
    o.rounds(1)
    want = wd - e * (wd - (wd + good.astype(np.float64) + bad.astype(np.float64)) / 3 + D)
    assert np.allclose(o.state(0), want, rtol=1e-6, atol=1e-6)
    # an all-zero buffer counts as empty (lambda of Eq. 3) even with the window off
    o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1, slots=3, parzen=0)
    o.put(0, 1, np.zeros_like(w))
    o.rounds(1)
    assert np.allclose(o.state(0), wd - e * D, rtol=1e-6, atol=1e-6)
    assert o.stats(0)["received"] == 1 and o.stats(0)["accepted"] == 0
    # a message is used once: the next step is a plain local step again
    assert o.last_step(0)["accept"].tolist() == [-1, 0, -1]
    o.rounds(1)
    assert o.last_step(0)["accept"].tolist() == [-1, -1, -1]


def test_delivery_is_atomic_last_sender_wins_and_counters_balance():
    rng = np.random.default_rng(8)
    k, d, W, b, T = 3, 2, 6, 5, 12
    mu = np.array([[0, 0], [6, 0], [0, 6]], np.float64)
    n = W * 40
    X = (mu[rng.integers(0, k, n)] + rng.normal(size=(n, d))).astype(np.float32)
    o = orc.Oracle(X, X[:k].copy(), W=W, b=b, eps=0.1, comm_interval=2, fanout=2, slots=2, seed=5)
    for t in range(T):
        o.rounds(1)
        if (t + 1) % 2 == 0:
            states = o.states()
            last = {}
            for i in range(W):
                peers, slots = o.recipients(i, t)
                for p, s in zip(peers, slots):
                    last[(int(p), int(s))] = i          # ascending sender order: later overwrites
            for (p, s), i in last.items():
                payload, seq, seen = o.mail(p, s)
                assert (payload == states[i]).all()
                assert seq > seen
    tot = {key: sum(o.stats(i)[key] for i in range(W)) for key in ("sent", "received", "accepted", "overwritten")}
    pending = 0
    for i in range(W):
        for s in range(2):
            _, seq, seen = o.mail(i, s)
            pending += seq - seen
    assert tot["sent"] == W * 2 * (T // 2)
    assert tot["received"] + tot["overwritten"] + pending == tot["sent"]
    assert tot["accepted"] <= tot["received"]
    assert all(o.stats(i)["steps"] == T for i in range(W))


def test_communication_pulls_workers_together():
    # Eq. 3 with the window off and eps = 1 on zero-gradient data averages states, so the spread
    # of the workers' states can only shrink; with communication off it stays what it was.
    k, d, W = 1, 2, 4
    w0 = np.zeros((k, d), np.float32)

    def spread(o):
        s = o.states().astype(np.float64)
        return float(((s - s.mean(0)) ** 2).sum())
    for c, shrink in ((1, True), (0, False)):
        # data placed at each worker's own state: the local gradient vanishes, only the merge acts
        Xi = np.repeat(np.arange(1, W + 1, dtype=np.float32), 8)[:, None] * np.ones((1, d), np.float32)
        o = orc.Oracle(Xi, w0, W=W, b=4, eps=1.0, comm_interval=c, fanout=1, parzen=0, seed=2)
        for i in range(W):
            o.set_state(i, np.full((k, d), float(i + 1), np.float32))
        s0 = spread(o)
        o.rounds(1)
        assert spread(o) == pytest.approx(s0)           # first round: nothing received yet
        o.rounds(1)
        if shrink:
            assert spread(o) < s0
        else:
            assert spread(o) == pytest.approx(s0)


@pytest.mark.parametrize("partial_rows", [0, 2])
def test_round_loop_on_several_threads_is_bit_identical_to_one_thread(partial_rows):
    # Algorithm 5: within a round a worker touches only its own state and its own receive buffers (the puts are
    # delivered after the round), so running the workers of a round on n threads must change nothing at all:
    # states, traces of the last step, counters and buffer contents, with communication switched on.
    rng = np.random.default_rng(11)
    W, k, d, b = 12, 5, 4, 16
    mu = rng.uniform(-4, 4, size=(k, d))
    X = (mu[rng.integers(0, k, W * b * 6 + 3)] + rng.normal(size=(W * b * 6 + 3, d))).astype(np.float32)
    w0 = X[rng.choice(X.shape[0], k, replace=False)].copy()
    kw = dict(W=W, b=b, eps=0.2, comm_interval=1, fanout=2, slots=2, seed=5, partial_rows=partial_rows)
    one = orc.Oracle(X, w0, threads=1, **kw)
    many = orc.Oracle(X, w0, threads=min(4, orc.max_threads()), **kw)
    if many.threads < 2:
        pytest.skip("the oracle was built without a parallel round loop")
    for T in (1, 7, 13):
        one.rounds(T)
        many.rounds(T)
        assert np.array_equal(one.states(), many.states())
        for i in range(W):
            assert one.stats(i) == many.stats(i)
            a, m = one.last_step(i), many.last_step(i)
            for key in a:
                assert np.array_equal(a[key], m[key]), (T, i, key)
            for s in range(2):
                va, m_seq, m_seen = one.mail(i, s)
                vb, n_seq, n_seen = many.mail(i, s)
                assert np.array_equal(va, vb) and (m_seq, m_seen) == (n_seq, n_seen)
    assert sum(one.stats(i)["accepted"] for i in range(W)) > 0        # messages did flow and were merged


# ---------------------------------------------------------------------------------------------
# Per-centre messages (Section 4.4): a put carries some of the centre rows; lambda, delta and the
# merge are taken row by row.
# ---------------------------------------------------------------------------------------------
def test_partial_rows_1d_hand_cases():
    for line in open(os.path.join(GOLD, "partial_rows_1d_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = [float(s) for s in line.split()]
        w0, w1, x0, x1, eps, v0, v1 = f[:7]
        has = [int(f[7]), int(f[8])]
        parzen, a0, a1 = int(f[9]), int(f[10]), int(f[11])
        want = f[12:14]
        batch = np.array([[x0], [x1], [x0], [x1]], np.float32)
        X = np.vstack([batch, batch])
        o = orc.Oracle(X, np.array([[w0], [w1]], np.float32), W=2, b=4, eps=eps, comm_interval=0, fanout=1,
                       parzen=parzen, shuffle=0, partial_rows=1)
        o.put_rows(0, 0, np.array([[v0], [v1]], np.float32), has)
        o.rounds(1)
        tr = o.last_step_rows(0)
        got = [int(tr["accept"][0, r]) if has[r] else 0 for r in range(2)]
        assert got == [a0, a1], line
        for r in range(2):
            if not has[r]:
                assert tr["accept"][0, r] == -1, line          # the row was not in the message
        assert np.allclose(o.state(0)[:, 0], want, atol=1e-6), line
        # the worker that got nothing takes the plain local step on both rows
        plain = [w0 - eps * (w0 - x0) / 2, w1 - eps * (w1 - x1) / 2]
        assert np.allclose(o.state(1)[:, 0], plain, atol=1e-6), line
        st = o.stats(0)
        assert st["received"] == 1 and st["accepted"] == int(a0 + a1 > 0), line
        assert o.last_step(0)["accept"][0] == a0 + a1, line      # accepted rows of the message


def test_partial_rows_single_centre_equals_whole_state_messages():
    # with k = 1 a row is the whole state: both modes must give the same trajectory bit for bit
    rng = np.random.default_rng(3)
    X = (rng.normal(size=(6000, 3)) + np.array([4.0, -2.0, 1.0])).astype(np.float32)
    w0 = np.array([[0.5, 0.5, 0.5]], np.float32)
    kw = dict(W=6, b=40, eps=0.2, comm_interval=2, fanout=2, slots=2, seed=11)
    a = orc.Oracle(X, w0, **kw)
    c = orc.Oracle(X, w0, partial_rows=1, **kw)
    a.rounds(25)
    c.rounds(25)
    assert np.array_equal(a.states(), c.states())
    sa, sc = [a.stats(i) for i in range(6)], [c.stats(i) for i in range(6)]
    assert sa == sc and sum(s["accepted"] for s in sa) > 0


def test_partial_rows_rows_outside_the_message_take_the_plain_step():
    # closed form per row: a row the message does not carry moves exactly as with no communication,
    # a carried row follows Eq. 6 with its own delta (checked in the inner-product form of Eq. 4)
    eps = 0.3
    rng = np.random.default_rng(21)
    seen_accept = seen_reject = 0
    for trial in range(30):
        X, w, D = _known_gradient_problem(seed=trial, k=3, d=4, b=30)
        v = (w + rng.normal(size=w.shape) * eps * np.abs(D).max()).astype(np.float32)
        has = np.zeros(3, np.uint8)
        has[rng.choice(3, size=int(rng.integers(1, 3)), replace=False)] = 1
        Xd = np.vstack([X, X])
        o = orc.Oracle(Xd, w, W=2, b=X.shape[0], eps=eps, shuffle=0, comm_interval=0, fanout=1, partial_rows=2)
        o.put_rows(0, 0, v, has)
        o.rounds(1)
        tr = o.last_step_rows(0)
        wd, vd = w.astype(np.float64), v.astype(np.float64)
        e = float(np.float32(eps))
        got = o.state(0).astype(np.float64)
        for r in range(3):
            plain = wd[r] - e * D[r]
            if not has[r]:
                assert tr["accept"][0, r] == -1
                assert np.allclose(got[r], plain, rtol=0, atol=1e-6)
                continue
            margin = 2 * (D[r] * (wd[r] - vd[r])).sum() - e * (D[r] ** 2).sum()
            if abs(margin) < 1e-9:
                continue
            acc = int(margin > 0)
            assert tr["accept"][0, r] == acc
            merged = wd[r] - e * (acc * (wd[r] - (wd[r] + vd[r]) / 2) + D[r])
            assert np.allclose(got[r], merged, rtol=0, atol=1e-6)
            seen_accept += acc
            seen_reject += 1 - acc
    assert seen_accept >= 5 and seen_reject >= 5


def test_partial_rows_schedule_and_delivery():
    k, d, W, m = 7, 2, 5, 3
    rng = np.random.default_rng(5)
    X = rng.normal(size=(5 * 40, d)).astype(np.float32)
    w0 = X[:k].copy()
    o = orc.Oracle(X, w0, W=W, b=8, eps=0.1, comm_interval=1, fanout=2, slots=3, seed=77, partial_rows=m)
    firsts = []
    for t in range(300):
        for i in range(W):
            for j in range(2):
                fl = o.put_row_flags(i, t, j)
                assert fl.sum() == m
                r0 = [r for r in range(k) if fl[r] and not fl[(r - 1) % k]]
                assert len(r0) == 1                       # one cyclic run of m consecutive rows
                assert all(fl[(r0[0] + q) % k] for q in range(m))
                firsts.append(r0[0])
    cnt = np.bincount(firsts, minlength=k)
    expect = len(firsts) / k
    assert ((cnt - expect) ** 2 / expect).sum() < 30.0     # chi-square, 6 degrees of freedom (p ~ 1e-5 at 30)
    # delivery: after one round a buffer holds the carried rows of the LAST sender's new state, flags of that message
    o.rounds(1)
    writers = {}
    for i in range(W):
        peers, slots = o.recipients(i, 0)
        for j in range(2):
            writers[(int(peers[j]), int(slots[j]))] = (i, j)        # ascending sender order: the last one stays
    assert writers
    for (r, s), (i, j) in writers.items():
        payload, seq, seen = o.mail(r, s)
        fl = o.put_row_flags(i, 0, j)
        assert np.array_equal(o.mail_rows(r, s), fl)
        assert np.array_equal(payload[fl == 1], o.state(i)[fl == 1])
        assert seq >= 1 and seen == 0
