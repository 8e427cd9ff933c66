"""Per-centre messages (Section 4.4) on the GPU against the oracle: a put carries some centre rows,
lambda, delta and the merge are taken row by row."""
import os

import numpy as np
import pytest
import torch

from tests.gpu_util import Pair, scaled

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _row_decided(tr, s, a):
    lhs, rhs = tr["lhs"][s, a], tr["rhs"][s, a]
    return abs(lhs - rhs) >= 1e-5 * rhs


# (workload overrides, rows per message, rounds): one case per kernel, plus shapes with ragged row runs
CASES = {
    "generic_7x9": (dict(N=5 * 37 * 6 + 2, d=9, k=7, W=5, b=37, comm_interval=1, fanout=2), 3, 12),
    "generic_one_row_of_many": (dict(N=4 * 40 * 5, d=6, k=50, W=4, b=40, comm_interval=2, fanout=1), 1, 10),
    "stream_10x10": (dict(N=6 * 100 * 5, d=10, k=10, W=6, b=100, comm_interval=1, fanout=2), 4, 12),
    "stream_16x16_all_rows": (dict(N=4 * 175 * 4, d=16, k=16, W=4, b=175, comm_interval=2, fanout=1), 16, 8),
    "tiled_32x37": (dict(N=5 * 100 * 4 + 1, d=32, k=37, W=5, b=100, comm_interval=1, fanout=2), 5, 8),
    "tiled_128x100": (dict(N=3 * 100 * 3, d=128, k=100, W=3, b=100, comm_interval=1, fanout=1), 33, 6),
    "tc_d128_k100_one_block": (dict(N=3 * 200 * 3, d=128, k=100, W=3, b=200, comm_interval=1, fanout=1), 33, 6),
    "tc_d64_k300": (dict(N=3 * 200 * 4 + 5, d=64, k=300, W=3, b=200, comm_interval=1, fanout=2), 70, 6),
}


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("parzen", [1, 0])
def test_partial_rows_trajectory_matches_oracle(case, parzen):
    over, m, rounds = CASES[case]
    wl = scaled("tiny", **over)
    pr = Pair(wl, parzen=parzen, slots=2, partial_rows=m)
    seen_rows = 0
    for r in range(rounds):
        pr.rounds(1)
        pr.gpu.sync()
        assert pr.max_rel_l2() < pr.centre_tol(), (case, r, pr.max_rel_l2())
        for i in range(wl.W):
            tr = pr.cpu.last_step_rows(i)
            got = np.array(pr.gpu.get_accept_rows(i))
            msgs = pr.gpu.get_accept(i)
            whole = pr.cpu.last_step(i)["accept"]
            for s in range(pr.S):
                carried = tr["accept"][s] >= 0
                assert np.array_equal(got[s] >= 0, carried), (case, r, i, s)         # which rows the message carried
                seen_rows += int(carried.sum())
                undecided = 0
                for a in np.nonzero(carried)[0]:
                    if parzen == 0 or _row_decided(tr, s, a):
                        assert got[s, a] == tr["accept"][s, a], (case, r, i, s, a)
                    else:
                        undecided += 1
                if whole[s] < 0:
                    assert msgs[s] == -1
                else:
                    assert abs(msgs[s] - whole[s]) <= undecided                        # accepted rows of the message
    for i in range(wl.W):
        g, c = pr.gpu.get_stats(i), pr.cpu.stats(i)
        for key in ("steps", "sent", "received", "overwritten"):
            assert g[key] == c[key], (case, i, key)
    assert seen_rows > 0
    pr.close()


def test_partial_rows_hand_cases_on_gpu():
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
        wl = scaled("tiny", N=8, d=1, k=2, W=2, b=4, eps=eps, comm_interval=0, fanout=1)
        pr = Pair(wl, parzen=parzen, X=X, w0=np.array([[w0], [w1]], np.float32), oracle=False, shuffle=0, partial_rows=1)
        first, n = (0, 2) if has == [1, 1] else ((0, 1) if has == [1, 0] else (1, 1))
        pr.gpu.put_rows(0, 0, torch.tensor([[v0], [v1]], dtype=torch.float32, device="cuda"), first, n)
        pr.gpu.step(1)
        pr.gpu.sync()
        rows = pr.gpu.get_accept_rows(0)[0]
        assert rows == [a0 if has[0] else -1, a1 if has[1] else -1], line
        assert pr.gpu.get_accept(0) == [a0 + a1], line
        assert np.allclose(pr.gpu.get_state(0).cpu().numpy()[:, 0], want, atol=2e-6), line
        plain = [w0 - eps * (w0 - x0) / 2, w1 - eps * (w1 - x1) / 2]
        assert np.allclose(pr.gpu.get_state(1).cpu().numpy()[:, 0], plain, atol=2e-6), line
        st = pr.gpu.get_stats(0)
        assert st["received"] == 1 and st["accepted"] == int(a0 + a1 > 0), line
        pr.close()


def test_partial_rows_free_running_stays_close_to_the_oracle():
    # races are part of the free-running mode: compare the quantisation error only
    wl = scaled("stream", N=37 * 500 * 9 + 13, W=37, comm_interval=2)
    pr = Pair(wl, partial_rows=3)
    steps = 2 * pr.cpu.B
    pr.gpu.run(steps)
    pr.gpu.sync()
    pr.cpu.rounds(steps)
    from oracle import asgd_oracle as orc
    Eg = orc.quantization_error(pr.Xh, pr.gpu.get_state(0).cpu().numpy())
    Ec = orc.quantization_error(pr.Xh, pr.cpu.state(0))
    assert abs(Eg - Ec) <= 0.01 * Ec, (Eg, Ec)
    assert sum(pr.gpu.get_stats(i)["received"] for i in range(wl.W)) > 0
    pr.close()


def test_partial_rows_argument_checks():
    wl = scaled("tiny", N=400, d=3, k=4, W=2, b=10, comm_interval=1, fanout=1)
    pr = Pair(wl, oracle=False)                            # whole-state messages
    v = torch.zeros((4, 3), device="cuda")
    with pytest.raises(Exception):
        pr.gpu.put_rows(0, 0, v, 0, 2)                     # only valid in per-centre mode
    with pytest.raises(Exception):
        pr.gpu.get_accept_rows(0)
    pr.close()
    pr = Pair(wl, oracle=False, partial_rows=2)
    for first, n in ((-1, 1), (4, 1), (0, 0), (0, 5)):
        with pytest.raises(Exception):
            pr.gpu.put_rows(0, 0, v, first, n)
    pr.close()
    import paper_1505_04956_b200 as pkg
    with pytest.raises(Exception):
        cfg = pkg.make_config(N=400, d=3, k=4, W=2, b=10, eps=0.1, comm_interval=1, fanout=1, partial_rows=5)
        pkg.Asgd(cfg, torch.zeros((400, 3), device="cuda"), torch.zeros((4, 3), device="cuda"))
