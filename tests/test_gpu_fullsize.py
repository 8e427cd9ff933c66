"""The workloads at their full sizes, in the launch configuration bench.py times.

The oracle cannot run a full pass of every workload in seconds, so it replays the first rounds: the rows
those rounds touch are gathered (on the device, then copied) into a compact matrix in visiting order, on
which the oracle with batches in plain order draws exactly the same mini-batches, recipients and buffers.
The free-running pass of the stream workload is checked through E(w) (Eq. 8) and its counters.
"""
import numpy as np
import pytest
import torch

import paper_1505_04956_b200 as pkg
from paper_1505_04956_b200 import inputs
from oracle import asgd_oracle as orc
from tests.gpu_util import CENTRE_TOL, decided

pytestmark = pytest.mark.gpu

REPLAY_ROUNDS = {"tiny": 40, "stream": 9, "mid": 2, "sweep": 3, "dense": 1, "codebook": 1}     # stream: the first 1 % of a pass


def _setup(name, record_assign=1):
    wl = inputs.WORKLOADS[name]
    need = wl.N * wl.d * 4 * (1.6 if name in ("dense", "codebook") else 1.1) + (2 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free device memory for the full %s workload" % name)
    X, _ = inputs.make_samples(wl, device="cuda")
    w0 = inputs.initial_centres(wl, X)
    cfg = pkg.make_config(N=wl.N, d=wl.d, k=wl.k, W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval,
                          fanout=wl.fanout, seed=wl.seed, record_assign=record_assign)
    return wl, X, w0, pkg.Asgd(cfg, X, w0)


def _compact_rows(wl, X, rounds):
    """Rows of the first `rounds` mini-batches of every worker, worker-major, in visiting order."""
    idx = np.empty((wl.W, rounds, wl.b), np.int64)
    ar = np.arange(wl.b, dtype=np.int64)
    for i in range(wl.W):
        order = orc.batch_order(wl.seed, i, wl.B)
        for t in range(rounds):
            idx[i, t] = i * wl.H + int(order[t % wl.B]) * wl.b + ar
    rows = torch.from_numpy(idx.reshape(-1)).to(X.device)
    return X.index_select(0, rows).cpu().numpy()


@pytest.mark.parametrize("name", list(REPLAY_ROUNDS))
def test_first_rounds_at_full_size_match_the_oracle(name):
    rounds = REPLAY_ROUNDS[name]
    wl, X, w0, ctx = _setup(name)
    Xc = _compact_rows(wl, X, rounds)
    cpu = orc.Oracle(Xc, w0.cpu().numpy(), W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval, fanout=wl.fanout,
                     shuffle=0, seed=wl.seed, threads=orc.max_threads())
    assert cpu.H == rounds * wl.b
    # all rounds but the last on both sides; then the last round from the oracle's states, so that the rounding
    # differences of the earlier rounds cannot move a sample across a bisecting plane and the assignments of the
    # last round compare exactly (the receive buffers keep their own rounding: it only enters the centres)
    if rounds > 1:
        ctx.step(rounds - 1)
        ctx.sync()
        cpu.rounds(rounds - 1)
        worst = 0.0
        for i in range(wl.W):
            g = ctx.get_state(i).cpu().numpy().astype(np.float64)
            c = cpu.state(i).astype(np.float64)
            worst = max(worst, float(np.linalg.norm(g - c) / np.linalg.norm(c)))
        assert worst < CENTRE_TOL, (name, "before the last round", worst)
        for i in range(wl.W):
            ctx.set_state(i, torch.from_numpy(cpu.state(i)).to(X.device))
    ctx.step(1)
    ctx.sync()
    cpu.rounds(1)
    got_assign = ctx.get_assign().cpu().numpy()
    sample = np.unique(np.linspace(0, wl.W - 1, 64).astype(int))
    worst = 0.0
    for i in range(wl.W):
        g = ctx.get_state(i).cpu().numpy().astype(np.float64)
        c = cpu.state(i).astype(np.float64)
        worst = max(worst, float(np.linalg.norm(g - c) / np.linalg.norm(c)))
    assert worst < CENTRE_TOL, (name, worst)
    for i in sample:
        gs, cs = ctx.get_stats(int(i)), cpu.stats(int(i))
        for key in ("steps", "sent", "received", "overwritten"):
            assert gs[key] == cs[key], (name, i, key, gs, cs)
        tr = cpu.last_step(int(i))
        ok = decided(tr["d1"], tr["d2"])
        assert (got_assign[i][ok] == tr["assign"][ok]).all(), (name, i)
        assert ok.mean() > 0.99
    ctx.destroy()


def test_stream_workload_free_running_pass():
    wl, X, w0, ctx = _setup("stream", record_assign=0)
    steps = wl.B
    ctx.run(steps)
    ctx.sync()
    tot = {key: 0 for key in ("steps", "sent", "received", "accepted", "overwritten")}
    for i in range(wl.W):
        st = ctx.get_stats(i)
        for key in tot:
            tot[key] += st[key]
        assert st["steps"] == steps
    assert tot["sent"] == wl.W * wl.fanout * (steps // wl.comm_interval)
    assert tot["received"] + tot["overwritten"] <= tot["sent"]
    assert 0 < tot["accepted"] <= tot["received"]
    # final quantisation error against the oracle's synchronous schedule on the same data
    Xh = X.cpu().numpy()
    cpu = orc.Oracle(Xh, w0.cpu().numpy(), W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval, fanout=wl.fanout,
                     seed=wl.seed, threads=orc.max_threads())
    cpu.rounds(steps)
    prefix = Xh[: 1 << 24]
    E_gpu = orc.quantization_error(prefix, ctx.get_state(0).cpu().numpy(), threads=orc.max_threads())
    E_cpu = orc.quantization_error(prefix, cpu.state(0), threads=orc.max_threads())
    assert abs(E_gpu - E_cpu) <= 0.01 * E_cpu, (E_gpu, E_cpu)
    # the library's own evaluation over all rows agrees with the oracle's evaluator on the prefix scale
    E_all = ctx.eval(0)
    assert abs(E_all / wl.N - E_gpu / prefix.shape[0]) <= 0.01 * E_gpu / prefix.shape[0]
    ctx.destroy()
