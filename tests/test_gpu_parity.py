"""CUDA library against the CPU oracle, element by element, on the same seeded inputs (C ABI calls)."""
import os

import numpy as np
import pytest
import torch

import paper_1505_04956_b200 as pkg
from oracle import asgd_oracle as orc
from tests.gpu_util import CENTRE_TOL, PARITY_WORKLOADS, Pair, decided, scaled

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _compare_stats(pr, exact_accept=True):
    for i in range(pr.wl.W):
        g, c = pr.gpu.get_stats(i), pr.cpu.stats(i)
        for key in ("steps", "sent", "received", "overwritten"):
            assert g[key] == c[key], (i, key, g, c)
        if exact_accept:
            assert g["accepted"] == c["accepted"], (i, g, c)


def _accept_decided(tr, s, eps_rel=1e-5):
    """True when the oracle's Eq. 4 comparison is decided beyond the relative gap."""
    return abs(tr["lhs"][s] - tr["rhs"][s]) >= eps_rel * tr["rhs"][s]


@pytest.mark.parametrize("name", list(PARITY_WORKLOADS))
def test_trajectory_matches_oracle(name):
    wl, rounds = PARITY_WORKLOADS[name]
    pr = Pair(wl)
    step = max(1, rounds // 8)
    done = 0
    undecided_accepts = 0
    while done < rounds:
        n = min(step, rounds - done)
        pr.rounds(n)
        done += n
        pr.gpu.sync()
        assert pr.max_rel_l2() < pr.centre_tol(), (name, done, pr.max_rel_l2())
        for i in range(wl.W):
            tr = pr.cpu.last_step(i)
            acc = pr.gpu.get_accept(i)
            for s in range(pr.S):
                if tr["accept"][s] < 0:
                    assert acc[s] == -1
                elif _accept_decided(tr, s):
                    assert acc[s] == tr["accept"][s], (name, done, i, s, tr["lhs"][s], tr["rhs"][s])
                else:
                    undecided_accepts += 1
    _compare_stats(pr, exact_accept=False)
    tot_g = sum(pr.gpu.get_stats(i)["accepted"] for i in range(wl.W))
    tot_c = sum(pr.cpu.stats(i)["accepted"] for i in range(wl.W))
    tot_r = sum(pr.cpu.stats(i)["received"] for i in range(wl.W))
    assert abs(tot_g - tot_c) <= max(2, 0.01 * tot_r), (tot_g, tot_c, tot_r)
    if wl.comm_interval > 0 and wl.fanout > 0:
        assert tot_r > 0
    pr.close()


@pytest.mark.parametrize("name", list(PARITY_WORKLOADS))
def test_single_step_assignments_bit_exact(name):
    wl, rounds = PARITY_WORKLOADS[name]
    pr = Pair(wl)
    warm = min(rounds, 5)
    pr.cpu.rounds(warm)
    pr.gpu.step(warm)
    # restart the GPU from the oracle's states so that an earlier rounding difference cannot matter
    pr.load_oracle_states_into_gpu()
    pr.rounds(1)
    pr.gpu.sync()
    got = pr.gpu.get_assign().cpu().numpy()
    checked = 0
    for i in range(wl.W):
        tr = pr.cpu.last_step(i)
        ok = decided(tr["d1"], tr["d2"])
        # every path, the split-precision tensor-core one included: the nearest centre of Eq. 8, exactly
        assert (got[i][ok] == tr["assign"][ok]).all(), (name, i)
        # counts n_k of Eq. 9: equal to the oracle's per centre, up to the undecided rows either side gave it
        und = ~ok
        slack = np.bincount(got[i][und], minlength=wl.k) + np.bincount(tr["assign"][und], minlength=wl.k)
        diff = np.abs(np.bincount(got[i], minlength=wl.k) - tr["counts"])
        assert (diff <= slack).all(), (name, i, diff, slack)
        checked += int(ok.sum())
    assert checked >= 0.99 * wl.W * wl.b
    assert pr.max_rel_l2() < pr.centre_tol()
    pr.close()


@pytest.mark.parametrize("name", ["dense", "codebook"])
@pytest.mark.parametrize("fmt", ["fp16", "bf16x3"])
def test_tensor_core_formats_decide_exactly(name, fmt):
    """Both operand formats of the tensor-core path (one FP16 term; two BF16 terms) against the oracle: the
    trajectory within the centre tolerance, the assignments of a round started from the oracle's states exactly."""
    wl, rounds = PARITY_WORKLOADS[name]
    pr = Pair(wl, dist_path=pkg.PATH_TC_FP16 if fmt == "fp16" else pkg.PATH_TC_BF16)
    assert pr.gpu.path_name() == "tcgen05-" + fmt
    pr.rounds(rounds)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL, (name, fmt, pr.max_rel_l2())
    pr.load_oracle_states_into_gpu()
    pr.rounds(1)
    pr.gpu.sync()
    got = pr.gpu.get_assign().cpu().numpy()
    for i in range(wl.W):
        tr = pr.cpu.last_step(i)
        ok = decided(tr["d1"], tr["d2"])
        assert (got[i][ok] == tr["assign"][ok]).all(), (name, fmt, i)
        assert ok.mean() > 0.99
    _compare_stats(pr, exact_accept=False)
    pr.close()


@pytest.mark.parametrize("fmt", ["fp16", "bf16x3"])
def test_tensor_core_rows_with_many_candidates(fmt):
    """Bundles of five centres a hair apart: for the rows of their clusters the rounding bound of the 16-bit scores
    leaves three, four or five candidates, so the triple settlement and the scans over all centres (batches of 16 and
    of 4 rows) decide them; every decided row must still get the oracle's centre."""
    rng = np.random.default_rng(77)
    k, d, b, W = 200, 64, 256, 2
    wl = scaled("dense", N=W * b * 3 + 9, k=k, d=d, b=b, W=W, comm_interval=2, eps=0.01)
    mu = rng.standard_normal((8, d)) * 5.0
    X = (mu[rng.integers(0, 8, wl.N)] + rng.standard_normal((wl.N, d))).astype(np.float32)
    w0 = (rng.standard_normal((k, d)) * 5.0 + 40.0).astype(np.float32)            # far from every sample ...
    for c in range(8):                                                             # ... but for a bundle of five per cluster
        for j in range(5):
            w0[5 * c + j] = (mu[c] + (2e-3 if fmt == "fp16" else 2e-4) * rng.standard_normal(d)).astype(np.float32)
    pr = Pair(wl, X=X, w0=w0, dist_path=pkg.PATH_TC_FP16 if fmt == "fp16" else pkg.PATH_TC_BF16)
    assert pr.gpu.path_name() == "tcgen05-" + fmt
    pr.rounds(1)
    pr.gpu.sync()
    got = pr.gpu.get_assign().cpu().numpy()
    decided_rows = 0
    for i in range(wl.W):
        tr = pr.cpu.last_step(i)
        ok = decided(tr["d1"], tr["d2"])
        assert (got[i][ok] == tr["assign"][ok]).all(), (fmt, i, int((got[i][ok] != tr["assign"][ok]).sum()))
        decided_rows += int(ok.sum())
    assert decided_rows > 0.5 * wl.W * wl.b
    assert pr.max_rel_l2() < CENTRE_TOL
    pr.close()


def test_fp16_format_refuses_samples_outside_its_range():
    wl = scaled("dense", N=2 * 256 * 3, W=2, b=256, k=200, d=64, comm_interval=1)
    X = np.random.default_rng(3).standard_normal((wl.N, wl.d)).astype(np.float32) * 3.0e4      # ||x|| far beyond 65504 / 8
    with pytest.raises(pkg.AsgdError) as err:
        Pair(wl, X=X, oracle=False, dist_path=pkg.PATH_TC_FP16)
    assert err.value.status == pkg.binding.ASGD_EUNSUPPORTED
    pr = Pair(wl, X=X, dist_path=pkg.PATH_AUTO)                   # AUTO: an fp32 path takes over
    assert pr.gpu.path_name().startswith("fp32")
    pr.rounds(2)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL
    pr.close()
    pr = Pair(wl, X=X, dist_path=pkg.PATH_TC_BF16)                # the two-term BF16 format has fp32's range
    assert pr.gpu.path_name() == "tcgen05-bf16x3"
    pr.rounds(2)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL
    pr.close()


def test_parzen_hand_cases_on_gpu():
    for line in open(os.path.join(GOLD, "parzen_1d_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w, x, eps, v, parzen, delta, w_new = (float(s) for s in line.split())
        wl = scaled("tiny", N=8, d=1, k=1, W=2, b=4, eps=eps, comm_interval=0, fanout=1)
        X = np.full((8, 1), x, np.float32)
        pr = Pair(wl, parzen=int(parzen), X=X, w0=np.array([[w]], np.float32), oracle=False)
        pr.gpu.put(0, 0, torch.tensor([[v]], dtype=torch.float32, device="cuda"))
        pr.gpu.step(1)
        pr.gpu.sync()
        assert pr.gpu.get_accept(0) == [int(delta)], line
        assert pr.gpu.get_accept(1) == [-1]
        assert abs(float(pr.gpu.get_state(0).cpu()[0, 0]) - w_new) < 2e-6, line
        assert abs(float(pr.gpu.get_state(1).cpu()[0, 0]) - (w - eps * (w - x))) < 2e-6
        st = pr.gpu.get_stats(0)
        assert st["received"] == 1 and st["accepted"] == int(delta) and st["steps"] == 1
        pr.close()


EDGE_CASES = {
    "one_worker": dict(N=997, d=3, k=4, W=1, b=33, comm_interval=1, fanout=0),
    "batch_of_one": dict(N=64, d=5, k=3, W=4, b=1, comm_interval=1, fanout=1),
    "one_centre": dict(N=640, d=7, k=1, W=4, b=40, comm_interval=2, fanout=2),
    "one_dim": dict(N=640, d=1, k=5, W=4, b=40, comm_interval=1, fanout=1),
    "more_centres_than_samples": dict(N=400, d=6, k=50, W=4, b=10, comm_interval=1, fanout=1),
    "silent": dict(N=4000, d=10, k=10, W=8, b=100, comm_interval=0, fanout=1),
    "fanout_all_peers": dict(N=4000, d=10, k=10, W=5, b=50, comm_interval=1, fanout=4),
    "ragged_rows": dict(N=4003, d=9, k=7, W=7, b=37, comm_interval=3, fanout=2),
    "odd_kd": dict(N=3000, d=3, k=3, W=3, b=97, comm_interval=1, fanout=1),
    # shapes of the streaming kernel: misaligned batch starts, a batch that ends on X's last row
    "stream_2x3_to_the_last_row": dict(N=582, d=2, k=3, W=3, b=97, comm_interval=1, fanout=1),
    "stream_4x5": dict(N=5 * 333 + 2, d=4, k=5, W=5, b=111, comm_interval=2, fanout=2),
    "stream_16x16": dict(N=6 * 700, d=16, k=16, W=6, b=175, comm_interval=1, fanout=1),
    "stream_10x10_one_sample": dict(N=40, d=10, k=10, W=4, b=1, comm_interval=1, fanout=1),
    "stream_10x10_to_the_last_row": dict(N=4 * 33 * 3, d=10, k=10, W=4, b=33, comm_interval=1, fanout=3),
    "stream_10x10_full_block": dict(N=3 * 512 * 3 + 7, d=10, k=10, W=3, b=512, comm_interval=2, fanout=1),
    "stream_10x10_odd_batch": dict(N=3 * 129 * 5, d=10, k=10, W=3, b=129, comm_interval=2, fanout=1),
    # shapes of the register-tiled kernel: padded centres, ragged last tile, several workers per block
    "tiled_32_k37_ragged_tile": dict(N=5 * 100 * 3 + 1, d=32, k=37, W=5, b=100, comm_interval=2, fanout=2),
    "tiled_32_many_workers": dict(N=700 * 12, d=32, k=8, W=700, b=4, comm_interval=1, fanout=1),
    "tiled_32_small_blocks_one_worker_each": dict(N=592 * 70 * 2, d=32, k=64, W=592, b=70, comm_interval=2, fanout=1),
    "tiled_128_k128": dict(N=3 * 200 * 2, d=128, k=128, W=3, b=200, comm_interval=1, fanout=1, path=pkg.PATH_FP32),
    "tiled_128_k5_tiny_batch": dict(N=4 * 7 * 3, d=128, k=5, W=4, b=7, comm_interval=1, fanout=3),
    # shapes of the tensor-core kernel: a centre block that is not full, one K chunk, a ragged last sample tile
    "tc_d64_k300_ragged": dict(N=3 * 200 * 3 + 5, d=64, k=300, W=3, b=200, comm_interval=2, fanout=1),
    "tc_d128_k129": dict(N=2 * 128 * 4, d=128, k=129, W=2, b=128, comm_interval=1, fanout=1),
    # ... a state of one centre block (narrower MMA), two blocks per SM, a block's workers taking turns
    "tc_d128_k128_one_block": dict(N=3 * 200 * 2, d=128, k=128, W=3, b=200, comm_interval=1, fanout=1),
    "tc_d64_k17_one_block": dict(N=4 * 150 * 3 + 2, d=64, k=17, W=4, b=150, comm_interval=2, fanout=2),
    "tc_d128_k100_two_blocks_per_sm_workers_in_turn": dict(N=310 * 128 * 2, d=128, k=100, W=310, b=128, comm_interval=1, fanout=2),
    "tc_d256_k40_workers_in_turn": dict(N=320 * 128 * 2 + 9, d=256, k=40, W=320, b=128, comm_interval=2, fanout=1),
    "general_10x10_big_batch": dict(N=2 * 700 * 3, d=10, k=10, W=2, b=700, comm_interval=2, fanout=1),
}


@pytest.mark.parametrize("case", list(EDGE_CASES))
@pytest.mark.parametrize("parzen", [1, 0])
def test_edge_cases(case, parzen):
    kw = dict(EDGE_CASES[case])
    path = kw.pop("path", pkg.PATH_AUTO)
    wl = scaled("tiny", eps=0.1, **kw)
    slots = 3 if case in ("fanout_all_peers", "ragged_rows") else None
    pr = Pair(wl, parzen=parzen, slots=slots, dist_path=path)
    if case.startswith(("tiled_", "tc_", "stream_")):
        assert pr.gpu.path_name().startswith({"tiled_": "fp32-tiled", "tc_": "tcgen05", "stream_": "fp32-stream"}[case[:case.index("_") + 1]])
    rounds = 2 * wl.B + 3
    pr.rounds(rounds)
    pr.gpu.sync()
    assert pr.max_rel_l2() < pr.centre_tol(), (case, pr.max_rel_l2())
    _compare_stats(pr, exact_accept=(parzen == 0))
    pr.close()


@pytest.mark.parametrize("shape", [(10, 10, 512), (10, 10, 500), (16, 16, 300), (4, 5, 111), (2, 3, 257)])
@pytest.mark.parametrize("split", ["one_centre_takes_all", "two_centres_share", "one_centre_takes_most"])
def test_stream_kernel_with_unbalanced_centres(shape, split):
    """Centres that take very different numbers of rows: a warp's rows of one centre then span many groups of
    eight (up to all sixteen), which is what the group sums and their totals in the update have to get right."""
    d, k, b = shape
    W = 3
    wl = scaled("tiny", N=W * b * 4 + 5, d=d, k=k, W=W, b=b, comm_interval=2, fanout=1, eps=0.1)
    rng = np.random.default_rng(1234 + d + k)
    X = rng.standard_normal((wl.N, d)).astype(np.float32)
    w0 = (50.0 + 10.0 * rng.standard_normal((k, d))).astype(np.float32)       # far from every sample
    if split == "one_centre_takes_all":
        w0[k - 1] = 0.0
    elif split == "two_centres_share":
        w0[0] = 0.3
        w0[k - 1] = -0.3
    else:
        w0[1] = 0.0
        w0[0] = 1.2                                                            # a small share for a second centre
    pr = Pair(wl, X=X, w0=w0)
    assert pr.gpu.path_name() == "fp32-stream"
    pr.rounds(9)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL, (shape, split, pr.max_rel_l2())
    _compare_stats(pr, exact_accept=False)
    pr.close()


def test_specialised_and_general_kernels_agree():
    wl = scaled("tiny", N=30_000)
    a = Pair(wl, oracle=False)
    g = Pair(wl, oracle=False, dist_path=pkg.PATH_FP32_GENERAL)
    assert a.gpu.path_name() == "fp32-stream" and g.gpu.path_name() == "fp32-generic"
    a.gpu.step(60)
    g.gpu.step(60)
    assert (a.gpu.get_assign() == g.gpu.get_assign()).all()
    sa, sg = a.gpu_states().astype(np.float64), g.gpu_states().astype(np.float64)
    assert np.sqrt(((sa - sg) ** 2).sum()) / np.sqrt((sg ** 2).sum()) < 1e-5
    for i in range(wl.W):
        assert a.gpu.get_stats(i) == g.gpu.get_stats(i)
    a.close()
    g.close()


def test_dense_shape_on_the_fp32_kernel_too():
    wl, rounds = PARITY_WORKLOADS["dense"]
    pr = Pair(wl, dist_path=pkg.PATH_FP32_GENERAL)
    assert pr.gpu.path_name().startswith("fp32-generic")
    pr.rounds(rounds)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL
    pr.close()


def test_unshuffled_batches_and_many_slots():
    wl = scaled("tiny", N=6000, W=6, comm_interval=1, fanout=3)
    pr = Pair(wl, shuffle=0, slots=2)
    pr.rounds(25)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL
    _compare_stats(pr, exact_accept=False)
    assert sum(pr.cpu.stats(i)["overwritten"] for i in range(wl.W)) > 0     # collisions did happen
    pr.close()


def test_eval_and_mean_state():
    wl = scaled("tiny", N=50_000)
    pr = Pair(wl)
    pr.rounds(30)
    E = pr.gpu.eval(0)
    want = orc.quantization_error(pr.Xh, pr.gpu.get_state(0).cpu().numpy())
    assert abs(E - want) <= 1e-5 * want
    mean = pr.gpu.get_state(-1).cpu().numpy()
    assert np.allclose(mean, pr.gpu_states().astype(np.float64).mean(0), rtol=1e-6, atol=1e-6)
    Em = pr.gpu.eval(-1)
    assert abs(Em - orc.quantization_error(pr.Xh, mean)) <= 1e-5 * Em
    pr.close()


def test_free_running_mode_reaches_the_oracles_error():
    wl = scaled("tiny")
    pr = Pair(wl, record_assign=0)
    steps = wl.steps_per_worker()
    pr.gpu.run(steps)
    pr.gpu.sync()
    pr.cpu.rounds(steps)
    E_gpu = orc.quantization_error(pr.Xh, pr.gpu.get_state(0).cpu().numpy())
    E_cpu = orc.quantization_error(pr.Xh, pr.cpu.state(0))
    assert abs(E_gpu - E_cpu) <= 0.01 * E_cpu, (E_gpu, E_cpu)
    tot = {key: sum(pr.gpu.get_stats(i)[key] for i in range(wl.W)) for key in
           ("steps", "sent", "received", "accepted", "overwritten")}
    assert tot["steps"] == wl.W * steps
    assert tot["sent"] == wl.W * wl.fanout * (steps // wl.comm_interval)
    assert tot["received"] + tot["overwritten"] <= tot["sent"]
    assert tot["accepted"] <= tot["received"]
    pr.close()


# One persistent launch of several steps with no messages (c = 0) is deterministic: a worker's states after it are
# those of the oracle's synchronous rounds.  The shapes take every worker kernel and every instance of the
# tensor-core one through what only a multi-step launch exercises: pipeline phases that run on from step to step, the
# two product-issuing threads with odd numbers of centre blocks and of sample tiles, three K chunks in a four-slot ring,
# the two-term format, workers that share a block in turn, two blocks on an SM.
SILENT_LAUNCHES = {
    "stream": (dict(N=4 * 100 * 4 + 3, d=10, k=10, W=4, b=100), pkg.PATH_AUTO, "fp32-stream"),
    "tiled_d32": (dict(N=5 * 100 * 3 + 1, d=32, k=37, W=5, b=100), pkg.PATH_AUTO, "fp32-tiled"),
    "tc_512_threads_three_blocks": (dict(N=2 * 300 * 3 + 5, d=128, k=600, W=2, b=300), pkg.PATH_AUTO, "tcgen05-fp16"),
    "tc_512_threads_one_chunk": (dict(N=2 * 256 * 3, d=64, k=520, W=2, b=256), pkg.PATH_AUTO, "tcgen05-fp16"),
    "tc_384_threads_three_chunks": (dict(N=2 * 300 * 3 + 5, d=192, k=600, W=2, b=300), pkg.PATH_AUTO, "tcgen05-fp16"),
    "tc_384_threads_d256": (dict(N=2 * 384 * 2 + 1, d=256, k=700, W=2, b=384), pkg.PATH_AUTO, "tcgen05-fp16"),
    "tc_two_terms_three_blocks": (dict(N=2 * 200 * 3, d=256, k=300, W=2, b=200), pkg.PATH_TC_BF16, "tcgen05-bf16x3"),
    "tc_two_terms_d128": (dict(N=3 * 200 * 3, d=128, k=300, W=3, b=200), pkg.PATH_TC_BF16, "tcgen05-bf16x3"),
    "tc_two_blocks_per_sm_workers_in_turn": (dict(N=310 * 128 * 2, d=128, k=100, W=310, b=128), pkg.PATH_AUTO, "tcgen05-fp16"),
    "general": (dict(N=3 * 50 * 4 + 2, d=9, k=7, W=3, b=50), pkg.PATH_AUTO, "fp32-generic"),
}


@pytest.mark.parametrize("case", list(SILENT_LAUNCHES))
def test_silent_multi_step_launch_equals_the_oracles_rounds(case):
    over, path, want = SILENT_LAUNCHES[case]
    wl = scaled("tiny", eps=0.1, comm_interval=0, fanout=1, **over)
    pr = Pair(wl, dist_path=path, record_assign=0)
    assert pr.gpu.path_name() == want, (case, pr.gpu.path_name())
    steps = 2 * wl.B + 3
    pr.gpu.run(steps)
    pr.gpu.sync()
    pr.cpu.rounds(steps)
    assert pr.max_rel_l2() < pr.centre_tol(), (case, pr.max_rel_l2())
    assert all(pr.gpu.get_stats(i)["steps"] == steps for i in range(wl.W))
    pr.gpu.run(2)                                         # a second launch picks the counters up where the first left them
    pr.gpu.sync()
    pr.cpu.rounds(2)
    assert pr.max_rel_l2() < pr.centre_tol(), (case, pr.max_rel_l2())
    pr.close()


def test_mixing_deterministic_rounds_and_free_running():
    wl = scaled("tiny", N=20_000)
    pr = Pair(wl, record_assign=0)
    pr.rounds(10)
    pr.gpu.sync()
    assert pr.max_rel_l2() < CENTRE_TOL
    pr.gpu.run(15)
    pr.gpu.step(5)
    pr.gpu.sync()
    assert all(pr.gpu.get_stats(i)["steps"] == 30 for i in range(wl.W))
    pr.close()


def test_fit_host_end_to_end():
    wl = scaled("tiny", N=20_000)
    pr = Pair(wl, record_assign=0)
    rounds = 40
    pr.rounds(rounds)
    cfg = pr.cfg
    cfg.record_assign = 0
    Xp = torch.from_numpy(pr.Xh).pin_memory()
    w0p = torch.from_numpy(pr.w0h).pin_memory()
    out = torch.empty((wl.k, wl.d), dtype=torch.float32).pin_memory()
    scratch = torch.empty(pkg.asgd_fit_host_bytes(cfg) + 256, dtype=torch.uint8, device="cuda")
    off = (-scratch.data_ptr()) % 256
    pkg.asgd_fit_host(cfg, Xp, w0p, rounds, False, out, scratch[off:])
    assert np.array_equal(out.numpy(), pr.gpu.get_state(0).cpu().numpy())
    pr.close()


def test_error_returns():
    import ctypes as C
    L = pkg.load()
    wl = scaled("tiny", N=2000)
    pr = Pair(wl, oracle=False)
    cfg = pr.cfg
    need = pkg.asgd_workspace_bytes(cfg)
    ws = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    base = (ws.data_ptr() + 255) // 256 * 256
    h = C.c_void_p()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (C.byref(cfg), C.c_void_p(pr.X.data_ptr()), None, C.c_void_p(pr.w0.data_ptr()))
    assert L.asgd_init(C.byref(h), *args, C.c_void_p(base), need - 1, st) == pkg.binding.ASGD_ENOMEM
    assert L.asgd_init(C.byref(h), *args, C.c_void_p(base + 8), need, st) == pkg.binding.ASGD_EINVAL
    assert L.asgd_init(C.byref(h), C.byref(cfg), C.c_void_p(pr.X.data_ptr() + 4), None, C.c_void_p(pr.w0.data_ptr()),
                       C.c_void_p(base), need, st) == pkg.binding.ASGD_EINVAL
    with pytest.raises(pkg.AsgdError):
        pr.gpu.get_state(wl.W)
    with pytest.raises(pkg.AsgdError):
        pr.gpu.put(0, pr.S, pr.w0)
    with pytest.raises(ValueError):
        pkg.Asgd(cfg, pr.X.cpu(), pr.w0.cpu())
    pr.close()
