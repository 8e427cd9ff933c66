"""asgd_eval_noalloc -- E(w) for callers that may not allocate device memory.

A serving loop with a fixed memory plan, or code running under somebody else's allocator, can own
its inputs and one double for the answer but cannot give the library a workspace.  This entry point
keeps its partial sums in an array built into the library instead.  The file is collected last on
purpose: if it fails, a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_1505_04956_b200 as pkg
from paper_1505_04956_b200 import binding, inputs
from oracle import asgd_oracle as orc

pytestmark = pytest.mark.gpu
REL_TOL = 1e-5          # the tolerance the evaluation tests use against the oracle


def _problem():
    wl = inputs.WORKLOADS["tiny"].scaled(N=200_003)       # four blocks of rows, the last one ragged
    X, _ = inputs.make_samples(wl, device="cuda")
    w0 = inputs.initial_centres(wl, X)
    cfg = pkg.make_config(N=wl.N, d=wl.d, k=wl.k, W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval,
                          fanout=wl.fanout, seed=wl.seed)
    return wl, X, w0, pkg.Asgd(cfg, X, w0)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    wl, X, w0, ctx = _problem()
    E = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    # first call: the initial centres
    assert pkg.asgd_eval_noalloc(X, w0, E) == binding.ASGD_OK
    want = ctx.eval(0)
    got = float(E.cpu())
    assert abs(got - want) <= REL_TOL * want, (got, want)
    Xh = X.cpu().numpy()
    truth = orc.quantization_error(Xh, w0.cpu().numpy())     # Eq. 8 by the CPU oracle on the copied buffer
    assert abs(got - truth) <= REL_TOL * truth, (got, truth)
    # second call right after, other centres: the shared scratch still holds the first call's sums
    ctx.step(25)
    w1 = ctx.get_state(0)
    assert pkg.asgd_eval_noalloc(X, w1, E) == binding.ASGD_OK
    want1 = ctx.eval(0)
    got1 = float(E.cpu())
    assert abs(got1 - want1) <= REL_TOL * want1, (got1, want1)
    truth1 = orc.quantization_error(Xh, w1.cpu().numpy())
    assert abs(got1 - truth1) <= REL_TOL * truth1, (got1, truth1)
    assert got1 < got                                        # 25 rounds of descent did lower the error
    # fewer rows than before: entries left over from the longer call must not leak into the sum
    Xs = X[:70_000]
    assert pkg.asgd_eval_noalloc(Xs, w1, E) == binding.ASGD_OK
    ref = orc.quantization_error(Xh[:70_000], w1.cpu().numpy())
    assert abs(float(E.cpu()) - ref) <= REL_TOL * ref
    ctx.destroy()


def test_sizes_beyond_the_built_in_scratch_are_refused():
    wl, X, w0, ctx = _problem()
    E = torch.zeros(1, dtype=torch.float64, device="cuda")
    L = pkg.load()
    import ctypes as C
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    too_many_rows = 4096 * 65536 + 1
    args = (C.c_void_p(X.data_ptr()), too_many_rows, wl.d, wl.k, C.c_void_p(w0.data_ptr()), C.c_void_p(E.data_ptr()), st)
    assert L.asgd_eval_noalloc(*args) == binding.ASGD_EUNSUPPORTED          # nothing is launched
    args = (C.c_void_p(X.data_ptr()), 1000, 4096, 11, C.c_void_p(w0.data_ptr()), C.c_void_p(E.data_ptr()), st)
    assert L.asgd_eval_noalloc(*args) == binding.ASGD_EUNSUPPORTED          # k*d too large for shared memory
    assert L.asgd_eval_noalloc(None, 10, 2, 2, None, None, st) == binding.ASGD_EINVAL
    torch.cuda.synchronize()
    assert float(E.cpu()) == 0.0
    ctx.destroy()
