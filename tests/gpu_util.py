"""Helpers of the GPU parity tests: build the same problem for the CUDA library and for the oracle."""
import numpy as np
import torch

import paper_1505_04956_b200 as pkg
from paper_1505_04956_b200 import inputs
from oracle import asgd_oracle as orc

# Tolerances of the deterministic mode (stated for the library): centres within 1e-4 relative L2 of
# the oracle's; assignments bit-exact except samples whose two smallest squared distances differ by
# less than 1e-5 relative (their fp32 order is not decided).
CENTRE_TOL = 1e-4           # every path: the tensor-core path decides Eq. 8 exactly and sums the fp32 samples
TIE_EXCLUSION = 1e-5


def scaled(name, **kw):
    return inputs.WORKLOADS[name].scaled(**kw)


PARITY_WORKLOADS = {
    # name: (workload, rounds)
    "tiny": (scaled("tiny"), 1000),
    "stream": (scaled("stream", N=37 * 500 * 7 + 13, W=37, comm_interval=4), 14),
    "mid": (scaled("mid", N=8 * 3000 + 5, W=8, comm_interval=2), 6),
    "sweep": (scaled("sweep", N=16 * 1024 + 3, W=16, comm_interval=1), 8),
    "dense": (scaled("dense", N=2 * 2048 + 1, W=2, b=1024, comm_interval=1), 3),
    "codebook": (scaled("codebook", N=2 * 1536 + 7, W=2, b=512, comm_interval=1), 3),
}


class Pair:
    """The CUDA context and the oracle on identical inputs."""

    def __init__(self, wl, *, parzen=1, slots=None, shuffle=1, record_assign=1, dist_path=pkg.PATH_AUTO,
                 X=None, w0=None, oracle=True, device="cuda", partial_rows=0):
        self.wl = wl
        if X is None:
            Xh, _ = inputs.make_samples(wl, device="cpu")
        else:
            Xh = torch.as_tensor(X, dtype=torch.float32)
        w0h = inputs.initial_centres(wl, Xh) if w0 is None else torch.as_tensor(w0, dtype=torch.float32)
        self.Xh, self.w0h = Xh.numpy(), w0h.numpy()
        self.X, self.w0 = Xh.to(device), w0h.to(device)
        S = slots if slots else max(1, wl.fanout)
        self.S = S
        self.cfg = pkg.make_config(N=Xh.shape[0], d=wl.d, k=wl.k, W=wl.W, b=wl.b, eps=wl.eps,
                                   comm_interval=wl.comm_interval, fanout=wl.fanout, slots=S, parzen=parzen,
                                   shuffle=shuffle, record_assign=record_assign, seed=wl.seed, dist_path=dist_path,
                                   partial_rows=partial_rows)
        self.gpu = pkg.Asgd(self.cfg, self.X, self.w0)
        self.cpu = None
        if oracle:
            self.cpu = orc.Oracle(self.Xh, self.w0h, W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval,
                                  fanout=wl.fanout, slots=S, parzen=parzen, shuffle=shuffle, seed=wl.seed,
                                  partial_rows=partial_rows)

    def centre_tol(self):
        return CENTRE_TOL

    def rounds(self, n):
        self.gpu.step(n)
        self.cpu.rounds(n)

    def gpu_states(self):
        return np.stack([self.gpu.get_state(i).cpu().numpy() for i in range(self.wl.W)])

    def max_rel_l2(self):
        g = self.gpu_states().astype(np.float64)
        c = self.cpu.states().astype(np.float64)
        num = np.sqrt(((g - c) ** 2).sum(axis=(1, 2)))
        den = np.sqrt((c ** 2).sum(axis=(1, 2)))
        return float((num / den).max())

    def load_oracle_states_into_gpu(self):
        for i in range(self.wl.W):
            self.gpu.set_state(i, torch.from_numpy(self.cpu.state(i)).to(self.X.device))

    def close(self):
        self.gpu.destroy()
        if self.cpu is not None:
            self.cpu.close()


def decided(d1, d2):
    """Mask of samples whose nearest centre is decided beyond the stated relative gap."""
    return (d2 - d1) >= TIE_EXCLUSION * d2
