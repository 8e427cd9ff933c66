"""Seeded random configurations through every kernel against the oracle: sizes, worker counts, batch
sizes, communication interval, fan-out, buffers, window on/off and rows per message are drawn at random
(fixed seeds), so that shapes nobody thought of still get a parity check."""
import numpy as np
import pytest

import paper_1505_04956_b200 as pkg
from tests.gpu_util import Pair, scaled

pytestmark = pytest.mark.gpu

# (d, k) pools per kernel family: streaming shapes, register-tiled shapes (asked for by name where the tensor-core
# path would be the library's choice), tensor-core shapes of several and of one centre block, everything else
FAMILIES = {
    "stream": [(10, 10), (16, 16), (4, 5), (2, 3)],
    "tiled": [(32, 64), (32, 9), (128, 100), (128, 17)],
    "tensor": [(64, 130), (128, 200), (256, 129)],
    "tensor_one_block": [(128, 100), (64, 17), (192, 128), (256, 33), (128, 3)],
    "general": [(3, 7), (9, 4), (12, 33), (1, 2), (20, 20), (64, 5)],
}


def _draw(family, seed):
    rng = np.random.default_rng(1000 * seed + sum(map(ord, family)))
    d, k = FAMILIES[family][rng.integers(len(FAMILIES[family]))]
    W = int(rng.integers(1, 9))
    if family == "stream":
        b = int(rng.integers(1, 513))
    elif family.startswith("tensor"):
        b = int(rng.integers(128, 400))
    else:
        b = int(rng.integers(1, 150))
    batches = int(rng.integers(1, 4))
    N = W * (b * batches + int(rng.integers(0, b))) + int(rng.integers(0, W))
    fanout = int(rng.integers(0, min(W - 1, 3) + 1)) if W > 1 else 0
    c = int(rng.integers(0, 4))
    slots = int(rng.integers(1, 4))
    parzen = int(rng.integers(0, 2))
    rows = int(rng.integers(1, k + 1)) if rng.integers(0, 2) else 0
    eps = float(rng.choice([0.02, 0.1, 0.5]))
    return dict(N=N, d=d, k=k, W=W, b=b, comm_interval=c, fanout=fanout, eps=eps), slots, parzen, rows, batches


@pytest.mark.parametrize("family", list(FAMILIES))
@pytest.mark.parametrize("seed", range(8))
def test_random_configuration_matches_oracle(family, seed):
    over, slots, parzen, rows, batches = _draw(family, seed)
    wl = scaled("tiny", **over)
    pr = Pair(wl, parzen=parzen, slots=slots, partial_rows=rows, shuffle=int(seed % 2),
              dist_path=pkg.PATH_FP32 if family == "tiled" else pkg.PATH_AUTO)
    want = {"stream": "fp32-stream", "tiled": "fp32-tiled", "tensor": "tcgen05-fp16", "tensor_one_block": "tcgen05-fp16",
            "general": "fp32-generic"}[family]
    assert pr.gpu.path_name() == want, (family, seed, over, pr.gpu.path_name())
    rounds = 2 * batches + 1
    pr.rounds(rounds)
    pr.gpu.sync()
    assert pr.max_rel_l2() < pr.centre_tol(), (family, seed, over, pr.gpu.path_name(), pr.max_rel_l2())
    for i in range(wl.W):
        g, c = pr.gpu.get_stats(i), pr.cpu.stats(i)
        for key in ("steps", "sent", "received", "overwritten"):
            assert g[key] == c[key], (family, seed, over, i, key, g, c)
        if parzen == 0:
            assert g["accepted"] == c["accepted"], (family, seed, over, i, g, c)
    pr.close()
