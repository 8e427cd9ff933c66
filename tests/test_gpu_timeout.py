"""The bounded device-side waits: a wait that runs out must end the kernel with ASGD_ETIMEOUT, not hang it.

A worker kernel waits only for its own asynchronous sample copies.  The drill announces one copy to its
barrier without issuing it (nothing faults, nothing is left in flight), so the wait expires after the
configured number of polls; the block raises the status word and returns through its abort path.  The
device must stay usable: a fresh context afterwards runs clean and matches the oracle.
"""
import pytest

import paper_1505_04956_b200 as pkg
from paper_1505_04956_b200 import binding
from tests.gpu_util import Pair, scaled

pytestmark = pytest.mark.gpu

CASES = {
    # kernel: (workload, path name)
    "stream": (scaled("tiny", N=4 * 100 * 6, comm_interval=2), "fp32-stream"),
    "tiled": (scaled("sweep", N=6 * 256 * 5 + 3, W=6, comm_interval=2), "fp32-tiled"),
    "tensor": (scaled("dense", N=2 * 512 * 5 + 1, W=2, b=512, comm_interval=2), "tcgen05-fp16"),
    "tensor_two_terms": (scaled("dense", N=2 * 512 * 5 + 1, W=2, b=512, comm_interval=2), "tcgen05-bf16x3"),
}


@pytest.mark.parametrize("kernel", list(CASES))
def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable(kernel):
    wl, path = CASES[kernel]
    dist_path = pkg.PATH_TC_BF16 if kernel == "tensor_two_terms" else pkg.PATH_AUTO
    pr = Pair(wl, oracle=False, record_assign=0, dist_path=dist_path)
    assert pr.gpu.path_name().startswith(path)
    pr.gpu.run(2)
    pr.gpu.sync()                                     # nothing wrong so far
    pr.gpu.set_wait_drill(3000, 1)                    # the next launch never gets the samples of its second step
    pr.gpu.run(4)
    with pytest.raises(pkg.AsgdError) as err:
        pr.gpu.sync()
    assert err.value.status == binding.ASGD_ETIMEOUT
    # every worker finished the launch's first step and gave up in the second
    assert [pr.gpu.get_stats(i)["steps"] for i in range(wl.W)] == [3] * wl.W
    pr.close()

    # a fresh context on the same device: the kernel left nothing behind (shared memory, tensor memory, status)
    again = Pair(wl, dist_path=dist_path)
    again.rounds(3)
    again.gpu.sync()
    assert again.max_rel_l2() < again.centre_tol()
    again.close()


def test_drill_arguments():
    wl, _ = CASES["stream"]
    pr = Pair(wl, oracle=False, record_assign=0)
    with pytest.raises(pkg.AsgdError):
        pr.gpu.set_wait_drill(0, 1)
    pr.gpu.set_wait_drill(1 << 22, -1)                # back to the defaults
    pr.gpu.run(3)
    pr.gpu.sync()
    pr.close()
