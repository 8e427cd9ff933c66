"""The C-ABI library loads without a GPU and exports every function include/asgd.h declares."""
import ctypes as C
import os
import re

import paper_1505_04956_b200 as pkg
from paper_1505_04956_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "asgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(asgd_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = libbuild.build()
    lib = C.CDLL(path)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(pkg.EXPORTS)


def test_probe_library_builds_and_exports_its_entry_point():
    text = open(os.path.join(ROOT, "include", "asgd_probe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = sorted(set(re.findall(r"\b(asgd_[a-z0-9_]+)\s*\(", text)))
    assert names == ["asgd_probe_issue_rates", "asgd_probe_mma_rates"]
    lib = C.CDLL(libbuild.build_probe())
    for n in names:
        assert hasattr(lib, n), n
    lib.asgd_probe_issue_rates.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int]
    assert lib.asgd_probe_issue_rates(None, 13, None, 148) == -1           # argument check, nothing launched


def test_argument_checks_need_no_gpu():
    L = pkg.load()
    cfg = pkg.make_config(N=1000, d=4, k=3, W=2, b=10, eps=0.1, comm_interval=1, fanout=1)
    assert pkg.asgd_workspace_bytes(cfg) > 0
    n = C.c_size_t(0)
    bad = pkg.make_config(N=1000, d=4, k=3, W=2, b=10, eps=0.1, comm_interval=1, fanout=2)   # f > W-1
    assert L.asgd_workspace_bytes(C.byref(bad), C.byref(n)) == pkg.binding.ASGD_EINVAL
    bad = pkg.make_config(N=10, d=4, k=3, W=2, b=10, eps=0.1)                                 # b > H
    assert L.asgd_workspace_bytes(C.byref(bad), C.byref(n)) == pkg.binding.ASGD_EINVAL
    bad = pkg.make_config(N=1000, d=4, k=3, W=2, b=10, eps=0.0)
    assert L.asgd_workspace_bytes(C.byref(bad), C.byref(n)) == pkg.binding.ASGD_EINVAL
    assert L.asgd_workspace_bytes(None, C.byref(n)) == pkg.binding.ASGD_EINVAL
    h = C.c_void_p()
    assert L.asgd_init(C.byref(h), C.byref(cfg), None, None, None, None, 0, None) == pkg.binding.ASGD_EINVAL
    assert L.asgd_step(None, 1) == pkg.binding.ASGD_EINVAL
    assert L.asgd_run(None, 1) == pkg.binding.ASGD_EINVAL
    assert pkg.binding.strerror(pkg.binding.ASGD_ETIMEOUT).startswith("a bounded")
    assert pkg.binding.strerror(0) == "ok"


def test_workspace_grows_with_the_problem():
    small = pkg.asgd_workspace_bytes(pkg.make_config(N=10000, d=8, k=4, W=4, b=10, eps=0.1))
    big = pkg.asgd_workspace_bytes(pkg.make_config(N=10000, d=8, k=64, W=16, b=10, eps=0.1, fanout=2, comm_interval=1))
    assert big > small
