"""Host-side arithmetic of bench.py: the roofline numerator and the key of the stored traffic record (no GPU)."""
import importlib.util
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes_of_the_stream_workload():
    """Section 5.3 shape: 592 workers x 906 batches of 500 rows of 40 bytes, one 400-byte state per put (every 20 steps)."""
    from paper_1505_04956_b200 import inputs
    bench = _bench()
    wl = inputs.WORKLOADS["stream"]
    assert wl.B == 906
    samples = 592 * 906 * 500 * 40
    puts = 592 * (906 // 20) * 400
    assert bench.algorithmic_bytes_per_pass(wl, wl.B) == samples + puts == 10_737_696_000
    # per-centre messages carry only their rows; silent mode sends nothing
    assert bench.algorithmic_bytes_per_pass(wl, wl.B, partial_rows=3) == samples + 592 * 45 * 3 * 40
    assert bench.algorithmic_bytes_per_pass(wl.scaled(comm_interval=0), wl.B) == samples


def test_traffic_records_are_keyed_on_the_kernel_sources():
    bench = _bench()
    for (kernel, workload), rec in bench.TRAFFIC_CAPTURES.items():
        assert kernel in bench.KERNEL_SOURCES
        assert re.fullmatch(r"[0-9a-f]{12}", bench.kernel_sha1(kernel))
        assert 0.5 <= rec["traffic_per_algorithmic_byte"] < 8.0
    # a record taken on other sources is not used
    bench.TRAFFIC_CAPTURES[("fp32-stream", "stream")] = {"kernel_sha1": "000000000000", "traffic_per_algorithmic_byte": 1.0}
    assert bench.captured_traffic("fp32-stream", "stream", 1000)[0] is None
    bench.TRAFFIC_CAPTURES[("fp32-stream", "stream")]["kernel_sha1"] = bench.kernel_sha1("fp32-stream")
    assert bench.captured_traffic("fp32-stream", "stream", 1000)[0] == 1000
    assert bench.captured_traffic("fp32-generic", "tiny", 1000)[0] is None
