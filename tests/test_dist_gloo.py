"""Multi-process host logic of the benchmark (rank rendezvous, max/sum over ranks) on gloo, 2 ranks."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_1505_04956_b200 import dist
    rank, world, local = dist.init_from_env(backend="gloo")
    assert world == 2
    dist.barrier()
    assert dist.max_over_ranks(1.0 + rank) == 2.0
    assert dist.sum_over_ranks(10.0 * (rank + 1)) == 30.0
    assert dist.shard_seed(1, rank, world) == 1 + 1000 * rank
    dist.barrier()
    dist.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def test_two_gloo_ranks(tmp_path):
    script = tmp_path / "w.py"
    script.write_text(WORKER)
    port = 29600 + os.getpid() % 300
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "rank %d ok" % r in out


def test_reference_arm_prints_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_1505_04956_b200 import dist
    assert dist.max_over_ranks(3.5) == 3.5 and dist.sum_over_ranks(2.0) == 2.0
    assert dist.shard_seed(7, 0, 1) == 7
    dist.barrier()
