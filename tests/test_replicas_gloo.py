"""The N > 1 path of bench.py (independent replicas; barrier + max-over-ranks of the timing) on the
gloo backend with two CPU processes."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2411_19460_b200.replicas import Replicas
    r = Replicas(backend="gloo")
    assert r.world == 2
    r.barrier()
    secs = 1.0 + r.rank            # rank 1 is the slow one
    assert r.max_over_ranks(secs) == 2.0
    rate = r.whole_job_rate(100.0, secs)
    assert abs(rate - 2 * 100.0 / 2.0) < 1e-12, rate
    r.barrier()
    r.close()
    print("rank", r.rank, "ok")
""") % ROOT


def test_two_replicas_on_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + (os.getpid() % 2000)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_replica_is_a_no_op_group(monkeypatch):
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    sys.path.insert(0, ROOT)
    from paper_2411_19460_b200.replicas import Replicas
    r = Replicas()
    assert (r.rank, r.world) == (0, 1)
    r.barrier()
    assert r.max_over_ranks(3.5) == 3.5
    assert r.whole_job_rate(10.0, 2.0) == 5.0
