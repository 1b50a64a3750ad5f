"""The N > 1 path of the benchmark on CPU: two gloo ranks stand in for two GPUs running independent
replicas; the whole-job figure must be (sum of units) / (slowest rank's time)."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2410_23608_b200 import replicas
    rank, local, n = replicas.world()
    assert replicas.init("gloo") == 2
    replicas.barrier()
    ms_local = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
    units_local = 1000.0 if rank == 0 else 3000.0
    rate, ms = replicas.whole_job_rate(units_local, ms_local)
    assert ms == 25.0, ms
    assert abs(rate - 4000.0 / 25e-3) < 1e-6, rate
    assert replicas.reduce_scalar(float(rank), "sum") == 1.0
    assert replicas.reduce_scalar(float(rank), "max") == 1.0
    replicas.barrier()
    replicas.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_like_two_replicas(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_is_a_no_op():
    from paper_2410_23608_b200 import replicas
    assert replicas.reduce_scalar(3.5, "max") == 3.5
    rate, ms = replicas.whole_job_rate(100.0, 50.0)
    assert ms == 50.0 and abs(rate - 2000.0) < 1e-9
    replicas.barrier()
