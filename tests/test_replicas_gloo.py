"""The N > 1 path (independent replicas; barrier + max-over-ranks timing) on CPU with gloo."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2306_00978_b200 import replicas
    replicas.init("gloo")
    rank, world, _ = replicas.env_world()
    replicas.barrier()
    t = replicas.max_over_ranks(0.5 + rank)          # rank 1 is the slow one
    v = replicas.aggregate_throughput(10.0, t)
    replicas.barrier()
    print("RESULT", rank, world, t, v, flush=True)
    replicas.shutdown()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_timing_protocol():
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
    for rank, o in enumerate(outs):
        line = [l for l in o.splitlines() if l.startswith("RESULT")][0].split()
        assert int(line[1]) == rank and int(line[2]) == 2
        assert float(line[3]) == 1.5                       # max over ranks
        assert abs(float(line[4]) - 2 * 10.0 / 1.5) < 1e-12   # both replicas' units / slowest time


def test_single_process_is_identity():
    from paper_2306_00978_b200 import replicas
    assert replicas.max_over_ranks(3.25) == 3.25
    assert replicas.env_world()[1] >= 1
