"""World-size-2 gloo test of the benchmark's multi-process plumbing (runs on CPU)."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2609_21264_b200 import launch
    rank, world, local = launch.init_process_group("gloo")
    assert world == 2
    launch.barrier(world)
    # rank 0 takes 1.0 s, rank 1 takes 2.0 s for 10 units each: job = 20 units / 2.0 s
    t = 1.0 + rank
    assert launch.max_over_ranks(t, world) == 2.0
    assert launch.sum_over_ranks(10.0, world) == 20.0
    v = launch.whole_job_throughput(10.0, t, world)
    assert abs(v - 10.0) < 1e-12, v
    launch.barrier(world)
    launch.destroy(world)
    print("rank", rank, "ok")
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_rank_aggregation_over_gloo():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_process_paths_need_no_process_group():
    from paper_2609_21264_b200 import launch
    assert launch.max_over_ranks(3.0, 1) == 3.0
    assert launch.whole_job_throughput(6.0, 2.0, 1) == 3.0
