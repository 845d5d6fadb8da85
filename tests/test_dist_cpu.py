"""The benchmark's multi-process plumbing on CPU: two gloo ranks, each a replica with its own units and
time; the job's throughput is all units over the slowest rank's time."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    from paper_2605_22269_b200 import dist as D
    rank, world, local = D.init_from_env("gloo")
    assert world == 2 and rank in (0, 1)
    D.barrier()
    ms, units = D.combine(10.0 * (rank + 1), 100.0 * (rank + 1))
    assert ms == 20.0 and units == 300.0, (ms, units)
    fps = D.throughput(10.0 * (rank + 1), 100.0 * (rank + 1))
    assert abs(fps - 300.0 / 0.020) < 1e-6, fps
    D.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_combine_time_and_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_is_a_no_op():
    from paper_2605_22269_b200 import dist as D
    assert D.combine(5.0, 7.0) == (5.0, 7.0)
    assert D.throughput(2000.0, 10.0) == 5.0
