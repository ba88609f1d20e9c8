"""bench.py at more than one rank runs independent replicas (requests never interact, so the path has no
collective): the process group carries only the barrier and the max-over-ranks of the timing.  That host logic,
on two CPU ranks over gloo."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_PROGRAM = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, os.environ["REPO_ROOT"])
    import bench
    world, rank, local = bench.dist_setup(2, backend="gloo")
    assert world == 2 and rank == int(os.environ["RANK"]) and local == int(os.environ["LOCAL_RANK"])
    bench.barrier(world)
    mine = 1.5 + rank                      # this rank's ms per step: rank 1 is the slow one
    worst = bench.max_over_ranks(world, mine)
    value = bench.whole_job_value(world, 256, worst)
    bench.barrier(world)
    if rank == 0:                          # rank 0 alone reports
        print(json.dumps({"worst_ms": worst, "value": value}), flush=True)
    import torch.distributed as dist
    dist.destroy_process_group()
""")


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_report_all_units_over_the_slowest_rank():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, REPO_ROOT=ROOT, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_PROGRAM], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert outs[1][0].strip() == ""                       # rank 1 prints nothing
    assert line["worst_ms"] == 2.5                        # max over ranks, not rank 0's own 1.5
    assert abs(line["value"] - 2 * 256 / 2.5e-3) < 1e-6   # units of BOTH replicas over the slowest time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1, 3.25) == 3.25
    assert bench.whole_job_value(1, 256, 0.25) == 256 / 0.25e-3
    bench.barrier(1)
