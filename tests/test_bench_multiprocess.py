"""Host-side logic of the multi-process benchmark path, on CPU with the gloo backend (world size 2).

The OSC linear has no exchange step: N GPUs run N independent replicas.  What the N > 1 path adds is
only the reduction of the per-rank time to the slowest rank and the whole-job rate; this test runs that
code in two real processes.
"""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["OSC_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms_local = 2.0 if rank == 0 else 5.0            # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local)
    value = bench.whole_job_value(1e12, world, ms)  # 1 TFLOP per rank and step
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms": ms, "value": value, "world": world}))
    dist.destroy_process_group()
""")


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_max_over_ranks_and_whole_job_value_with_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, OSC_ROOT=ROOT, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["world"] == 2
    assert line["ms"] == 5.0                                  # the slowest rank's time
    assert abs(line["value"] - 2 * 1e12 / 5e-3 / 1e12) < 1e-9   # two replicas' work over that time
    assert outs[1][0].strip() == ""                            # only rank 0 prints


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25) == 3.25
    assert bench.whole_job_value(2e12, 1, 1.0) == 2000.0
