"""bench.py at N > 1 runs independent replicas; the only cross-rank steps are a barrier and the
max-over-ranks of the elapsed time.  This runs bench.py's own reduction (max_over_ranks, whole_job_rate) in two
gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

from conftest import ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_max_over_ranks_two_gloo_processes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(textwrap.dedent("""
        import os, sys, json
        import torch, torch.distributed as dist
        sys.path.insert(0, os.getcwd())
        import bench                                # the functions under test are the benchmark's own
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", rank=rank, world_size=world)
        elapsed_ms = [12.5, 20.25][rank]            # what each replica measured for K steps
        dist.barrier()
        slowest = bench.max_over_ranks(elapsed_ms, world, dist, torch.device("cpu"), torch)
        steps = 5
        value = bench.whole_job_rate(world, steps, slowest)   # all replicas' steps over the slowest replica's time
        alone = bench.max_over_ranks(elapsed_ms, 1)           # a single replica needs no reduction
        if rank == 0:
            print(json.dumps({"max_ms": slowest, "value": value, "alone": alone}))
        dist.destroy_process_group()
    """))
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True, cwd=ROOT))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["max_ms"] == 20.25 and line["alone"] == 12.5
    assert abs(line["value"] - 2 * 5 / 0.02025) < 1e-9
