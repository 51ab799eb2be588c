"""The multi-GPU form of the benchmark is replicas only: no data-path collective, every rank times the same
work and the job's time is the slowest rank's.  This covers that plumbing with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, {root!r})
    import torch, torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]          # no group yet: identity
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 10.0 - rank, 3.0]                                   # per-rank device times (ms)
    got = bench.max_over_ranks(mine, "cpu")
    dist.barrier()
    out = {{"rank": rank, "max": got, "value": bench.whole_job(1e9, world, got[0])}}
    print("RESULT " + json.dumps(out), flush=True)
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_max_over_ranks_with_two_gloo_ranks():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    for rank, p in enumerate(procs):
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        line = [ln for ln in out.splitlines() if ln.startswith("RESULT ")][-1]
        res = json.loads(line[len("RESULT "):])
        assert res["rank"] == rank
        assert res["max"] == [2.0, 10.0, 3.0]                 # the slowest rank decides, element by element
        assert res["value"] == 2 * 1e9 / 2.0e-3                # whole-job units over the slowest rank's time


def test_reference_arm_runs_on_rank_zero_only():
    # under torchrun the other ranks of `--impl reference` exit 0 without work and without output
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=240)
    assert p.returncode == 0, p.stderr[-2000:]
    assert p.stdout.strip() == ""
