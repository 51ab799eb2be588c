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
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=240)
    assert p.returncode == 0, p.stderr[-2000:]
    assert p.stdout.strip() == ""


TP_WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, {root!r})
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from paper_2608_30386_b200 import tp_exchange
    from paper_2608_30386_b200.binding import dasc_tp_balance
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    U = {units!r}
    width, send = dasc_tp_balance(U)
    o_width, o_send = oracle.tp_balance(U)
    assert width == o_width and np.array_equal(send, o_send)
    # row i of rank r carries the value 1000 * r + i in every column: the global sequence is then recognisable
    mine = (1000.0 * rank + torch.arange(U[rank], dtype=torch.float32)).unsqueeze(1).repeat(1, 4)
    assert tp_exchange.gather_unit_counts(U[rank]) == U
    stored = tp_exchange.store_exchange(mine, U)
    seq = np.concatenate([1000.0 * r + np.arange(U[r]) for r in range(world)])
    want = seq[rank * width: (rank + 1) * width]                  # rank s stores global positions [sC, sC + C)
    assert stored.shape == (len(want), 4) and np.array_equal(stored[:, 0].numpy(), want), (stored[:, 0], want)
    assert stored.shape[0] <= width
    back = tp_exchange.load_exchange(stored, U)
    assert torch.equal(back, mine)                                 # Load is the exact inverse
    dist.barrier()
    print("RESULT ok", flush=True)
    dist.destroy_process_group()
""")


def _run_ranks(script, world):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-3000:]
        assert "RESULT ok" in out


def test_tp_balanced_store_and_load_exchange_two_ranks():
    # Section 4.3: an uneven pair (the heavy rank ships its excess), and an empty rank
    _run_ranks(TP_WORKER.format(root=ROOT, units=[11, 2]), 2)
    _run_ranks(TP_WORKER.format(root=ROOT, units=[0, 5]), 2)


def test_tp_balanced_store_and_load_exchange_three_ranks():
    _run_ranks(TP_WORKER.format(root=ROOT, units=[10, 1, 4]), 3)


def test_bench_starts_its_own_ranks_when_asked_for_several_gpus():
    # `python bench.py --gpus 2` with no launcher around it starts two ranks itself; --dry-launch makes them meet over
    # gloo and count themselves instead of touching a GPU
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-launch"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line == {"dry_launch": True, "n_gpus": 2, "ranks": 2}
    # a rank count that does not match --gpus is refused instead of being printed as n_gpus
    env2 = dict(env, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--dry-launch"], env=env2,
                       capture_output=True, text=True, timeout=120)
    assert p.returncode != 0 and "does not match" in p.stderr
    # without GPUs the real run fails loudly, after both ranks were started
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert p.returncode != 0 and "2 of 2 ranks failed" in p.stderr


def test_serving_trace_is_seeded_bounded_and_hazard_free():
    from paper_2608_30386_b200 import synth
    rounds, st = synth.serving_trace(4, n_requests=64, n_slots=256, batch=16)
    rounds2, st2 = synth.serving_trace(4, n_requests=64, n_slots=256, batch=16)
    assert st == st2 and [r.store_slots for r in rounds] == [r.store_slots for r in rounds2]
    assert st["stores"] == st["checkpoints_total"] and st["evictions"] > 0 and st["hits"] > 0
    resident = {}
    for r in rounds:
        assert 0 < len(r.store_slots) + len(r.hit_slots) and len(r.store_slots) <= 16 and len(r.hit_slots) <= 16
        assert len(set(r.store_slots)) == len(r.store_slots)            # distinct destination slots in one pack
        assert not set(r.store_slots) & set(r.hit_slots)                # the two sides of a round are independent
        assert all(0 < s < 256 for s in r.store_slots + r.hit_slots)    # slot 0 is reserved
        assert all(s in resident for s in r.hit_slots)                  # a hit reads a slot stored in an earlier round
        assert all(1 <= n <= 1024 for n in r.suffix) and len(r.suffix) == len(r.hit_slots)
        for s in r.store_slots:
            resident[s] = True
