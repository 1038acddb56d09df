"""Multi-rank host logic on CPU (gloo, world size 2): slots are sharded over ranks with no data-path
collective; only the timing (MAX) and the unit counts (SUM) are reduced.  The second test drives the
launcher `bench.py --gpus N` uses on a GPU node, here with two gloo ranks and a stubbed step."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from paper_2604_11035_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload(0, rank)
    st = wl.make_state(w, "cpu")
    red = bench.reduce_over_ranks(dist, "cpu", [1.0 + rank, 0.5 - 0.1 * rank], [100 * (rank + 1), 7, 3 + rank, 6])
    dist.barrier()
    out.put((rank, w.seed, int(st["block_tok"][0, 0]), red))
    dist.destroy_process_group()


def test_two_ranks_shard_slots_and_reduce_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, tok0, red0), (r1, seed1, tok1, red1) = res
    assert seed0 != seed1                      # independent slots per rank (own pools, own random stream)
    assert red0 == red1                        # every rank sees the same reduced numbers
    assert red0["max"] == [2.0, 0.5]           # slowest rank decides the time
    assert red0["sum"] == [300, 14, 7, 12]     # units of all ranks are added


def test_bench_launcher_starts_the_ranks_itself():
    # `python bench.py --gpus 2` with no WORLD_SIZE in the environment: the script starts two ranks of itself
    # (127.0.0.1 rendezvous), they reduce over gloo, rank 0 prints the one line.  The step is a stub whose
    # duration grows with the rank, so the line shows MAX-over-ranks timing and SUM-over-ranks units.
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-step", "--steps", "4",
                        "--config", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                      # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["stub"] is True
    # each rank "processed" steps * batch * Q positions; rank 1 took 1.25 x as long as rank 0
    per_rank = 4 * 1 * 7
    assert abs(line["ms_per_step"] - 1.25) < 1e-9
    assert abs(line["value"] - 2 * per_rank / (4 * 1.25e-3)) < 1e-6


def test_bench_launcher_single_rank_stub_needs_no_process_group():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--stub-step", "--steps", "2", "--config", "0"],
                       capture_output=True, text=True, timeout=300,
                       env={k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE")})
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads([l for l in p.stdout.splitlines() if l.startswith("{")][0])
    assert line["n_gpus"] == 1 and abs(line["ms_per_step"] - 1.0) < 1e-9
