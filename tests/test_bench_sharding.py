"""Host-side logic of the multi-GPU bench (one independent session per rank, no data-path collective),
exercised with two gloo ranks on the CPU."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    local = {"ms": 10.0 + 5 * rank, "bytes": 1000.0 * (rank + 1), "hashed": 7.0, "launches": 50 + rank}
    tot = bench.reduce_over_ranks(local, dist, "cpu")
    setup, turns, _ = bench.make_turns(1 + rank, 6)
    first_tokens = int(turns[0][0][0][2][0])
    out.put((rank, tot, len(turns), first_tokens))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_and_get_different_sessions():
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
    for _rank, tot, _n, _t in res:
        assert tot["ms"] == 15.0             # slowest rank
        assert tot["bytes"] == 3000.0        # units of all ranks
        assert tot["hashed"] == 14.0 and tot["launches"] == 101.0
    assert res[0][3] != res[1][3]            # each rank replays its own seeded session


def test_single_rank_passthrough():
    import bench
    assert bench.reduce_over_ranks({"ms": 3.0, "bytes": 5.0}) == {"ms": 3.0, "bytes": 5.0}


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_turn_split_covers_the_trace():
    import bench
    from paper_2609_39819_b200 import workloads as W
    trace = W.trace_c2(1, scale=1 / 32)
    setup, turns = bench.split_turns(trace)
    n_events = len(setup) + sum(len(pre) + 1 + len(post) for pre, _c, post in turns)
    assert n_events == len(trace) and all(len(post) == 1 and post[0][0] == "remove" for _p, _c, post in turns)
