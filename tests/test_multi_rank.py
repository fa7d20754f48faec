"""The benchmark's multi-rank logic on CPU: two gloo ranks, no GPU.  The path shards over independent
batches with no data-path collective; what ranks share is only the timing reduction."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    import workloads as W
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        w = bench.rank_workload(W.get_workload("llama3_8b"), rank, world)
        lens = W.seq_lens(w)
        # every rank's timing is the maximum over ranks, whoever was slowest
        times = bench.max_over_ranks([10.0 + rank, 5.0 - rank], world, torch.device("cpu"))
        q.put((rank, w.seed, lens.tolist(), (w.n_layers, w.q_heads, w.kv_heads, w.batch), times))
    finally:
        dist.destroy_process_group()


def test_two_ranks_get_their_own_batches_and_the_slowest_rank_sets_the_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, lens0, shape0, t0), (r1, seed1, lens1, shape1, t1) = got
    assert (r0, r1) == (0, 1)
    assert shape0 == shape1 and seed0 != seed1 and lens0 != lens1          # same shape, different data
    assert len(lens0) == len(lens1) and all(1024 <= n <= 4096 for n in lens0 + lens1)
    assert t0 == t1 == [11.0, 5.0]


def test_one_rank_is_the_identity_and_rates_add_up_over_ranks():
    sys.path.insert(0, ROOT)
    import bench
    import workloads as W
    w = W.get_workload("llama3_8b")
    assert bench.rank_workload(w, 0, 1) is w
    assert bench.max_over_ranks([3.0, 4.0], 1, torch.device("cpu")) == [3.0, 4.0]
    # weak scaling: N ranks doing the same per-rank work in the same time give N times the rate
    one = bench.whole_job_rate(1e9, 10, 20.0, 1)
    assert one == 1e9 * 10 / 0.020
    assert bench.whole_job_rate(1e9, 10, 20.0, 4) == 4 * one
