"""The N > 1 path on CPU: two gloo ranks, each with its own sequences, agree on the
maximum of their times and on the aggregate rate; no other communication exists."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_11236_b200 import sharding
from paper_2510_11236_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = sharding.rank_workload(dict(W.CONFIGS["c0"], seq=64), rank)
        k0, _, _, _ = W.pair_tokens(w, 0, 0, 64, "cpu")
        q = W.queries(w, 0, 0, "cpu")
        local_ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
        dist.barrier()
        ms_max = sharding.max_over_ranks(local_ms)
        rate = sharding.aggregate_rate(1000.0, ms_max, world)
        out.put((rank, w["seed"], float(k0.float().sum()), float(q.float().sum()), ms_max, rate))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_and_time_by_the_slowest():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, k0, q0, ms0, rate0), (r1, seed1, k1, q1, ms1, rate1) = res
    assert (r0, r1) == (0, 1)
    assert seed0 != seed1 and k0 != k1 and q0 != q1      # different sequences on each rank
    assert ms0 == ms1 == 15.0                             # both report the slower rank's time
    assert rate0 == rate1 == 2 * 1000.0 / 15.0e-3         # whole-job rate: both ranks' units over that time


def test_single_process_needs_no_group():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.rank_workload({"seed": 7}, 0)["seed"] == 7
