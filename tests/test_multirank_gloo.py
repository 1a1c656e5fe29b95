"""The N > 1 path of the benchmark on CPU: two gloo ranks.  Sequences are independent, so the only
cross-rank step is the aggregation of per-rank figures (max of times, sum of counts) and the rule
that every rank draws its own batch."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from workloads import get_config, make_step
    cfg = get_config("cfg1_tiny")
    inp = make_step(cfg, seed=bench.rank_seed(rank))
    # per-rank figures: rank r "took" 1 + r ms and committed 10 + r tokens
    times, counts = bench.reduce_over_ranks([1.0 + rank, 5.0 - rank], [10 + rank], "cpu")
    dist.barrier()
    out.put((rank, times, counts, int(inp["filled"].sum()), inp["logits"][0, 0, :4].tolist(), inp["q"].shape))
    dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_max_time_and_summed_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, counts, _, _, shape in res:
        assert times == [2.0, 5.0]          # max over ranks of each time
        assert counts == [21.0]             # 10 + 11 tokens
        assert shape == res[0][5]           # same shapes on every rank (weak scaling)
    assert res[0][4] != res[1][4]           # but different data


def test_single_process_reduce_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([3.5], [7], "cpu") == ([3.5], [7.0])
    assert bench.rank_seed(0) != bench.rank_seed(1)
