"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank logic: per-rank seeds differ, the reported time is
the maximum over ranks, throughput aggregates all ranks' tokens."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    from paper_2501_14183_b200 import dist_util, inputs
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.WORKLOADS["tiny"]
    x = inputs.make_windows(w, seed=dist_util.rank_seed(w.seed, rank))
    local_ms = [10.0 + 5.0 * rank, 3.0 - rank]
    mx = dist_util.max_over_ranks(local_ms, dist)
    value = dist_util.aggregate_throughput(w.tokens, world, mx[0] * 1e-3)
    gathered = [None] * world
    dist.all_gather_object(gathered, float(x.sum()))
    if rank == 0:
        out.put((mx, value, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    mx, value, sums = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert mx == [15.0, 3.0]
    from paper_2501_14183_b200 import inputs
    assert abs(value - inputs.WORKLOADS["tiny"].tokens * 2 / 15e-3) < 1e-6
    assert sums[0] != sums[1]                       # ranks work on different batches


def test_single_process_identity():
    from paper_2501_14183_b200 import dist_util
    assert dist_util.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert dist_util.rank_seed(7, 3) == 3007
