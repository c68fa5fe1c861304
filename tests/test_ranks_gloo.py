"""World-size-2 gloo test of the benchmark's multi-rank bookkeeping (CPU only)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_13057_b200.ranks import reduce_step
    # every rank builds its own seeded workload: different routed batches, different unit counts
    import bench
    wl = bench.make_workload("cfg1", rank)
    st = bench.workload_stats(wl)
    ms, units = reduce_step(1.0 + rank, float(st["G_act"]))
    q.put((rank, ms, units, st["G_act"], int(wl.topk_ids.sum())))
    dist.destroy_process_group()


def test_reduce_step_takes_max_time_and_sums_units():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == 2.0                       # makespan = slowest rank
    assert res[0][2] == res[1][2] == res[0][3] + res[1][3]     # units add up
    assert res[0][4] != res[1][4]                              # ranks really got different batches


def test_single_rank_passthrough():
    from paper_2608_13057_b200.ranks import reduce_step
    assert reduce_step(3.5, 20.0) == (3.5, 20.0)
