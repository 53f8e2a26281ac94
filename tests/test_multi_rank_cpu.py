"""The N > 1 path on CPU: two gloo ranks run the benchmark's rank-aggregation (whole-job
elapsed time = max over ranks, units = sum over ranks) and the replica seeding, with no GPU."""

import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from synth_inputs import WORKLOADS, Synth
    import dataclasses
    # each rank is an independent replica with its own seeded batch
    wl = dataclasses.replace(WORKLOADS["tiny"], V=512)
    z, d = Synth(wl, seed=rank, device="cpu").step(0)
    dist.barrier()
    sec, units = bench.reduce_over_ranks(0.25 * (rank + 1), 1000.0 * (rank + 1), dist, torch.device("cpu"))
    out.put((rank, sec, units, float(z.float().sum()), d.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, u0, z0, d0), (r1, s1, u1, z1, d1) = res
    assert s0 == s1 == 0.5 and u0 == u1 == 3000.0          # max of times, sum of units, same on every rank
    assert z0 != z1                                          # replicas draw different batches


def test_single_rank_is_identity():
    import bench
    assert bench.reduce_over_ranks(1.5, 7.0) == (1.5, 7.0)
