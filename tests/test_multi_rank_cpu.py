"""world_size-2 gloo test (CPU) of the benchmark's only multi-rank step: max-over-ranks timing and aggregation."""
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_06763_b200 import multi
    ms_local = 0.10 if rank == 0 else 0.25          # rank 1 is the slow one
    value, ms = multi.aggregate_throughput(3072, ms_local)
    out.put((rank, value, ms, multi.reduce_max(float(rank))))
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_max_over_ranks_and_aggregate():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms, mx in res:
        assert abs(ms - 0.25) < 1e-12                # the slowest rank sets the time
        assert abs(value - 2 * 3072 / 0.25e-3) < 1e-3  # both replicas' nodes over that time
        assert mx == 1.0


def test_single_process_is_identity():
    from paper_2607_06763_b200 import multi
    assert multi.reduce_max(3.5) == 3.5
    v, ms = multi.aggregate_throughput(100, 2.0)
    assert ms == 2.0 and abs(v - 100 / 2e-3) < 1e-9
