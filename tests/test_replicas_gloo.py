"""The N > 1 path of the benchmark is "replicas only": ranks share nothing but the timing
reduction.  Two gloo ranks on CPU check that reduction (max over ranks, work summed)."""
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
    from paper_2309_12307_b200.replicas import slowest_rank_ms, whole_job_rate

    local_ms = 10.0 if rank == 0 else 12.5          # rank 1 is the slow one
    slow = slowest_rank_ms(local_ms)
    rate = whole_job_rate(units_per_rank=7.0e12, local_ms=local_ms)
    dist.barrier()
    out.put((rank, slow, rate))
    dist.destroy_process_group()


def test_two_rank_timing_reduction():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, slow, rate in results:
        assert slow == 12.5
        assert abs(rate - 2 * 7.0e12 / 12.5e-3) < 1e3


def test_single_process_is_identity():
    from paper_2309_12307_b200.replicas import slowest_rank_ms, whole_job_rate

    assert slowest_rank_ms(3.0) == 3.0
    assert whole_job_rate(6.0, 2.0) == 3000.0
