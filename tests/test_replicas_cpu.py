"""World-size-2 gloo test (CPU) of the multi-GPU bookkeeping: replicas only, barrier + max-over-ranks
timing, aggregate = units of all ranks / slowest rank's time.  No data-path collective exists."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_30379_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world_info() == (rank, world)
        replicas.barrier()
        local_ms = 10.0 if rank == 0 else 25.0          # rank 1 is the slow replica
        assert replicas.max_over_ranks(local_ms) == 25.0
        value = replicas.aggregate_throughput(1000.0, local_ms)
        out.put((rank, value))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    # 2 ranks x 1000 units in 25 ms
    assert abs(res[0] - 80000.0) < 1e-6 and abs(res[1] - 80000.0) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2609_30379_b200 import replicas
    assert replicas.world_info() == (0, 1)
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.aggregate_throughput(100.0, 50.0) == 2000.0
