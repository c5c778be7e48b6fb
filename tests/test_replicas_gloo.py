"""Multi-GPU runs are independent replicas; what the ranks combine is the result line.
Two gloo ranks on CPU check that combination: slowest rank's time, bytes of all ranks."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2407_13585_b200.replicas import combine_replicas, effective_gbs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, total = combine_replicas(2.0 + rank, 1000 * (rank + 1), dist)
    dist.barrier()
    if rank == 0:
        out.put((ms, total, effective_gbs(total, ms)))
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_all_bytes():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 2, 29517, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, total, gbs = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert ms == 3.0 and total == 3000
    assert abs(gbs - 3000 / 3.0e-3 / 1e9) < 1e-12


def test_single_process_passes_through():
    sys.path.insert(0, ROOT)
    from paper_2407_13585_b200.replicas import combine_replicas
    assert combine_replicas(1.5, 42) == (1.5, 42)
