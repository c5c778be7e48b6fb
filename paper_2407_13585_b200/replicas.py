"""Bookkeeping for runs on several GPUs.

A program's clusters never exchange data between GPUs, so N GPUs run N independent
replicas (one process per GPU).  The only thing the ranks share is the result line:
the job took as long as its slowest rank and moved the bytes of all ranks.
"""


def combine_replicas(ms_local, bytes_local, dist=None, device="cpu"):
    """(slowest rank's milliseconds, bytes summed over ranks).

    `dist` is an initialised torch.distributed module (any backend) or None for a
    single process.  Every rank must call this the same number of times.
    """
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms_local), int(bytes_local)
    import torch
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    b = torch.tensor([int(bytes_local)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), int(b.item())


def effective_gbs(total_bytes, ms):
    """Bytes over milliseconds as GB/s."""
    return total_bytes / (ms * 1e-3) / 1e9
