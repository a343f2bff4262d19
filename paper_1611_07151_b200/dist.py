"""Data-parallel plumbing: images of a batch are independent, so the forward shards by
image with no collective on the data path.  Only timing is reduced across ranks."""
import os


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment (1 process: 0, 0, 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def shard(total, rank, world):
    """Contiguous share [lo, hi) of `total` images for `rank`; sizes differ by at most one."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def init(backend):
    """Initialise torch.distributed from the environment when WORLD_SIZE > 1; returns world size."""
    import torch.distributed as dist
    rank, _local, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def reduce_scalar(value, op="max", device="cpu"):
    """max or sum of a float over all ranks (identity in a single process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_local, ms_local, device="cpu"):
    """Whole-job units/s: units summed over ranks / the slowest rank's time."""
    units = reduce_scalar(units_local, "sum", device)
    ms = reduce_scalar(ms_local, "max", device)
    return units / (ms * 1e-3), ms
