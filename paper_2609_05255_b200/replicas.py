"""Host-side logic of a multi-GPU run.  Views of a training step are independent and a view does not
shard without an all-to-all of the instance lists, so N GPUs run N replicas of the step ("replicas
only"): no collective is on the data path.  What the ranks exchange is the timing only - a barrier on
both sides of the timed region and the maximum of the per-rank step times.

Nothing here touches a GPU API directly: `device` is whatever the process group's backend reduces on
(a CUDA device under NCCL, the CPU under gloo), which is how the tests run it with two CPU ranks."""
import os


def rank_env():
    """(rank, world_size, local_rank) as torch.distributed.run exports them; (0, 1, 0) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend, world, device=None):
    """Join the job's process group (no-op for a single rank).  The rendezvous address comes from the
    launcher's MASTER_ADDR / MASTER_PORT."""
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kw)
    return dist


def barrier(dist):
    if dist is not None:
        dist.barrier()


def max_over_ranks(value, dist, device):
    """Slowest rank's value, on every rank."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, dist, device):
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_ms_per_iteration(slowest_ms, iterations_per_rank_step, total_iterations_per_step):
    """Whole-job time per training iteration when every rank finishes `iterations_per_rank_step`
    iterations in `slowest_ms` (the max over ranks) and the job `total_iterations_per_step` of them."""
    return slowest_ms * iterations_per_rank_step / total_iterations_per_step
