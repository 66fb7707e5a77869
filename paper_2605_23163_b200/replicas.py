"""Multi-GPU plumbing of the benchmark: independent replicas, no data-path collective.

One denoising step does not shard across GPUs (the rollouts of a scene share one prefix cache
in one GPU's memory), so N GPUs decode N independent scenes.  The only communication is the
bookkeeping below: every rank's elapsed time is reduced with MAX, the token counts add up.
The functions take the process group module as an argument so that the same code runs over
NCCL on GPUs and over gloo in the CPU tests.
"""
import torch


def replica_workload(w, rank):
    """The workload of replica `rank`: same shapes, a different seed (a different scene)."""
    if rank == 0:
        return w
    return type(w)(**{**w.__dict__, "seed": w.seed + 100 * rank})


def max_over_ranks(value, dist=None, device="cpu"):
    """MAX of a python float over all ranks (the value itself without a process group)."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, dist=None, device="cpu"):
    """SUM of a python number over all ranks."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
