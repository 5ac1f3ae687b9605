"""Multi-GPU plumbing for data-parallel replicas of the decode step.

Sequences are independent (every sequence owns its cache pages), so N GPUs run N batches with no
collective on the data path.  The only cross-rank traffic is bookkeeping: a barrier around the
timed region and a max-reduction of the per-rank times, so that a whole-job rate is the work of all
ranks divided by the time of the slowest one.  Works with any torch.distributed backend (nccl on
GPUs, gloo on CPU).
"""
import torch
import torch.distributed as dist


def world():
    """(rank, world_size) of the initialised process group, or (0, 1) without one."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def rank_seed(seed, rank):
    """Seed of a rank's own batch: replicas draw different data from the same recipe."""
    return seed + 100 * rank


def barrier(device='cpu'):
    if world()[1] > 1:
        dist.barrier()
    if str(device).startswith('cuda'):
        torch.cuda.synchronize()


def max_over_ranks(values, device='cpu'):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if world()[1] > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_rate(units_per_rank_per_step, steps, total_ms):
    """Units per second of the whole job: every rank did `units_per_rank_per_step` per step, the job took
    `total_ms` (already the maximum over ranks)."""
    return units_per_rank_per_step * world()[1] * steps / (total_ms * 1e-3)
