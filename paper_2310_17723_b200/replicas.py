"""Host-side logic of the multi-GPU run: the layer shards by sequence (per-token scales, static calibrated
scales, per-sequence attention, read-only weights), so N GPUs are N replicas working on their own batches with
no exchange step.  What the ranks share is only the clock: a barrier on both sides of the timed region and the
maximum of their device times."""
import os


def rank_info():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")))


def batch_tensor_index(rank):
    """Which seeded activation tensor a rank draws: every replica gets its own batch."""
    return 2 + 10 * rank


def max_over_ranks(value, dist=None, device="cpu"):
    """The slowest rank's time decides the job's throughput."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_per_step, steps, world, seconds_max):
    """Whole-job units per second: every rank processed its own units in the slowest rank's time."""
    return world * units_per_rank_per_step * steps / seconds_max
