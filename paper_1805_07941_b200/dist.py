"""Multi-GPU plumbing: one process per GPU, images sharded over ranks.

Inference needs no exchange (images are independent, weights and tables are replicated).  The one
exchange of the method is in calibration, when the calibration batch itself is split over ranks: the
threshold of a tensor is its maximum |x| over the WHOLE batch (Section 3 of the paper), so ranks
combine their partial statistics before choosing the exponent -- MAX of the maxima, SUM of counts,
sums and (when all ranks used the same fixed range) histogram bins.  A few KB per layer; it goes
through torch.distributed (NCCL on GPUs, gloo in the CPU tests).
"""
import numpy as np
import torch
import torch.distributed as dist


def shard_range(total, rank, world):
    """Contiguous share [lo, hi) of `total` items for `rank` of `world` (sizes differ by at most 1)."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_calib(stats, group=None, device="cpu"):
    """Combine per-rank calibration statistics (dicts as returned by qcalib_collect) into those of the
    union of the shards.  Histograms are summed only if every rank binned over the same range
    (a fixed range_hi); with per-rank automatic ranges the combined histogram is dropped (None)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return dict(stats)
    mx = torch.tensor([float(stats["maxabs"]), float(stats["range_hi"]), -float(stats["range_hi"])],
                      dtype=torch.float64, device=device)
    dist.all_reduce(mx, op=dist.ReduceOp.MAX, group=group)
    same_range = (mx[1].item() == -mx[2].item())
    sums = torch.tensor([stats["sum"], stats["sumsq"]], dtype=torch.float64, device=device)
    dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
    counts = torch.tensor([stats["count"], stats["nonfinite"]], dtype=torch.int64, device=device)
    dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    out = dict(maxabs=np.float32(mx[0].item()), range_hi=np.float32(mx[1].item()), count=int(counts[0].item()),
               nonfinite=int(counts[1].item()), sum=float(sums[0].item()), sumsq=float(sums[1].item()), hist=None)
    if same_range:
        h = torch.from_numpy(stats["hist"].astype(np.int64)).to(device)
        dist.all_reduce(h, op=dist.ReduceOp.SUM, group=group)
        out["hist"] = h.cpu().numpy().astype(np.uint64)
    return out


def collect_synced(collect, group=None, device="cpu"):
    """Statistics of the union of the shards INCLUDING the histogram (what the threshold search needs).
    collect(range_hi) returns this rank's statistics binned on [0, range_hi], or on its own maximum when
    range_hi is 0.  First pass: the maximum over all ranks; second pass: every rank bins on that common
    range, so the bins add up exactly to those of the whole batch."""
    first = collect(0.0)
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return first
    gmax = max_over_ranks(float(first["maxabs"]), group, device)
    if not gmax > 0.0:                                       # all zeros everywhere: nothing to bin
        first = dict(first)
        first["range_hi"] = np.float32(0.0)
        return allreduce_calib(first, group, device)
    second = dict(collect(gmax))
    second["range_hi"] = np.float32(gmax)
    return allreduce_calib(second, group, device)


def max_over_ranks(value, group=None, device="cpu"):
    """Largest `value` (a float, e.g. elapsed milliseconds) over the ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def whole_job_rate(units_per_rank, steps, elapsed_ms, group=None, device="cpu"):
    """Units all ranks processed divided by the slowest rank's time."""
    world = dist.get_world_size(group) if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank * steps / (max_over_ranks(elapsed_ms, group, device) * 1e-3)
