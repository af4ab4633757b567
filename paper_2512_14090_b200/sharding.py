"""Data-parallel use of the evaluator: every (scheme, image) pair is independent, so the
validation images are split across ranks, each rank counts agreements on its shard with
its own copy of the model, and one sum of the per-scheme integer counts finishes the job.
Only host-side bookkeeping lives here; the counting itself runs in the CUDA library."""
import numpy as np


def shard_bounds(n_items, rank, world_size):
    """Half-open range [lo, hi) of the items rank `rank` owns: contiguous, sizes differ by
    at most one, every item owned exactly once."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, extra = divmod(n_items, world_size)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def reduce_counts(counts, n_local, group=None, device=None):
    """Sum per-scheme correct counts and image totals over all ranks.

    counts: int array [S] of this rank's shard; n_local: images in this rank's shard.
    Returns (global_counts int64 [S], global_n, accuracy float64 [S]).  Uses
    torch.distributed when it is initialised (NCCL needs `device`), else returns the input.
    """
    import torch
    import torch.distributed as dist
    buf = torch.tensor(list(np.asarray(counts, dtype=np.int64)) + [int(n_local)], dtype=torch.int64,
                       device=device if device is not None else "cpu")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
    out = buf.cpu().numpy()
    total = int(out[-1])
    return out[:-1].copy(), total, out[:-1].astype(np.float64) / max(total, 1)
