"""Host-side data parallelism: users are independent units of the path, so a batch is split by user across
ranks (one process per GPU) and no rank ever needs another rank's data; results are concatenated in rank order."""
from __future__ import annotations

import numpy as np


def user_shard(num_users: int, rank: int, world_size: int) -> range:
    """Users [lo, hi) owned by `rank`: contiguous blocks whose sizes differ by at most one."""
    if world_size < 1 or not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, rem = divmod(int(num_users), world_size)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))


def shard_batch_arrays(items, lengths, cands, cand_offsets, rank: int, world_size: int):
    """Slice a batch (numpy or torch arrays) to the users of `rank`.

    Returns (items_r, lengths_r, cands_r, cand_offsets_r, cand_range) where cand_offsets_r starts at 0 and
    cand_range = (first, last) locates the shard's candidates (rows of z / H') in the full batch."""
    us = user_shard(len(lengths), rank, world_size)
    lo, hi = us.start, us.stop
    c0, c1 = int(cand_offsets[lo]), int(cand_offsets[hi])
    offs = cand_offsets[lo:hi + 1] - cand_offsets[lo]
    return items[lo:hi], lengths[lo:hi], cands[c0:c1], offs, (c0, c1)
