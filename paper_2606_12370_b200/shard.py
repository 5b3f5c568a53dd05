"""Batch sharding across GPUs.  Sequences are independent (Algorithm 3 couples nothing across b), so
rank r of N verifies a contiguous block of the batch with its own kernel launches and there is no
collective on the data path; only timings (a max) or, if one rank wants everything, the few-KB outputs
are exchanged."""
from typing import Optional, Sequence, Tuple


def shard_range(batch: int, rank: int, world: int, draft_len: Optional[Sequence[int]] = None) -> Tuple[int, int]:
    """[begin, end) of the sequences rank `rank` of `world` verifies.

    Without lengths the blocks differ by at most one sequence.  With ragged `draft_len` the cut points
    balance the rows each rank has to read, 2*len_b + 1 per sequence (len_b target/draft pairs plus the
    bonus row), and the blocks stay contiguous and in order."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard request: batch=%d rank=%d world=%d" % (batch, rank, world))
    if draft_len is None:
        base, extra = divmod(batch, world)
        begin = rank * base + min(rank, extra)
        return begin, begin + base + (1 if rank < extra else 0)
    if len(draft_len) != batch:
        raise ValueError("draft_len has %d entries for a batch of %d" % (len(draft_len), batch))
    weights = [2 * int(l) + 1 for l in draft_len]
    total = sum(weights)
    cuts = [0]
    acc, b = 0, 0
    for r in range(1, world):
        want = total * r / world
        while b < batch and acc + weights[b] / 2 <= want:
            acc += weights[b]
            b += 1
        cuts.append(b)
    cuts.append(batch)
    return cuts[rank], cuts[rank + 1]


def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum of a list of floats over all ranks (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]
