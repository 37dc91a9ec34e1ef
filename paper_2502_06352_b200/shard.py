"""Partition of a batch of sequences over ranks.

Verification of one sequence's tree never needs another sequence's data, so ranks
split the batch and exchange nothing on the data path; only timings are reduced.
"""


def shard_range(total, rank, world):
    """Half-open range [begin, end) of the `total` items that `rank` of `world` owns.

    Contiguous, disjoint, covering; sizes differ by at most one (lower ranks take
    the remainder)."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard request")
    base, rem = divmod(total, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def whole_job_rate(units_per_rank, elapsed_ms_max):
    """Aggregate rate (units / s) of a job whose ranks each processed
    units_per_rank[r] units and whose slowest rank took elapsed_ms_max."""
    return sum(units_per_rank) / (elapsed_ms_max * 1e-3)
