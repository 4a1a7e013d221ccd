"""Which tensors of a role to materialise for a run of whole buckets.

The library cuts a role into runs of whole buckets itself (tm_plan_create_range, tm_xfer_*).  A role
whose state does not fit one GPU at all — the 200 000-tensor adversarial set is about 257 GB — also
needs its *inputs* generated run by run; this module tells the input generators which tensors, and
which byte range of a tensor that straddles a cut, belong to each run.  Buckets are independent
units (each has its own checksum, word index restarting at 0), and a cut lies on a multiple of the
bucket size, hence of 256, so the runs' streams and checksum lists concatenate to the complete ones.

`offsets` are the stream offsets of the complete descriptor list as reported by the planner
(`Plan.offsets()`); this module only compares them with multiples of the bucket size.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple


@dataclasses.dataclass(frozen=True)
class Part:
    tensor: int       # index in the complete descriptor list
    byte_start: int   # first byte of the tensor that belongs to this wave
    nbytes: int


@dataclasses.dataclass(frozen=True)
class Wave:
    first_bucket: int
    n_buckets: int            # whole buckets, except that the last wave may end with a short bucket
    stream_begin: int         # offset of the wave in the complete stream
    stream_end: int
    parts: Tuple[Part, ...]


def cut_waves(sizes: Sequence[int], offsets: Sequence[int], total_bytes: int, bucket_bytes: int,
              budget_bytes: int) -> List[Wave]:
    """Greedy cut: every wave takes as many whole buckets as fit in `budget_bytes` of stream."""
    per_wave = max(1, budget_bytes // bucket_bytes)
    n_buckets = -(-total_bytes // bucket_bytes)
    waves: List[Wave] = []
    k = 0  # first tensor that may intersect the current wave
    for first in range(0, n_buckets, per_wave):
        count = min(per_wave, n_buckets - first)
        lo, hi = first * bucket_bytes, min((first + count) * bucket_bytes, total_bytes)
        parts: List[Part] = []
        while k < len(sizes) and offsets[k] + sizes[k] <= lo:
            k += 1
        j = k
        while j < len(sizes) and offsets[j] < hi:
            a, b = max(lo, offsets[j]), min(hi, offsets[j] + sizes[j])
            if a < b:
                parts.append(Part(j, a - offsets[j], b - a))
            j += 1
        waves.append(Wave(first, count, lo, hi, tuple(parts)))
    return waves
