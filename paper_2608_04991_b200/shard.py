"""Token sharding across ranks (one process per GPU).

Tokens are independent units for encode and reconstruct, and the wire payload is token-major, so a rank's
share is a contiguous token range and a contiguous byte range of the payload.  No collective is needed on the
data path; the helpers below only compute the ranges.
"""
from __future__ import annotations

from typing import List, Tuple


def token_range(T: int, rank: int, world: int) -> Tuple[int, int]:
    """[start, stop) of the tokens rank `rank` codes: contiguous, sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or T < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(T, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def payload_range(record_bytes: int, start: int, stop: int) -> Tuple[int, int]:
    """Byte range of tokens [start, stop) in a token-major payload."""
    return start * record_bytes, stop * record_bytes


def all_ranges(T: int, world: int) -> List[Tuple[int, int]]:
    return [token_range(T, r, world) for r in range(world)]
