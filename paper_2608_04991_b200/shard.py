"""Token sharding across ranks (one process per GPU).

Tokens are independent units for encode and reconstruct, and the wire payload is token-major, so a rank's
share is a contiguous token range and a contiguous byte range of the payload.  No collective is needed on the
data path; the helpers below only compute the ranges.
"""
from __future__ import annotations

from typing import List, Optional, Tuple


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


def all_gather_ranges(buf, ranges: List[Tuple[int, int]], rank: int, group=None) -> None:
    """Every rank holds its own byte range [ranges[rank]) of `buf` (a 1-D uint8 tensor of the full length, in this
    rank's OWN memory); on return every rank holds all ranges.  The ranges must tile [0, len(buf)) in rank order.
    Equal ranges go through one in-place all-gather; unequal ones (a token count that the world size does not
    divide) are padded to the largest.  Nothing but `torch.distributed` touches another rank's memory."""
    import torch
    import torch.distributed as dist
    world = len(ranges)
    if world == 1:
        return
    assert ranges[0][0] == 0 and ranges[-1][1] == buf.numel() and all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    sizes = [hi - lo for lo, hi in ranges]
    lo, hi = ranges[rank]
    if len(set(sizes)) == 1 and dist.get_backend(group) == "nccl":
        dist.all_gather_into_tensor(buf, buf[lo:hi], group=group)
        return
    biggest = max(sizes)
    mine = torch.zeros(biggest, dtype=buf.dtype, device=buf.device)
    mine[: hi - lo] = buf[lo:hi]
    got = [torch.empty(biggest, dtype=buf.dtype, device=buf.device) for _ in range(world)]
    dist.all_gather(got, mine, group=group)
    for r, (a, b) in enumerate(ranges):
        if r != rank:
            buf[a:b] = got[r][: b - a]


def sharded_encode(encode_range, T: int, record_bytes: int, payload, rank: int, world: int, group=None) -> Tuple[int, int]:
    """One tensor of T tokens coded by `world` ranks: this rank calls `encode_range(a, b)` for its contiguous token
    range (the callback writes the records of tokens [a, b) into payload[a*record_bytes : b*record_bytes]), then the
    byte ranges are exchanged so that every rank holds the whole payload.  Returns the rank's token range."""
    a, b = token_range(T, rank, world)
    if b > a:
        encode_range(a, b)
    all_gather_ranges(payload, [payload_range(record_bytes, x, y) for x, y in all_ranges(T, world)], rank, group)
    return a, b
