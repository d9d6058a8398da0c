"""Sharding of one tensor across ranks (one process per GPU).

Chunks (1024 elements) are independent units of the stream and a chunk boundary
is a window boundary, so a tensor can be cut at chunk boundaries, each rank can
compress its own range into its own payload and offset table, and the single
stream of the whole tensor is simply the concatenation of the rank payloads in
rank order.  The only thing the ranks exchange is one integer each (their
payload size) to turn local table entries into global ones -- there is no
collective on the data path.

Host-side bookkeeping only; holds no codec arithmetic.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

CHUNK = 1024


def partition(n: int, world: int) -> List[Tuple[int, int]]:
    """Chunk-aligned element ranges [lo, hi) per rank, as even as possible.
    Ranks past the last chunk get empty ranges."""
    if world < 1:
        raise ValueError("world must be >= 1")
    chunks = (n + CHUNK - 1) // CHUNK
    base, extra = divmod(chunks, world)
    out, c = [], 0
    for r in range(world):
        take = base + (1 if r < extra else 0)
        lo = min(c * CHUNK, n)
        hi = min((c + take) * CHUNK, n)
        out.append((lo, hi))
        c += take
    return out


def exclusive_offsets(sizes: Sequence[int]) -> List[int]:
    """Byte offset of every rank's payload in the concatenated stream."""
    out, acc = [], 0
    for s in sizes:
        out.append(acc)
        acc += int(s)
    return out


def gather_payload_sizes(local_bytes: int, group=None) -> List[int]:
    """All ranks' payload sizes (one int64 each) via torch.distributed."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    mine = torch.tensor([int(local_bytes)], dtype=torch.int64)
    backend = dist.get_backend(group)
    if backend == "nccl":
        mine = mine.cuda()
    got = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(got, mine, group=group)
    return [int(t.item()) for t in got]


def globalize_table(local_table, rank_offset: int, is_last: bool):
    """Local table (numpy uint64, K_r+1 entries) -> this rank's slice of the
    global table.  Every rank drops its closing entry except the last rank,
    whose closing entry becomes the global payload size."""
    t = local_table + local_table.dtype.type(rank_offset)
    return t if is_last else t[:-1]
